#!/usr/bin/env python
"""Benchmark of the KV-cache compression event (fused alpha_compress_event).

One *step* = one pass of the whole hot path (score -> greedy selection -> ordering -> in-place
compaction) over one batch of synthetic input. The default workload, and the one the headline
metric is quoted on, is C3: Llama-8B-shaped, batch 16 x 32 layers x 8 KV heads = 4096 events,
N = 192 -> b = 64, d = 128, bf16, lambda = 0.5, 5 % near-duplicate V rows. `--config` times the
other four configurations the same way (C4: one step = the batch at lambda 0, 0.5 and 1.0;
C5: one step = the 32 events of the decode cadence, the refill between them outside the timed
regions). Prints one JSON line.

    python bench.py [--config C3] [--gpus N] [--steps K] [--warmup W] [--impl reference]

N > 1 is launched by torch.distributed.run: events are independent, so every rank processes
its own batch (weak scaling, no data-path collective); the time is the max over ranks.
`--impl reference` times the CPU oracle on the host cores instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "compression events/sec (all layers x KV heads)"
UNIT = "events/s"
L2_BYTES = 126 * 1024 * 1024

WORKLOADS = {
    "C1": "C1 single (layer, KV head): N=192 -> b=64, d=128, fp32, lambda=0.5",
    "C2": "C2 Qwen-7B-shaped: batch 1 x 28 layers x 4 KV heads, N=256 -> b=128, d=128, bf16, lambda=0.5",
    "C3": "C3 Llama-8B-shaped: batch 16 x 32 layers x 8 KV heads, N=192 -> b=64, d=128, bf16, lambda=0.5",
    "C4": "C4 large pool: batch 8 x 28 layers x 4 KV heads, N=4096 -> b=128, d=128, bf16, lambda in {0, 0.5, 1.0}",
    "C5": "C5 decode cadence: batch 64 x 32 layers x 8 KV heads, 32 events of N=256 -> b=128 in a paged buffer, "
          "d=128, bf16, lambda=0.5",
    "C6": "C6 flat signature (Eq. 1) with one cosine matrix per sequence: Qwen-7B shape, batch 16 x 28 layers x 4 KV heads, "
          "N=256 -> b=128, d=128, bf16, lambda=0.5; a step = signature pass + cosine matrix + fused events",
}
# kernel(s) one call of the fused entry point launches for each workload
KERNELS = {"C1": "event_resident_kernel<float>", "C2": "event_pool_kernel<fused>", "C3": "event_tri_kernel<fused>",
           "C4": "event_stream_kernel", "C5": "event_pool_kernel<fused>",
           "C6": "flat_signature_kernel + gram_shared_kernel + event_pool_kernel<fused>"}

# dram__bytes_read.sum + dram__bytes_write.sum per step from the ncu captures summarised under profiles/,
# keyed by workload, each with the source revision of csrc/ it was taken at (see kernel_revision()); a
# capture of another revision is reported as null.
NCU_TRAFFIC = {
    # one launch of 4096 events captured whole (profiles/event_tri_kernel_bf16_C3.md)
    "C3": {"bytes": 323675904 + 98740992, "revision": "2ef03d00f108"},
    # one launch of 4096 events (16 sequences) captured; a step is 4 x 32 launches of that size
    # (profiles/event_pool_kernel_bf16_C5.md)
    "C5": {"bytes": (489861376 + 230915584) * 128, "revision": "2ef03d00f108"},
    # the same kernel and capture, scaled to 112 events
    "C2": {"bytes": (489861376 + 230915584) * 112 // 4096, "revision": "2ef03d00f108"},
    # the three launches (lambda 0, 0.5, 1) of a 2-sequence batch captured; the bench batch has 8 sequences
    # (profiles/event_stream_kernel_bf16_C4.md)
    "C4": {"bytes": ((249109504 + 12716032) + (256418560 + 10868480) + (256417536 + 11575296)) * 4, "revision": "2ef03d00f108"},
}


def algorithmic_bytes(N, b, d, esize):
    """HBM bytes one event has to move: read K and V once, write b rows of each, positions in, positions and
    indices out, the query statistic."""
    return 2 * N * d * esize + 2 * b * d * esize + 4 * N + 8 * b + 4 * d


def kernel_revision():
    """Hash of the CUDA sources: ties a stored ncu traffic figure to the kernels it was measured on."""
    import glob
    import hashlib
    h = hashlib.sha1()
    for p in sorted(glob.glob(os.path.join(ROOT, "paper_2605_14292_b200", "csrc", "*"))):
        with open(p, "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:12]


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Polls SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.002):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self.period = period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def reduce_max(value: float, world: int, device) -> float:
    """Max over ranks of a host scalar (no-op for one rank)."""
    if world == 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def events_per_second(events_per_rank: int, world: int, steps: int, total_ms: float) -> float:
    return events_per_rank * world * steps / (total_ms * 1e-3)


# ------------------------------------------------------------------------------------------------ CPU oracle legs
def oracle_sample(config: str, seed: int = 0):
    """A bounded sample of the workload for the CPU oracle: (batch, lambdas, description). The oracle runs
    whole events of the same seeded recipe; C4 and C5 take a subset of the sequences (C5: its first event)."""
    from paper_2605_14292_b200 import synth
    if config == "C1":
        return synth.make_c1(seed), [0.5], "the single event, 20 repetitions", 20
    if config == "C2":
        return synth.make_c2(seed), [0.5], "all 112 events once", 1
    if config == "C3":
        return synth.make_c3(seed, B=2), [0.5], "512 of 4096 events (batch 2 of 16)", 1
    if config == "C4":
        return synth.make_c4(seed, B=1, L=4, H=4), [0.0, 0.5, 1.0], "16 of 896 events (4 layers of one sequence) at each of the three lambdas", 1
    if config == "C6":
        return synth.make_c2(seed, B=1), [0.5], "112 of 1792 events (batch 1 of 16), flat signatures", 1
    c5 = synth.make_c5(seed, B=2, rounds=1)
    K = synth.paged_gather_dense(c5.pool_K, c5.block_table)
    V = synth.paged_gather_dense(c5.pool_V, c5.block_table)
    ev = synth.EventBatch("C5-round0", synth.BF16, K, V, c5.pos, c5.qstat, np.full((2,), 256, dtype=np.int32), c5.budget, c5.lam)
    return ev, [0.5], "512 of 16384 events (batch 2 of 64), the first of the 32 events only", 1


def oracle_time(ev, lams, reps=1, threads=None, min_seconds=0.0):
    """Times the C oracle, as it stands, on whole events of `ev` with `threads` host threads: `reps` passes
    over the sample, repeated until `min_seconds` of wall time have gone by. Returns events/s, threads, seconds
    and the events processed."""
    from oracle import c_oracle as CO
    threads = threads or (os.cpu_count() or 1)
    CO.build()
    E = ev.n_events
    CO.event_batch(ev.K, ev.V, ev.pos, ev.qstat, ev.p_ref, ev.budget, lams[0], events=(0, min(E, threads)), threads=threads)
    done = 0
    t0 = time.perf_counter()
    while True:
        for _ in range(reps):
            for lam in lams:
                CO.event_batch(ev.K, ev.V, ev.pos, ev.qstat, ev.p_ref, ev.budget, lam, threads=threads)
        done += E * reps * len(lams)
        dt = time.perf_counter() - t0
        if dt >= min_seconds:
            break
    return done / dt, threads, dt, done


def flat_oracle_time(ev, lams):
    """The NumPy oracle with Eq. 1's flat signature (the C twin has per-head signatures only), one process."""
    from oracle import alpha_oracle as O
    B, L, H, N, d = ev.shape
    t0 = time.perf_counter()
    for lam in lams:
        for b in range(B):
            sig = O.signatures_flat(ev.V[b])
            for l in range(L):
                for h in range(H):
                    O.compress_event(ev.K[b, l, h], ev.V[b, l, h], ev.pos[b, l, h], ev.qstat[l, h], int(ev.p_ref[b]),
                                     ev.budget, lam, sig=sig)
    dt = time.perf_counter() - t0
    return ev.n_events * len(lams) / dt, 1, dt


def cpu_baseline(config: str):
    ev, lams, what, reps = oracle_sample(config)
    if config == "C6":
        v, threads, dt = flat_oracle_time(ev, lams)
        return {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle",
                "sample": f"{what}, NumPy oracle in float64, {dt:.1f} s wall in one process",
                "single_thread": {"value": v, "events": ev.n_events, "wall_s": round(dt, 2)}}
    v, threads, dt, done = oracle_time(ev, lams, reps, min_seconds=10.0)
    # one thread on a smaller slice of the same sample
    one = ev
    if ev.n_events > 32:
        from paper_2605_14292_b200 import synth
        one = synth.EventBatch(ev.name, ev.dtype, ev.K[:1, :2], ev.V[:1, :2], ev.pos[:1, :2], ev.qstat[:2], ev.p_ref[:1],
                               ev.budget, ev.lam)
    v1, _, dt1, done1 = oracle_time(one, lams, reps, threads=1, min_seconds=5.0)
    return {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{what}, repeated to {done} events, C oracle in float64, {dt:.1f} s wall on {threads} threads",
            "single_thread": {"value": v1, "events": done1, "wall_s": round(dt1, 2)}}


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    ev, lams, what, reps = oracle_sample(args.config)
    threads = os.cpu_count() or 1
    # a step repeats the sample for about a second (less when many steps are asked for: the whole run stays
    # within two minutes or so)
    per_step = min(1.0, 100.0 / max(args.steps + args.warmup, 1))
    if args.config == "C6":
        threads = 1
        work = lambda: flat_oracle_time(ev, lams)
    else:
        work = lambda: oracle_time(ev, lams, reps, threads, min_seconds=per_step)
    events = 0
    for _ in range(args.warmup):
        work()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        r = work()
        events += r[3] if len(r) > 3 else ev.n_events * len(lams)
    dt = time.perf_counter() - t0
    value = events / dt
    sample = (f"per step: {what}, repeated for {per_step:.2f} s, {'NumPy' if args.config == 'C6' else 'C'} oracle in float64, "
              f"{threads} threads")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOADS[args.config], "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------ GPU workloads
class DenseWorkload:
    """C1-C4: a dense batch [B, L, H, N, d]; one step = one fused call per lambda, each on a pristine copy of
    the batch (the event rewrites its inputs). Pristine copies are restored outside the timed regions."""

    def __init__(self, config, rank, dev, steps, akv, synth, torch, batch=None):
        self.akv, self.torch = akv, torch
        make = {"C1": synth.make_c1, "C2": synth.make_c2, "C3": synth.make_c3, "C4": synth.make_c4, "C6": synth.make_c2}[config]
        if config == "C6" and batch is None:
            batch = 16
        ev = make(seed=rank) if batch is None or config == "C1" else make(seed=rank, B=batch)
        self.flat = config == "C6"
        self.ev = ev
        self.lams = [0.0, 0.5, 1.0] if config == "C4" else [ev.lam]
        B, L, H, N, d = ev.shape
        self.esize = 2 if ev.dtype == synth.BF16 else 4
        self.events_per_step = ev.n_events * len(self.lams)
        self.bytes_per_step = algorithmic_bytes(N, ev.budget, d, self.esize) * self.events_per_step
        if self.flat:   # the shared signatures and their cosine matrix, written once and read once per sequence
            self.bytes_per_step += 2 * B * (N * d * 4 + N * N * 4)
        self.launches_hint = len(self.lams)
        self.LH = L * H
        self.K0, self.V0, self.P0 = akv.to_device(ev.K, dev), akv.to_device(ev.V, dev), akv.to_device(ev.pos, dev)
        self.q, self.pref = akv.to_device(ev.qstat, dev), akv.to_device(ev.p_ref, dev)
        set_bytes = (self.K0.numel() + self.V0.numel()) * self.esize
        self.set_bytes = set_bytes
        # how many steps run back to back inside one timed region: bounded by 24 steps and ~40 GB of copies
        per_step = set_bytes * len(self.lams)
        self.group = max(1, min(steps, 24, int(40e9 // max(per_step, 1))))
        self.bufs = [(torch.empty_like(self.K0), torch.empty_like(self.V0), torch.empty_like(self.P0))
                     for _ in range(self.group * len(self.lams))]
        self.sel = akv.api._alloc_sel(akv.Layout.dense(self.K0), ev.budget, dev, detail=False)
        self.opts = [akv.Options(lam=lam) for lam in self.lams]
        if self.flat:
            self.sig = torch.empty((B, N, d), dtype=torch.float32, device=dev)
            self.gram = torch.empty((B, N, N), dtype=torch.float32, device=dev)
            self.opts = [akv.Options(lam=lam, sig_mode=akv.SIG_FLAT, shared_gram=self.gram) for lam in self.lams]
        self.flush = None
        if per_step * self.group < 2 * L2_BYTES:       # working set may stay in L2: evict it before each region
            self.flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev)
        self.l2 = (f"inputs larger than L2 ({set_bytes / 1e6:.0f} MB per call, fresh copy per call)" if self.flush is None
                   else f"L2 flushed (a {2 * L2_BYTES >> 20} MiB buffer written) before every timed region; "
                        f"{set_bytes / 1e6:.2f} MB per call, fresh copy per call")

    def prepare(self, k):
        for i in range(k * len(self.lams)):
            self.bufs[i][0].copy_(self.K0); self.bufs[i][1].copy_(self.V0); self.bufs[i][2].copy_(self.P0)
        if self.flush is not None:
            self.flush.fill_(1)

    def call(self, Kb, Vb, Pb, o, sel):
        akv = self.akv
        if self.flat:   # Eq. 1 over all layers and heads, its cosine matrix once per sequence, then the events
            akv.alpha_signature_flat(Vb, o, out=self.sig)
            akv.alpha_gram_shared(self.sig, akv.Layout.dense(Vb), o, out=self.gram)
            akv.alpha_compress_event(Kb, Vb, Pb, self.q, self.ev.budget, o, p_ref=self.pref, flat_sig=self.sig, out=sel)
        else:
            akv.alpha_compress_event(Kb, Vb, Pb, self.q, self.ev.budget, o, p_ref=self.pref, out=sel)

    def step(self, i):
        for j, o in enumerate(self.opts):
            Kb, Vb, Pb = self.bufs[i * len(self.lams) + j]
            self.call(Kb, Vb, Pb, o, self.sel)

    def timed(self, steps, barrier, stream):
        """Runs `steps` steps in groups; returns the summed device time in ms."""
        torch = self.torch
        total, done = 0.0, 0
        while done < steps:
            k = min(self.group, steps - done)
            self.prepare(k)
            barrier()
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0.record(stream)
            for i in range(k):
                self.step(i)
            t1.record(stream)
            barrier()
            total += t0.elapsed_time(t1)
            done += k
        return total

    def e2e(self, steps, barrier, stream):
        """Pinned host inputs -> device, the same calls, sorted indices and kept counts back to pinned host
        memory, all inside the timed region. The compacted K/V rows stay on the device: the cache lives there."""
        torch, akv = self.torch, self.akv
        hK, hV, hP = (torch.empty(x.shape, dtype=x.dtype).pin_memory() for x in (self.K0, self.V0, self.P0))
        hK.copy_(self.K0); hV.copy_(self.V0); hP.copy_(self.P0)
        sel2 = akv.api._alloc_sel(akv.Layout.dense(self.K0), self.ev.budget, self.K0.device, detail=True)
        h_idx = torch.empty(sel2.idx_sorted.shape, dtype=torch.int32).pin_memory()
        h_kept = torch.empty(sel2.n_kept.shape, dtype=torch.int32).pin_memory()
        Kb, Vb, Pb = self.bufs[0]

        def one():
            for o in self.opts:
                Kb.copy_(hK, non_blocking=True); Vb.copy_(hV, non_blocking=True); Pb.copy_(hP, non_blocking=True)
                self.call(Kb, Vb, Pb, o, sel2)
                h_idx.copy_(sel2.idx_sorted, non_blocking=True); h_kept.copy_(sel2.n_kept, non_blocking=True)

        one()
        barrier()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        for _ in range(steps):
            one()
        t1.record(stream)
        barrier()
        assert int(h_kept.min()) == self.ev.budget
        h2d = sum(x.numel() * x.element_size() for x in (hK, hV, hP)) * len(self.opts)
        d2h = sum(x.numel() * x.element_size() for x in (h_idx, h_kept)) * len(self.opts)
        return t0.elapsed_time(t1), h2d, d2h


class CadenceWorkload:
    """C5: a paged pool; one step = 32 rounds of (compress 256 -> 128 in place, then 128 fresh rows per head
    appended). Each round's call is timed by its own pair of events; the refill runs between them, untimed."""

    def __init__(self, rank, dev, akv, synth, torch, batch=None, rounds=None):
        self.akv, self.torch = akv, torch
        c5 = synth.make_c5(seed=rank, **({} if batch is None else {"B": batch}), **({} if rounds is None else {"rounds": rounds}))
        self.c5 = c5
        self.rounds = c5.rounds
        B, L, H, N, d, b = c5.B, c5.L, c5.H, c5.N, c5.d, c5.budget
        self.esize = 2
        self.events_per_step = B * L * H * c5.rounds
        self.bytes_per_step = algorithmic_bytes(N, b, d, 2) * self.events_per_step
        self.launches_hint = c5.rounds
        self.LH = L * H
        self.pool_K0, self.pool_V0 = akv.to_device(c5.pool_K, dev), akv.to_device(c5.pool_V, dev)
        self.pool_K, self.pool_V = torch.empty_like(self.pool_K0), torch.empty_like(self.pool_V0)
        self.table = akv.to_device(c5.block_table, dev)
        self.pos0 = akv.to_device(c5.pos, dev)
        self.pos = torch.empty_like(self.pos0)
        self.q = akv.to_device(c5.qstat, dev)
        self.rK, self.rV = akv.to_device(c5.refill_K, dev), akv.to_device(c5.refill_V, dev)
        self.lay = akv.Layout.paged(self.pool_K, self.table)
        self.opts = akv.Options(lam=c5.lam)
        self.sel = akv.api._alloc_sel(self.lay, b, dev, detail=True)
        slots = torch.arange(b, N, device=dev)
        self.pg = self.table.long()[:, (slots // c5.page)]                       # [B, n_new] page of every refilled slot
        self.off = (slots % c5.page)[None, :].expand(B, -1)
        self.n_new = N - b
        self.new_pos = torch.arange(self.n_new, device=dev, dtype=torch.int32)
        self.set_bytes = (self.pool_K0.numel() + self.pool_V0.numel()) * 2
        self.l2 = f"inputs larger than L2 ({self.set_bytes / 1e6:.0f} MB touched per event call)"

    def reset(self):
        self.pool_K.copy_(self.pool_K0); self.pool_V.copy_(self.pool_V0); self.pos.copy_(self.pos0)

    def refill(self, r, srcK=None, srcV=None):
        c5 = self.c5
        blk = r % self.rK.shape[0]
        sK = self.rK[blk] if srcK is None else srcK
        sV = self.rV[blk] if srcV is None else srcV
        for l in range(c5.L):
            self.pool_K[l, self.pg, :, self.off] = sK[l].permute(1, 0, 2)[None].expand(c5.B, -1, -1, -1)
            self.pool_V[l, self.pg, :, self.off] = sV[l].permute(1, 0, 2)[None].expand(c5.B, -1, -1, -1)
        self.pos[..., c5.budget:] = c5.N + r * self.n_new + self.new_pos

    def call(self):
        self.akv.alpha_compress_event(self.pool_K, self.pool_V, self.pos, self.q, self.c5.budget, self.opts,
                                      layout=self.lay, out=self.sel)

    def timed(self, steps, barrier, stream):
        torch = self.torch
        total = 0.0
        for _ in range(steps):
            self.reset()
            pairs = []
            barrier()
            for r in range(self.rounds):
                t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                t0.record(stream)
                self.call()
                t1.record(stream)
                pairs.append((t0, t1))
                self.refill(r)
            barrier()
            total += sum(a.elapsed_time(b) for a, b in pairs)
        return total

    def e2e(self, steps, barrier, stream):
        """Per round: the 128 new rows per head come from pinned host memory (copied in and scattered into the
        pages), then the call, then sorted indices and kept counts back to pinned host memory."""
        torch = self.torch
        hK = torch.empty(self.rK[0].shape, dtype=self.rK.dtype).pin_memory()
        hV = torch.empty(self.rV[0].shape, dtype=self.rV.dtype).pin_memory()
        hK.copy_(self.rK[0]); hV.copy_(self.rV[0])
        dK, dV = torch.empty_like(self.rK[0]), torch.empty_like(self.rV[0])
        h_idx = torch.empty(self.sel.idx_sorted.shape, dtype=torch.int32).pin_memory()
        h_kept = torch.empty(self.sel.n_kept.shape, dtype=torch.int32).pin_memory()
        rounds = min(self.rounds, 4)
        self.reset()
        self.call()
        barrier()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        for _ in range(steps):
            for r in range(rounds):
                dK.copy_(hK, non_blocking=True); dV.copy_(hV, non_blocking=True)
                self.refill(r, dK, dV)
                self.call()
                h_idx.copy_(self.sel.idx_sorted, non_blocking=True); h_kept.copy_(self.sel.n_kept, non_blocking=True)
        t1.record(stream)
        barrier()
        assert int(h_kept.min()) == self.c5.budget
        scale = self.rounds / rounds                                  # reported per step of 32 rounds
        h2d = (hK.numel() + hV.numel()) * 2 * self.rounds
        d2h = (h_idx.numel() + h_kept.numel()) * 4 * self.rounds
        return t0.elapsed_time(t1) * scale, h2d, d2h


def run_gpu(args):
    import torch
    import paper_2605_14292_b200 as akv
    from paper_2605_14292_b200 import synth

    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    akv.load_library()

    if args.config == "C5":
        wl = CadenceWorkload(rank, dev, akv, synth, torch, args.batch, args.rounds)
    else:
        wl = DenseWorkload(args.config, rank, dev, args.steps, akv, synth, torch, args.batch)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    stream = torch.cuda.current_stream()
    wl.timed(args.warmup, barrier, stream)
    launches0 = akv.launch_count()
    with ClockSampler(local_rank) as clocks:
        total_ms = wl.timed(args.steps, barrier, stream)
    launches = akv.launch_count() - launches0
    total_ms = reduce_max(total_ms, world, dev)
    ms_per_step = total_ms / args.steps
    value = events_per_second(wl.events_per_step, world, args.steps, total_ms)

    # roofline: algorithmic bytes of a step / device time of a step (the step's kernels run back to back on
    # one stream; for the one-launch routes this is the mean launch duration of the one kernel)
    peak, peak_kind = load_peaks()
    achieved = wl.bytes_per_step / (ms_per_step * 1e-3) / 1e9
    rev = kernel_revision()
    traffic = NCU_TRAFFIC.get(args.config)
    traffic_bytes = traffic["bytes"] if traffic and traffic.get("revision") == rev else None
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": traffic_bytes, "peak_kind": f"of {peak_kind}", "kernel": KERNELS[args.config],
                "algorithmic_bytes_per_step": wl.bytes_per_step, "launches_per_step": launches / args.steps,
                "frac_of_nominal_8TBs": achieved / 8000.0, "kernel_revision": rev,
                # bytes the kernels really moved (ncu) over the same time: what the memory system delivered
                "dram_gbs_from_traffic": None if traffic_bytes is None else traffic_bytes / (ms_per_step * 1e-3) / 1e9,
                "dram_frac_from_traffic": None if traffic_bytes is None else traffic_bytes / (ms_per_step * 1e-3) / 1e9 / peak}

    e2e = None
    if not args.no_e2e:
        e2e_steps = max(1, min(args.steps, 10 if args.config in ("C1", "C2", "C3") else 2))
        e2e_ms, h2d, d2h = wl.e2e(e2e_steps, barrier, stream)
        e2e_ms = reduce_max(e2e_ms, world, dev)
        e2e = {"value": events_per_second(wl.events_per_step, world, e2e_steps, e2e_ms), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
               "copied_back": "sorted indices and kept counts (the compacted K/V stay on the device)"}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(args.config)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if wl.esize == 2 else "f32", "data": "synthetic",
            "config": {"workload": WORKLOADS[args.config] + (f" [batch overridden: {args.batch}]" if args.batch else "") +
                       (f" [rounds overridden: {args.rounds}]" if args.rounds else ""),
                       "events_per_gpu_per_step": wl.events_per_step,
                       "storage": "bf16" if wl.esize == 2 else "fp32", "accumulate": "f32", "l2": wl.l2,
                       "sequence_events_per_s": value / wl.LH},
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches),
            "clocks": clocks.summary(),
        }
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--config", default="C3", choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="alphakv", choices=["alphakv", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the end-to-end leg (profiler captures)")
    ap.add_argument("--batch", type=int, default=None,
                    help="number of sequences instead of the workload's own (smaller cases for profiler captures)")
    ap.add_argument("--rounds", type=int, default=None, help="C5 only: events per step instead of 32 (profiler captures)")
    args = ap.parse_args()
    if args.steps is None:
        args.steps = {"C1": 100, "C2": 100, "C3": 100, "C4": 10, "C5": 3, "C6": 50}[args.config]
    if args.impl == "reference" and args.config == "C6":
        args.steps, args.warmup = min(args.steps, 3), 3
    if args.warmup is None:
        args.warmup = 5 if args.config != "C5" else 3
    args.warmup = max(args.warmup, 3)
    if args.config == "C5":
        args.warmup = min(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
