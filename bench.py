#!/usr/bin/env python
"""Benchmark of the KV-cache compression event (fused alpha_compress_event).

One *step* = one pass of the whole hot path (score -> greedy selection -> ordering -> in-place
compaction) over one batch of synthetic input shaped like the Llama-8B configuration
(batch 16 x 32 layers x 8 KV heads = 4096 events, N = 192 -> b = 64, d = 128, bf16,
lambda = 0.5, 5 % near-duplicate V rows). Prints one JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

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
WORKLOAD = "C3 Llama-8B-shaped: batch 16 x 32 layers x 8 KV heads, N=192 -> b=64, d=128, bf16, lambda=0.5"
# Algorithmic HBM bytes of one event: read K and V once, write b rows of each, plus positions in,
# positions + indices out and the query statistic.
def algorithmic_bytes(N, b, d, esize):
    return 2 * N * d * esize + 2 * b * d * esize + 4 * N + 8 * b + 4 * d

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the fused kernel on this workload, from
# the ncu capture summarised under profiles/ (None until a capture of the current kernel exists).
NCU_TRAFFIC_BYTES_PER_LAUNCH = 328119296 + 97766400


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
def oracle_time(ev, reps=1, threads=None):
    """Times the C oracle, as it stands, on whole events of `ev` with `threads` host threads."""
    from oracle import c_oracle as CO
    threads = threads or (os.cpu_count() or 1)
    CO.build()
    E = ev.n_events
    CO.event_batch(ev.K, ev.V, ev.pos, ev.qstat, ev.p_ref, ev.budget, ev.lam, events=(0, min(E, threads)), threads=threads)
    t0 = time.perf_counter()
    for _ in range(reps):
        CO.event_batch(ev.K, ev.V, ev.pos, ev.qstat, ev.p_ref, ev.budget, ev.lam, threads=threads)
    dt = time.perf_counter() - t0
    return E * reps / dt, threads, dt


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    from paper_2605_14292_b200 import synth
    B_sample = 2                                                     # 512 of the 4096 events per step
    ev = synth.make_c3(seed=0, B=B_sample)
    threads = os.cpu_count() or 1
    for _ in range(args.warmup):
        oracle_time(ev, 1, threads)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_time(ev, 1, threads)
    dt = time.perf_counter() - t0
    value = ev.n_events * args.steps / dt
    sample = f"{ev.n_events} of 4096 events per step (batch {B_sample} of 16), C oracle in float64, {threads} threads"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------ GPU arm
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

    ev = synth.make_c3(seed=rank)                                    # every rank: its own batch of 4096 events
    B, L, H, N, d = ev.shape
    E, b = ev.n_events, ev.budget
    esize = 2
    opts = akv.Options(lam=ev.lam)
    K0, V0, P0 = akv.to_device(ev.K, dev), akv.to_device(ev.V, dev), akv.to_device(ev.pos, dev)
    q, pref = akv.to_device(ev.qstat, dev), akv.to_device(ev.p_ref, dev)

    # The event rewrites K/V/pos in place, so every timed step gets a pristine copy of the batch:
    # nbuf working sets (each ~405 MB, larger than the 126 MB L2), restored outside the timed regions.
    nbuf = max(1, min(args.steps, 24))
    bufs = [(torch.empty_like(K0), torch.empty_like(V0), torch.empty_like(P0)) for _ in range(nbuf)]
    sel = akv.api._alloc_sel(akv.Layout.dense(K0), b, dev, detail=False)

    def restore(k):
        for i in range(k):
            bufs[i][0].copy_(K0); bufs[i][1].copy_(V0); bufs[i][2].copy_(P0)

    def step(i):
        Kb, Vb, Pb = bufs[i]
        akv.alpha_compress_event(Kb, Vb, Pb, q, b, opts, p_ref=pref, out=sel)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    done = 0
    while done < args.warmup:
        k = min(nbuf, args.warmup - done)
        restore(k)
        for i in range(k):
            step(i)
        done += k
    torch.cuda.synchronize()

    stream = torch.cuda.current_stream()
    total_ms, done = 0.0, 0
    launches0 = akv.launch_count()
    with ClockSampler(local_rank) as clocks:
        while done < args.steps:
            k = min(nbuf, args.steps - done)
            restore(k)
            barrier()
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0.record(stream)
            for i in range(k):
                step(i)
            t1.record(stream)
            barrier()
            total_ms += t0.elapsed_time(t1)
            done += k
    launches = akv.launch_count() - launches0
    total_ms = reduce_max(total_ms, world, dev)
    ms_per_step = total_ms / args.steps
    value = events_per_second(E, world, args.steps, total_ms)

    # roofline of the dominant (only) kernel: algorithmic bytes per launch / mean launch duration
    peak, peak_kind = load_peaks()
    bytes_per_launch = algorithmic_bytes(N, b, d, esize) * E
    kernel_ms = ms_per_step                                          # one launch per step, timed back to back
    achieved = bytes_per_launch / (kernel_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH, "peak_kind": f"of {peak_kind}",
                "kernel": "event_tri_kernel<fused>", "algorithmic_bytes_per_launch": bytes_per_launch}

    # end to end: pinned host buffers -> device, the same C-ABI call, indices and kept counts back
    hK, hV, hP = (torch.empty(x.shape, dtype=x.dtype).pin_memory() for x in (K0, V0, P0))
    hK.copy_(K0); hV.copy_(V0); hP.copy_(P0)
    sel2 = akv.api._alloc_sel(akv.Layout.dense(K0), b, dev, detail=True)
    h_idx = torch.empty(sel2.idx_sorted.shape, dtype=torch.int32).pin_memory()
    h_kept = torch.empty(sel2.n_kept.shape, dtype=torch.int32).pin_memory()
    Kb, Vb, Pb = bufs[0]
    e2e_steps = max(3, min(args.steps, 10))

    def e2e_step():
        Kb.copy_(hK, non_blocking=True); Vb.copy_(hV, non_blocking=True); Pb.copy_(hP, non_blocking=True)
        akv.alpha_compress_event(Kb, Vb, Pb, q, b, opts, p_ref=pref, out=sel2)
        h_idx.copy_(sel2.idx_sorted, non_blocking=True); h_kept.copy_(sel2.n_kept, non_blocking=True)

    for _ in range(2):
        e2e_step()
    barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    t1.record(stream)
    barrier()
    e2e_ms = reduce_max(t0.elapsed_time(t1), world, dev)
    h2d = sum(x.numel() * x.element_size() for x in (hK, hV, hP))
    d2h = sum(x.numel() * x.element_size() for x in (h_idx, h_kept))
    e2e = {"value": events_per_second(E, world, e2e_steps, e2e_ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h, "steps": e2e_steps}
    assert int(h_kept.min()) == b

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, threads, dt = oracle_time(ev, reps=1)
        cpu = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": f"all {E} events of the same batch once, C oracle in float64, {dt:.1f} s wall"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": WORKLOAD, "events_per_gpu": E, "storage": "bf16", "l2": "inputs larger than L2 "
                       f"({(K0.numel() + V0.numel()) * esize / 1e6:.0f} MB per step, fresh copy per step)",
                       "sequence_events_per_s": value / (L * H)},
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
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="alphakv", choices=["alphakv", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
