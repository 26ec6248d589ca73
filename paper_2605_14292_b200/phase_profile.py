"""Per-phase cycle counts of the fused event kernels, from the profiling build of the library.

    python -m paper_2605_14292_b200.phase_profile --config C3 [--batch 16] [--lam 0.5]

Builds libalphakv_phase.so (the same sources with -DAKV_PHASE_CLOCKS: thread 0 of every event CTA stores
clock64() at the kernel's phase boundaries), runs one fused call of the named workload shape and prints, per
phase, the median and the mean number of SM cycles over the call's events, plus the CTA lifetime. The stamps
cost a few global stores per event; use bench.py (default library) for throughput.
"""
from __future__ import annotations

import argparse
import ctypes as C

import numpy as np
import torch

from . import api, build, synth

PHASES = {
    "event_tri_kernel": ["tensor memory claimed", "K scored", "s_(b) + pool", "V operand", "product", "triangle",
                         "picks (one warp)", "sort + outputs", "compaction"],
    "event_pool_kernel": ["tensor memory claimed", "K scored", "s_(b) + pool", "V operand", "product", "triangle",
                          "picks (one warp)", "sort + outputs", "compaction"],
    "event_tc_kernel": ["K scored", "ranks + pool", "V operand + tensor memory", "product + norms", "picks",
                        "sort + outputs", "compaction"],
    "event_stream_kernel": ["tables + positions", "K streamed and scored", "s_(b)", "pool / top-k", "V rows + norms",
                            "picks", "sort + outputs", "compaction"],
}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="C3", choices=["C2", "C3", "C4", "C5"])
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--lam", type=float, default=0.5)
    ap.add_argument("--flat", action="store_true", help="Eq. 1's flat signature with one cosine matrix per sequence (C2 shape)")
    args = ap.parse_args()
    lib = api.load_library(build.build_phase_clocks())
    api._lib = lib                                    # the binding's entry points now call the profiling build
    lib.akv_debug_phase_buffer.argtypes = [C.c_void_p]
    slots = int(lib.akv_debug_phase_slots())
    dev = torch.device("cuda")
    if args.config == "C2":
        ev, kernel = synth.make_c2(B=args.batch or 1), "event_pool_kernel"
    elif args.config == "C3":
        ev, kernel = synth.make_c3(B=args.batch or 16), "event_tri_kernel"
    elif args.config == "C4":
        ev, kernel = synth.make_c4(B=args.batch or 2, lam=args.lam), "event_stream_kernel"
    else:
        c5 = synth.make_c5(B=args.batch or 8, rounds=1)
        K = synth.paged_gather_dense(c5.pool_K, c5.block_table)
        V = synth.paged_gather_dense(c5.pool_V, c5.block_table)
        ev = synth.EventBatch("C5-round0", synth.BF16, K, V, c5.pos, c5.qstat, np.full((c5.B,), 256, dtype=np.int32),
                              c5.budget, c5.lam)
        kernel = "event_pool_kernel"
    K, V, pos = api.to_device(ev.K, dev), api.to_device(ev.V, dev), api.to_device(ev.pos, dev)
    q, pref = api.to_device(ev.qstat, dev), api.to_device(ev.p_ref, dev)
    E = ev.n_events
    buf = torch.zeros((E, slots), dtype=torch.int64, device=dev)
    K0, V0, P0 = K.clone(), V.clone(), pos.clone()
    opts, sig = api.Options(lam=args.lam), None
    if args.flat:
        sig = api.alpha_signature_flat(V)
        gram = api.alpha_gram_shared(sig, api.Layout.dense(V), api.Options(sig_mode=api.SIG_FLAT))
        opts = api.Options(lam=args.lam, sig_mode=api.SIG_FLAT, shared_gram=gram)
    for it in range(2):                               # second pass: kernels loaded, clocks settled
        K.copy_(K0); V.copy_(V0); pos.copy_(P0)
        buf.zero_()
        assert lib.akv_debug_phase_buffer(C.c_void_p(buf.data_ptr())) == 0
        api.alpha_compress_event(K, V, pos, q, ev.budget, opts, p_ref=pref, flat_sig=sig, detail=False)
        torch.cuda.synchronize()
    lib.akv_debug_phase_buffer(None)
    st = buf.cpu().numpy()
    names = PHASES[kernel]
    print(f"{kernel}, {args.config}-shaped, {E} events, lambda {args.lam}: SM cycles per phase (median / mean over events)")
    for k, name in enumerate(names):
        ok = (st[:, k + 1] > 0) & (st[:, k] > 0)
        d = (st[ok, k + 1] - st[ok, k]).astype(np.float64)
        if d.size:
            print(f"  {name:32s} {np.median(d):10.0f} {d.mean():10.0f}")
    if kernel == "event_stream_kernel" and np.any(st[:, 10] > 0):
        for k, name in ((10, "  of picks: arg-max + exchange"), (11, "  of picks: products (misses)"), (12, "  of picks: tensor-memory read")):
            print(f"  {name:32s} {np.median(st[:, k]):10.0f} {st[:, k].mean():10.0f}")
    if kernel == "event_stream_kernel" and np.any(st[:, 13] > 0):
        print(f"  {'  of K streamed: warp 0 waiting for a stage':32s} {np.median(st[:, 13]):10.0f} {st[:, 13].mean():10.0f}")
    if kernel == "event_pool_kernel" and np.any(st[:, 10] > 0):
        ok = (st[:, 10] > 0) & (st[:, 1] > 0)
        d = (st[ok, 10] - st[ok, 1]).astype(np.float64)
        print(f"  {'  of K scored: until K arrived':32s} {np.median(d):10.0f} {d.mean():10.0f}")
        if np.any(st[:, 12] > 0):
            d = (st[ok, 12] - st[ok, 10]).astype(np.float64)
            print(f"  {'  of K scored: scoring loop':32s} {np.median(d):10.0f} {d.mean():10.0f}")
            print(f"  {'    of which rotations (fresh or chained)':32s} {np.median(st[ok, 11]):10.0f} {st[ok, 11].mean():10.0f}")
    life = (st[:, len(names)] - st[:, 0]).astype(np.float64)
    life = life[(st[:, len(names)] > 0) & (st[:, 0] > 0)]
    print(f"  {'CTA lifetime':32s} {np.median(life):10.0f} {life.mean():10.0f}")


if __name__ == "__main__":
    main()
