"""Helpers for the GPU-vs-oracle parity tests. Acceptance rules:
scores within 1e-5 relative (to the Cauchy-Schwarz scale), pick sequences identical
except where the oracle's own margin is below 1e-6 (checked by replaying the GPU's
sequence in float64), compacted K/V/pos bit-exact."""
import math

import numpy as np

from oracle import alpha_oracle as O
from oracle import c_oracle as CO

SCORE_RTOL = 1e-5
MARGIN_TOL = 1e-6


def score_scale(K_bits, qstat_lh, d):
    """||q|| * ||k_i|| / sqrt(d): the scale a relative score tolerance refers to."""
    K = O.widen(K_bits)
    return np.linalg.norm(qstat_lh.astype(np.float64)) * np.linalg.norm(K, axis=-1) / math.sqrt(d)


# worst |error| / |s_ref| seen over the scores that are not cancellation-dominated, and worst error
# relative to the scale, over everything checked in this process (reported by the tests that print it)
WORST = {"rel_to_score": 0.0, "rel_to_scale": 0.0, "n": 0}
# a score counts as cancellation-dominated when it is below this fraction of the Cauchy-Schwarz scale:
# its 64 complex terms of size ~scale/8 each then cancel to less than a tenth of their own size
CANCELLATION = 0.1


def check_scores(s_gpu, s_ref, scale):
    """1e-5 relative to max(|s_ref|, scale) for every score, and 1e-5 relative to the score itself wherever
    the score is not cancellation-dominated (|s_ref| >= 0.1 scale, with the tolerance floor that fp32
    accumulation of terms of size `scale` cannot avoid: 64 roundings of 6e-8 scale / 8)."""
    tol = SCORE_RTOL * np.maximum(np.abs(s_ref), scale)
    err = np.abs(s_gpu.astype(np.float64) - s_ref)
    assert np.all(err <= tol), f"score error {err.max():.3e} exceeds {tol[np.argmax(err - tol)]:.3e}"
    big = np.abs(s_ref) >= CANCELLATION * scale
    if np.any(big):
        rel = err[big] / np.abs(s_ref[big])
        assert np.all(rel <= SCORE_RTOL), f"relative score error {rel.max():.3e} above {SCORE_RTOL}"
        WORST["rel_to_score"] = max(WORST["rel_to_score"], float(rel.max()))
    WORST["rel_to_scale"] = max(WORST["rel_to_scale"], float((err / np.maximum(scale, 1e-30)).max()))
    WORST["n"] += int(err.size)
    return float((err / np.maximum(scale, 1e-30)).max())


def check_event(K, V, pos, q, p_ref, budget, lam, gpu_scores, gpu_order, gpu_idx, K_new, V_new, pos_new,
                W=1, base=10000.0, eps=1e-8, sig=None, ref_scores=None, ref_order=None, n=None, log=None):
    """One event: K, V are the PRE-event rows [N, d] (raw dtype), *_new the post-event buffers.
    Returns the number of logged near-tie divergences."""
    N, d = K.shape
    n = N if n is None else n
    Kc, Vc = K[:n], V[:n]
    posc = None if pos is None else pos[:n]
    if ref_scores is None:
        pr = p_ref if (p_ref is not None or posc is None) else O.default_p_ref(posc)
        ref_scores = O.triattention_score(Kc, posc, q, pr, W, base)
    if gpu_scores is not None:
        check_scores(gpu_scores[:n], ref_scores, score_scale(Kc, q, d))
    kept = min(budget, n)
    order = np.asarray(gpu_order[:kept], dtype=np.int64)
    idx = np.asarray(gpu_idx[:kept], dtype=np.int64)
    assert np.all(np.asarray(gpu_idx[kept:]) == -1)
    assert len(set(order.tolist())) == kept and np.all((order >= 0) & (order < n))
    assert np.array_equal(np.sort(order), idx), "idx_sorted is not sort(pick order)"
    n_div = 0
    if ref_order is None or not np.array_equal(order, np.asarray(ref_order[:kept])):
        if sig is None:
            sig = O.signatures_per_head(Vc, eps)
        if lam == 0:
            rep = O.replay_pick_order(ref_scores, sig, 0.0, order, MARGIN_TOL)
        else:
            rep = O.replay_pick_order(ref_scores, sig, lam, order, MARGIN_TOL)
        assert rep.ok, f"pick sequence leaves the oracle's by {rep.worst_deficit:.3e} > {MARGIN_TOL}: {rep.log[:3]}"
        n_div = rep.n_diverged
        if log is not None and rep.n_diverged:
            log.extend(rep.log)
    # compaction, bit exact against the pre-event rows
    if K_new is not None:
        assert np.array_equal(K_new[:kept], K[idx]), "compacted K differs"
    if V_new is not None:
        assert np.array_equal(V_new[:kept], V[idx]), "compacted V differs"
    if pos is not None and pos_new is not None:
        assert np.array_equal(pos_new[:kept], pos[idx]), "compacted positions differ"
    return n_div


def oracle_batch(ev, budget, lam, threads=8, **kw):
    return CO.event_batch(ev.K, ev.V, ev.pos, ev.qstat, ev.p_ref, budget, lam, W=ev.future_window,
                          base=ev.rope_base, eps=ev.eps, threads=threads, **kw)
