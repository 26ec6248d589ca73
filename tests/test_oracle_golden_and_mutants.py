"""(1) The stored oracle outputs for configs[0] still come out of the oracle.
(2) The pins have teeth: plausible mistakes planted in a copy of the selection
loop (on the CPU, in this file) are each caught by one of the closed-form pins."""
import json
import os

import numpy as np

from oracle import alpha_oracle as O
from paper_2605_14292_b200 import synth

GOLD = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "c1_event.json")


def test_c1_matches_stored_oracle_values():
    g = json.load(open(GOLD))
    ev = synth.make_c1(seed=0)
    K, V, pos, q = ev.K[0, 0, 0], ev.V[0, 0, 0], ev.pos[0, 0, 0], ev.qstat[0, 0]
    for lam in (0.0, 0.5, 1.0):
        r = O.compress_event(K, V, pos, q, int(ev.p_ref[0]), ev.budget, lam)
        e = g[f"lambda_{lam}"]
        assert r.sel.idx_sorted.tolist() == e["idx_sorted"]
        assert r.sel.order.tolist() == e["pick_order"]
        assert np.allclose(r.scores[:8], e["scores_first8"], rtol=0, atol=1e-12)
        assert abs(r.scores.sum() - e["score_sum"]) < 1e-10


def mutant_select(s, sig, k, lam, floor=True, sign=+1.0, update_after_first=True, use_min=False):
    """A copy of the greedy loop with switches for planted mistakes."""
    n = len(s)
    m = np.zeros(n) if floor else np.full(n, -np.inf)
    S = []
    i = int(np.argmax(s))
    S.append(i)
    if update_after_first:
        m = np.maximum(m, sig @ sig[i])
    for _ in range(1, k):
        pen = np.where(np.isfinite(m), m, 0.0)
        a = s - sign * lam * pen
        a[S] = -np.inf
        i = int(np.argmin(np.where(np.isfinite(a), a, np.inf))) if use_min else int(np.argmax(a))
        S.append(i)
        m = np.maximum(m, sig @ sig[i])
    return S


def _pins(select):
    """Returns the list of pins (by name) that the given selector fails."""
    failed = []
    rng = np.random.default_rng(0)
    # anti-aligned V: must be top-k
    n = 12
    s = rng.standard_normal(n)
    sig = O.signatures_per_head((np.eye(n) - 1.0 / n).astype(np.float32))
    if select(s, sig, 7, 2.0) != O.topk_indices(s, 7).tolist():
        failed.append("antialigned->topk")
    # duplicate pairs: leaders only
    sc, V, leaders = synth.make_duplicate_pairs(8, 16, 0.01, seed=1)
    sg = O.signatures_per_head(V)
    lam = float(sc[0] - 0.01 - sc[14]) + 0.05
    if sorted(select(sc, sg, 5, lam)) != leaders[:5].tolist():
        failed.append("duplicate-pairs->leaders")
    # first pick's duplicate must be penalised at once
    s2 = np.array([2.0, 1.99, 1.0, 0.5])
    V2 = np.array([[1, 0], [1, 0], [0, 1], [0, 1]], dtype=np.float32)
    if select(s2, O.signatures_per_head(V2), 2, 1.5) != [0, 2]:
        failed.append("first-pick-updates-m")
    # an exactly opposite V row earns no bonus (floor at zero)
    s3 = np.array([2.0, 1.0, 1.1])
    V3 = np.array([[1, 0], [-1, 0], [0, 1]], dtype=np.float32)
    if select(s3, O.signatures_per_head(V3), 2, 0.5) != [0, 2]:
        failed.append("opposite-row-no-bonus")
    return failed


def test_true_loop_passes_and_each_mutant_fails_some_pin():
    true = lambda s, sig, k, lam: O.alpha_select(s, sig, k, lam).order.tolist()
    assert _pins(true) == []
    assert _pins(lambda *a: mutant_select(*a)) == []                         # the faithful copy passes too
    assert _pins(lambda *a: mutant_select(*a, floor=False))                  # no floor at zero (Eq. 2)
    assert _pins(lambda *a: mutant_select(*a, sign=-1.0))                    # penalty turned into a bonus
    assert _pins(lambda *a: mutant_select(*a, update_after_first=False))     # m not updated after i_1
    assert _pins(lambda *a: mutant_select(*a, use_min=True))                 # argmin instead of argmax
