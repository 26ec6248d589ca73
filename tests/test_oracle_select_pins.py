"""Pins for the oracle's signatures, selection and compaction (Section 4.1,
Eq. 1-3, Algorithm 1). Each pin is something the paper or the mathematics
fixes independently of the oracle's own loop."""
import itertools
import math

import numpy as np
import pytest

from oracle import alpha_oracle as O
from oracle import c_oracle as CO
from paper_2605_14292_b200 import synth


def rand_problem(n, d, seed, corr=0.0):
    rng = np.random.default_rng(seed)
    s = rng.standard_normal(n)
    V = rng.standard_normal((n, d)).astype(np.float32)
    if corr:
        common = rng.standard_normal(d).astype(np.float32)
        V = V + corr * common
    return s, V


# ----------------------------------------------------------------- signatures
def test_signature_row_norm_and_eps_form():
    rng = np.random.default_rng(0)
    V = rng.standard_normal((7, 16)).astype(np.float32)
    V[3] = 0.0
    for eps in (1e-8, 0.25):
        sig = O.signatures_per_head(V, eps)
        nrm = np.linalg.norm(V.astype(np.float64), axis=1)
        assert np.allclose(np.linalg.norm(sig, axis=1), nrm / (nrm + eps), rtol=0, atol=1e-15)
        assert np.all(sig[3] == 0.0)           # zero row -> zero signature -> cosine 0
        assert np.max(np.abs(CO.signature(V, eps) - sig)) < 1e-15


def test_signature_flat_reduces_to_per_head_and_is_the_mean():
    rng = np.random.default_rng(1)
    V = rng.standard_normal((3, 2, 9, 8)).astype(np.float32)
    one = O.signatures_flat(V[:1, :1], 1e-8)
    assert np.max(np.abs(one - O.signatures_per_head(V[0, 0], 1e-8))) < 1e-15
    flat = O.signatures_flat(V, 1e-3)
    u = np.zeros((9, 8))
    for l in range(3):
        for h in range(2):
            u += V[l, h].astype(np.float64)
    u /= 6.0
    want = u / (np.linalg.norm(u, axis=1) + 1e-3)[:, None]
    assert np.max(np.abs(flat - want)) < 1e-15


def test_selection_invariant_to_positive_row_scaling_of_V():
    s, V = rand_problem(40, 16, 3, corr=1.0)
    c = np.random.default_rng(9).uniform(0.1, 10.0, size=(40, 1)).astype(np.float32)
    a = O.alpha_select(s, O.signatures_per_head(V), 15, 0.7)
    b = O.alpha_select(s, O.signatures_per_head(V * c), 15, 0.7)
    assert np.array_equal(a.order, b.order)


# ----------------------------------------------------------------- lambda = 0
@pytest.mark.parametrize("seed", range(5))
def test_lambda0_is_topk_in_every_path(seed):
    s, V = rand_problem(60, 8, seed)
    s[7] = s[3]                                  # exact ties: lower index first
    s[50] = s[20]
    sig = O.signatures_per_head(V)
    k = 25
    want = sorted(range(60), key=lambda i: (-s[i], i))[:k]   # stable sort by (-s, index)
    fast = O.alpha_select(s, sig, k, 0.0)
    loop = O.alpha_select(s, sig, k, 0.0, force_greedy=True)
    assert list(fast.order) == want and list(loop.order) == want
    assert list(O.topk_indices(s, k)) == want
    assert list(O.alpha_select_from_definition(s, sig, k, 0.0)) == sorted(want)
    for fg in (False, True):
        oc, _, _, _ = CO.select(s, sig, k, 0.0, force_greedy=fg)
        assert list(oc) == want


def test_topk_boundary_tie_goes_to_lower_index():
    s = np.array([1.0, 5.0, 3.0, 3.0, 3.0, 0.0])
    assert list(O.topk_indices(s, 3)) == [1, 2, 3]
    assert list(O.alpha_select(s, np.eye(6), 3, 0.0).idx_sorted) == [1, 2, 3]


# ----------------------------------------------------------------- the step rule (Eq. 2, Eq. 3)
@pytest.mark.parametrize("n,d,k,lam,seed", [(6, 2, 4, 0.5, 0), (9, 4, 9, 1.0, 1), (12, 8, 7, 1.5, 2),
                                            (12, 4, 12, 0.5, 3), (10, 2, 5, 3.0, 4), (11, 8, 6, 0.25, 5)])
def test_each_pick_maximises_eq2_from_the_definition(n, d, k, lam, seed):
    s, V = rand_problem(n, d, seed, corr=0.5)
    sig = O.signatures_per_head(V)
    for order in (O.alpha_select(s, sig, k, lam).order, CO.select(s, sig, k, lam)[0]):
        S = []
        for t, pick in enumerate(order):
            cand = [i for i in range(n) if i not in S]
            vals = {i: O.marginal_gain(i, S, s, sig, lam) for i in cand}
            best = max(vals.values())
            winners = [i for i in cand if vals[i] == best]
            assert pick == min(winners), (t, pick, winners)
            S.append(int(pick))


@pytest.mark.parametrize("seed", range(4))
def test_invariants_distinct_sorted_first_pick_gains_monotone(seed):
    n, d, k, lam = 80, 16, 30, 0.5
    s, V = rand_problem(n, d, 10 + seed, corr=0.8)
    sig = O.signatures_per_head(V)
    sel = O.alpha_select(s, sig, k, lam)
    assert len(set(sel.order.tolist())) == k
    assert np.all(np.diff(sel.idx_sorted) > 0)
    assert sorted(sel.order.tolist()) == sel.idx_sorted.tolist()
    assert sel.order[0] == int(np.argmax(s))
    assert np.all(np.diff(sel.gains) <= 1e-15)          # m only grows, so the best value only falls
    assert np.all(sel.margins >= 0)


def test_running_max_vector_stays_in_unit_interval():
    s, V = rand_problem(50, 8, 21, corr=2.0)
    sig = O.signatures_per_head(V)
    sel = O.alpha_select(s, sig, 20, 0.5)
    m = np.zeros(50)
    for i in sel.order:
        m = np.maximum(m, sig @ sig[i])
        assert m.min() >= 0.0 and m.max() <= 1.0 + 1e-12


def test_on_demand_rows_equal_full_gram_variant_and_c_twin():
    for seed in range(6):
        n, d, k = 24, 8, 11
        s, V = rand_problem(n, d, 30 + seed, corr=1.0)
        sig = O.signatures_per_head(V)
        for lam in (0.3, 0.5, 1.0, 2.0):
            a = O.alpha_select(s, sig, k, lam)
            assert np.array_equal(a.idx_sorted, O.alpha_select_from_definition(s, sig, k, lam))
            oc, gc, mc, st = CO.select(s, sig, k, lam)
            assert np.array_equal(oc, a.order) and st == 0
            assert np.max(np.abs(gc - a.gains)) < 1e-13
            assert np.max(np.abs(mc - a.margins)) < 1e-13


def test_permutation_of_candidates_permutes_the_result():
    n, d, k, lam = 40, 16, 17, 0.5
    s, V = rand_problem(n, d, 44, corr=0.7)
    sig = O.signatures_per_head(V)
    base = O.alpha_select(s, sig, k, lam)
    assert base.margins.min() > 1e-9            # no near ties, so the result is unique
    rng = np.random.default_rng(45)
    for _ in range(5):
        perm = rng.permutation(n)               # new slot j holds old candidate perm[j]
        got = O.alpha_select(s[perm], O.signatures_per_head(V[perm]), k, lam)
        assert [int(perm[j]) for j in got.order] == base.order.tolist()


# ----------------------------------------------------------------- closed forms
@pytest.mark.parametrize("lam", [0.5, 1.0, 5.0])
def test_identical_V_rows_give_topk(lam):
    rng = np.random.default_rng(50)
    s = rng.standard_normal(30)
    V = np.tile(rng.standard_normal((1, 8)).astype(np.float32), (30, 1))
    got = O.alpha_select(s, O.signatures_per_head(V), 12, lam)
    assert got.order.tolist() == O.topk_indices(s, 12).tolist()   # every penalty is the same constant


@pytest.mark.parametrize("lam", [0.5, 2.0])
def test_orthogonal_or_antialigned_V_gives_topk(lam):
    """Floor at 0 (Eq. 2): candidates orthogonal to or anti-aligned with S_t get no bonus."""
    rng = np.random.default_rng(51)
    n = 16
    s = rng.standard_normal(n)
    V_orth = np.eye(n, dtype=np.float32) * rng.uniform(0.5, 2, size=(n, 1)).astype(np.float32)
    assert O.alpha_select(s, O.signatures_per_head(V_orth), 9, lam).order.tolist() == O.topk_indices(s, 9).tolist()
    # simplex-like directions: all pairwise cosines are negative
    V_neg = (np.eye(n) - 1.0 / n).astype(np.float32)
    sig = O.signatures_per_head(V_neg)
    off = (sig @ sig.T)[~np.eye(n, dtype=bool)]
    assert off.max() < 0
    assert O.alpha_select(s, sig, 9, lam).order.tolist() == O.topk_indices(s, 9).tolist()


def test_duplicate_pairs_keep_one_of_each_pair():
    """Appendix A: the base score dominates except where attention-equivalent candidates are
    V-redundant. P pairs of identical V rows, orthogonal across pairs, follower = leader - delta.
    With lambda > s_1 - delta - s_P and b <= P the result is exactly the b best leaders; lambda = 0
    takes the top-b of the 2P scores."""
    P, d, delta = 10, 16, 0.01
    s, V, leaders = synth.make_duplicate_pairs(P, d, delta, seed=3)
    sig = O.signatures_per_head(V)
    lam = float(s[0] - delta - s[2 * (P - 1)]) + 0.05
    for b in (1, 4, P):
        got = O.alpha_select(s, sig, b, lam)
        assert got.idx_sorted.tolist() == leaders[:b].tolist()
        assert CO.select(s, sig, b, lam)[0].tolist() == got.order.tolist()
    top = O.alpha_select(s, sig, 6, 0.0).idx_sorted.tolist()
    assert top == sorted(sorted(range(2 * P), key=lambda i: (-s[i], i))[:6])
    assert top != leaders[:6].tolist()


def test_small_lambda_cannot_reorder_well_separated_scores():
    """If consecutive scores differ by more than lambda, the penalty (<= lambda) can never flip a pair."""
    n, lam = 20, 0.3
    s = np.arange(n)[::-1] * (lam + 0.01)
    _, V = rand_problem(n, 8, 60, corr=3.0)
    got = O.alpha_select(s, O.signatures_per_head(V), 8, lam)
    assert got.order.tolist() == list(range(8))


def test_exact_pruning_proposition():
    """m <= 1, so a candidate with s_i < s_(k) - lambda can never be an argmax while fewer than k are
    chosen: selecting on the pruned pool equals selecting on the full pool."""
    for seed in range(8):
        n, d, k, lam = 120, 16, 20, 0.5
        s, V = rand_problem(n, d, 70 + seed, corr=1.0)
        sig = O.signatures_per_head(V)
        full = O.alpha_select(s, sig, k, lam)
        thr = np.sort(s)[::-1][k - 1] - lam
        pool = np.nonzero(s >= thr)[0]
        assert len(pool) < n
        sub = O.alpha_select(s[pool], sig[pool], k, lam)
        assert pool[sub.order].tolist() == full.order.tolist()


def test_exhaustive_tiny_greedy_value_never_beaten_at_first_two_steps():
    """Brute force over all ordered pairs on tiny n: the greedy's first two picks maximise
    s_i + Delta(j | {i}) among pairs that start with argmax s (Eq. 3 taken literally)."""
    for seed in range(10):
        n, d = 7, 2
        s, V = rand_problem(n, d, 90 + seed)
        sig = O.signatures_per_head(V)
        lam = 0.8
        sel = O.alpha_select(s, sig, 2, lam)
        i1 = int(np.argmax(s))
        best = max((O.marginal_gain(j, [i1], s, sig, lam), -j) for j in range(n) if j != i1)
        assert sel.order[0] == i1 and sel.order[1] == -best[1]


# ----------------------------------------------------------------- edge cases
def test_budget_equals_n_and_budget_above_n():
    s, V = rand_problem(9, 4, 100)
    sig = O.signatures_per_head(V)
    a = O.alpha_select(s, sig, 9, 0.5)
    assert a.idx_sorted.tolist() == list(range(9)) and a.status == O.STATUS_OK
    b = O.alpha_select(s, sig, 12, 0.5)
    assert b.idx_sorted.tolist() == list(range(9)) and b.status == O.STATUS_SHORT
    oc, _, _, st = CO.select(s, sig, 12, 0.5)
    assert sorted(oc.tolist()) == list(range(9)) and st == O.STATUS_SHORT


def test_nonfinite_scores_are_never_preferred():
    s, V = rand_problem(12, 4, 101)
    s[2], s[5], s[7] = np.nan, np.inf, -np.inf
    sig = O.signatures_per_head(V)
    a = O.alpha_select(s, sig, 9, 0.5)
    assert a.status == O.STATUS_NONFINITE
    assert not ({2, 5, 7} & set(a.order.tolist()))
    oc, _, _, st = CO.select(s, sig, 9, 0.5)
    assert oc.tolist() == a.order.tolist() and st == O.STATUS_NONFINITE


# ----------------------------------------------------------------- compaction and whole event
def test_compaction_is_bit_copy_in_ascending_order():
    ev = synth.make_plain(1, 1, 1, 33, 16, 8, 0.5, dtype=synth.BF16, seed=7)
    K, V, pos = ev.K[0, 0, 0], ev.V[0, 0, 0], ev.pos[0, 0, 0]
    r = O.compress_event(K, V, pos, ev.qstat[0, 0], ev.p_ref[0], 8, 0.5)
    idx = r.sel.idx_sorted
    assert np.all(np.diff(idx) > 0)
    assert r.K_new.dtype == np.uint16 and np.array_equal(r.K_new, K[idx]) and np.array_equal(r.V_new, V[idx])
    assert np.array_equal(r.pos_new, pos[idx])
    # in place, moving rows in ascending slot order, gives the same cache
    Kb = K.copy()
    for slot, src in enumerate(idx):
        Kb[slot] = Kb[src]
    assert np.array_equal(Kb[:8], r.K_new)


def test_event_batch_c_matches_numpy_event():
    ev = synth.make_c3(seed=5, B=1, L=2, H=2, N=48, budget=16)
    out = CO.event_batch(ev.K, ev.V, ev.pos, ev.qstat, ev.p_ref, 16, 0.5, threads=2)
    for l in range(2):
        for h in range(2):
            r = O.compress_event(ev.K[0, l, h], ev.V[0, l, h], ev.pos[0, l, h], ev.qstat[l, h], ev.p_ref[0], 16, 0.5)
            assert np.max(np.abs(out["scores"][0, l, h] - r.scores)) < 1e-12
            assert out["order"][0, l, h].tolist() == r.sel.order.tolist()
            assert out["idx_sorted"][0, l, h].tolist() == r.sel.idx_sorted.tolist()
            assert np.array_equal(out["K"][0, l, h], r.K_new) and np.array_equal(out["V"][0, l, h], r.V_new)
            assert np.array_equal(out["pos"][0, l, h], r.pos_new)


def test_default_reference_position_is_one_past_newest():
    ev = synth.make_plain(1, 1, 1, 20, 8, 5, 0.5, dtype=synth.F32, seed=8)
    pos = ev.pos[0, 0, 0] * 3 + 5
    a = O.compress_event(ev.K[0, 0, 0], ev.V[0, 0, 0], pos, ev.qstat[0, 0], None, 5, 0.5)
    b = O.compress_event(ev.K[0, 0, 0], ev.V[0, 0, 0], pos, ev.qstat[0, 0], int(pos.max()) + 1, 5, 0.5)
    assert np.array_equal(a.scores, b.scores)
    out = CO.event_batch(ev.K, ev.V, pos.reshape(1, 1, 1, -1), ev.qstat, None, 5, 0.5)
    assert np.max(np.abs(out["scores"][0, 0, 0] - a.scores)) < 1e-12


def test_duplicated_rows_in_c3_recipe_change_the_selection():
    """The C3 recipe plants near-duplicate V rows; with lambda = 0.5 some event must differ from top-k,
    and a planted pair is never kept together unless scores force it."""
    ev = synth.make_c3(seed=0, B=1, L=2, H=4, N=192, budget=64)
    differ = 0
    for l in range(2):
        for h in range(4):
            r = O.compress_event(ev.K[0, l, h], ev.V[0, l, h], ev.pos[0, l, h], ev.qstat[l, h], ev.p_ref[0], 64, 0.5)
            top = np.sort(O.topk_indices(r.scores, 64))
            differ += int(not np.array_equal(top, r.sel.idx_sorted))
    assert differ > 0


def test_replay_accepts_oracle_order_and_rejects_a_wrong_pick():
    s, V = rand_problem(30, 8, 111, corr=1.0)
    sig = O.signatures_per_head(V)
    sel = O.alpha_select(s, sig, 10, 0.5)
    rep = O.replay_pick_order(s, sig, 0.5, sel.order)
    assert rep.ok and rep.n_diverged == 0
    bad = sel.order.copy()
    unused = [i for i in range(30) if i not in set(bad.tolist())]
    bad[4] = min(unused, key=lambda i: s[i])
    rep = O.replay_pick_order(s, sig, 0.5, bad)
    assert not rep.ok and rep.n_diverged >= 1
    dup = sel.order.copy()
    dup[3] = dup[1]
    assert not O.replay_pick_order(s, sig, 0.5, dup).ok


def test_too_few_finite_scores_still_gives_distinct_indices():
    s = np.array([np.nan, 1.0, np.inf, 0.5, -np.inf, np.nan])
    sig = O.signatures_per_head(np.eye(6, dtype=np.float32))
    for lam in (0.0, 0.5):
        a = O.alpha_select(s, sig, 4, lam)
        assert a.order[:2].tolist() == [1, 3]
        assert len(set(a.order.tolist())) == 4 and a.order[2:].tolist() == [0, 2]
        oc, _, _, st = CO.select(s, sig, 4, lam)
        assert oc.tolist() == a.order.tolist() and st == O.STATUS_NONFINITE


# ----------------------------------------------------------------- per-layer signatures, per-head budgets (Section 6)
def test_signature_per_layer_is_the_head_mean_and_reduces_to_the_other_modes():
    rng = np.random.default_rng(41)
    V = rng.standard_normal((3, 4, 9, 8)).astype(np.float32)           # [L, H, n, d]
    for l in range(3):
        sig = O.signatures_per_layer(V[l], 1e-3)
        u = np.zeros((9, 8))
        for h in range(4):                                               # the sum of Eq. 1 over this layer's heads only
            u += V[l, h].astype(np.float64)
        u /= 4.0
        assert np.max(np.abs(sig - u / (np.linalg.norm(u, axis=1) + 1e-3)[:, None])) < 1e-15
        # Eq. 1 over a cache that has only this layer is the same thing
        assert np.max(np.abs(sig - O.signatures_flat(V[l:l + 1], 1e-3))) < 1e-15
    # one head per layer: the per-layer signature is the per-head one
    assert np.max(np.abs(O.signatures_per_layer(V[1, 2:3], 1e-8) - O.signatures_per_head(V[1, 2], 1e-8))) < 1e-15


def test_smaller_budget_is_a_prefix_of_the_larger_one():
    """Eq. 3 defines pick t from the picks before it only, so the selection at budget k' < k is the first k'
    picks of the selection at budget k: what per-(layer, head) budgets rely on."""
    s, V = rand_problem(60, 16, 42, corr=0.8)
    sig = O.signatures_per_head(V)
    full = O.alpha_select(s, sig, 40, 0.6)
    for k in (1, 7, 25, 39):
        part = O.alpha_select(s, sig, k, 0.6)
        assert np.array_equal(part.order, full.order[:k])
        assert np.array_equal(CO.select(s, sig, k, 0.6)[0], full.order[:k])


def test_event_batch_with_per_head_budgets():
    ev = synth.make_plain(2, 3, 2, 48, 16, 20, 0.5, dtype=synth.BF16, seed=43)
    same = CO.event_batch(ev.K, ev.V, ev.pos, ev.qstat, ev.p_ref, 20, 0.5)
    uni = CO.event_batch(ev.K, ev.V, ev.pos, ev.qstat, ev.p_ref, 20, 0.5, budgets=np.full((3, 2), 20))
    for k in same:
        assert np.array_equal(same[k], uni[k]), k                       # uniform budgets = the scalar call
    bud = np.array([[1, 20], [7, 13], [20, 5]], dtype=np.int32)
    rag = CO.event_batch(ev.K, ev.V, ev.pos, ev.qstat, ev.p_ref, 20, 0.5, budgets=bud)
    assert int((rag["idx_sorted"] >= 0).sum()) == 2 * int(bud.sum())    # total kept = sum of the budgets
    for b in range(2):
        for l in range(3):
            for h in range(2):
                k = int(bud[l, h])
                r = O.compress_event(ev.K[b, l, h], ev.V[b, l, h], ev.pos[b, l, h], ev.qstat[l, h], int(ev.p_ref[b]), k, 0.5)
                assert np.array_equal(rag["order"][b, l, h, :k], r.sel.order) and np.all(rag["order"][b, l, h, k:] == -1)
                assert np.array_equal(rag["idx_sorted"][b, l, h, :k], r.sel.idx_sorted)
                assert np.array_equal(rag["K"][b, l, h, :k], r.K_new) and np.array_equal(rag["V"][b, l, h, :k], r.V_new)
                assert np.array_equal(rag["order"][b, l, h, :k], same["order"][b, l, h, :k])
