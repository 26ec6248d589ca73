"""GPU-vs-oracle parity, through the C ABI (via the thin binding), element by element."""
import numpy as np
import pytest
import torch

import __graft_entry__ as entry
import paper_2605_14292_b200 as akv
from oracle import alpha_oracle as O
from oracle import c_oracle as CO
from paper_2605_14292_b200 import synth

import akv_check as chk

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    entry.build()
    akv.load_library()


def dev(x):
    return akv.to_device(x, "cuda")


def run_fused(ev, lam=None, flags=0, n_cand=None, p_ref=True, W=None, budgets=None):
    lam = ev.lam if lam is None else lam
    K, V, pos, q = dev(ev.K), dev(ev.V), dev(ev.pos), dev(ev.qstat)
    pref = dev(ev.p_ref) if p_ref else None
    nc = None if n_cand is None else dev(np.asarray(n_cand, dtype=np.int32))
    hb = None if budgets is None else dev(np.ascontiguousarray(budgets, dtype=np.int32))
    opts = akv.Options(lam=lam, eps=ev.eps, rope_base=ev.rope_base, future_window=W or ev.future_window, flags=flags,
                       head_budgets=hb)
    sel = akv.alpha_compress_event(K, V, pos, q, ev.budget, opts, p_ref=pref, n_cand=nc, want_scores=True)
    torch.cuda.synchronize()
    return dict(K=akv.to_host_bits(K), V=akv.to_host_bits(V), pos=pos.cpu().numpy(), idx=sel.idx_sorted.cpu().numpy(),
                order=sel.pick_order.cpu().numpy(), gain=sel.pick_gain.cpu().numpy(), scores=sel.scores.cpu().numpy(),
                n_kept=sel.n_kept.cpu().numpy(), status=sel.status.cpu().numpy())


def check_all(ev, g, lam, events=None, n_cand=None, p_ref=True, W=None, threads=8, budgets=None):
    B, L, H, N, d = ev.shape
    W = W or ev.future_window
    E = B * L * H
    log = []
    ref = None
    if n_cand is None and p_ref and events is None:
        ref = CO.event_batch(ev.K, ev.V, ev.pos, ev.qstat, ev.p_ref, ev.budget, lam, W=W, base=ev.rope_base,
                             eps=ev.eps, threads=threads, want_rows=False, budgets=budgets)
    todo = range(E) if events is None else events
    for e in todo:
        b, l, h = e // (L * H), (e // H) % L, e % H
        n = N if n_cand is None else int(n_cand[b])
        k_e = ev.budget if budgets is None else int(budgets[l][h])
        chk.check_event(ev.K[b, l, h], ev.V[b, l, h], ev.pos[b, l, h], ev.qstat[l, h],
                        int(ev.p_ref[b]) if p_ref else None, k_e, lam,
                        g["scores"][b, l, h], g["order"][b, l, h], g["idx"][b, l, h],
                        g["K"][b, l, h], g["V"][b, l, h], g["pos"][b, l, h], W=W, base=ev.rope_base, eps=ev.eps,
                        ref_scores=None if ref is None else ref["scores"][b, l, h],
                        ref_order=None if ref is None else ref["order"][b, l, h], n=n, log=log)
        assert g["n_kept"][b, l, h] == min(k_e, n)
        assert g["status"][b, l, h] == (2 if n < k_e else 0)
    return log


# ------------------------------------------------------------------ small shapes: several tiles, ragged tails
@pytest.mark.parametrize("dtype", [synth.BF16, synth.F32])
@pytest.mark.parametrize("N,d,budget", [(100, 128, 37), (77, 64, 77), (192, 128, 64), (33, 16, 5), (130, 256, 40),
                                        (50, 8, 20), (96, 40, 31)])
@pytest.mark.parametrize("lam", [0.0, 0.5, 1.5])
def test_fused_event_small(dtype, N, d, budget, lam):
    ev = synth.make_c3(seed=N + d, B=2, L=2, H=3, N=N, budget=budget) if d == 128 else \
        synth.make_plain(2, 2, 3, N, d, budget, lam, dtype=dtype, seed=N + d)
    if d == 128 and dtype == synth.F32:
        ev = synth.make_plain(2, 2, 3, N, d, budget, lam, dtype=dtype, seed=N + d)
    g = run_fused(ev, lam=lam)
    check_all(ev, g, lam)


def test_lambda0_greedy_loop_equals_fast_path_equals_topk():
    ev = synth.make_plain(2, 3, 2, 150, 128, 50, 0.0, dtype=synth.BF16, seed=3)
    fast = run_fused(ev, lam=0.0)
    loop = run_fused(ev, lam=0.0, flags=akv.FLAG_FORCE_GREEDY)
    assert np.array_equal(fast["order"], loop["order"]) and np.array_equal(fast["idx"], loop["idx"])
    assert np.array_equal(fast["K"][..., :50, :], loop["K"][..., :50, :])
    # top-k of the GPU's own scores, ties to the lower index
    for b in range(2):
        for l in range(3):
            for h in range(2):
                s = fast["scores"][b, l, h].astype(np.float64)
                assert fast["order"][b, l, h].tolist() == O.topk_indices(s, 50).tolist()


def test_ragged_candidate_counts_and_short_events():
    ev = synth.make_plain(4, 2, 2, 120, 128, 40, 0.5, dtype=synth.BF16, seed=9)
    n_cand = [120, 41, 40, 17]          # last one is below the budget: keep all, status 2
    g = run_fused(ev, n_cand=n_cand)
    check_all(ev, g, 0.5, n_cand=n_cand)
    # rows beyond n_cand were never read as candidates: no index >= n_cand
    for b, n in enumerate(n_cand):
        kept = min(40, n)
        assert g["idx"][b, :, :, :kept].max() < n


def test_default_reference_position_and_future_window():
    ev = synth.make_plain(2, 2, 2, 90, 128, 30, 0.5, dtype=synth.BF16, seed=12)
    ev.pos[:] = (np.sort(np.random.default_rng(1).choice(5000, size=90, replace=False))).astype(np.int32)
    g = run_fused(ev, p_ref=False, W=4)
    check_all(ev, g, 0.5, p_ref=False, W=4)


def test_large_positions_keep_score_accuracy():
    ev = synth.make_plain(1, 2, 2, 64, 128, 16, 0.5, dtype=synth.BF16, seed=13)
    ev.pos[:] = (1_000_000 + np.arange(64) * 997).astype(np.int32)
    ev.p_ref[:] = 1_100_000
    g = run_fused(ev)
    check_all(ev, g, 0.5)


def test_repeat_runs_are_bit_identical():
    ev = synth.make_c3(seed=4, B=2, L=2, H=2, N=192, budget=64)
    a, b = run_fused(ev), run_fused(ev)
    for k in ("K", "V", "pos", "idx", "order", "scores", "gain"):
        assert np.array_equal(a[k], b[k]), k


def test_nonfinite_scores_are_flagged_and_never_preferred():
    ev = synth.make_plain(1, 1, 2, 64, 128, 20, 0.5, dtype=synth.F32, seed=14)
    ev.K[0, 0, 0, 5, 3] = np.inf
    ev.K[0, 0, 0, 9, 100] = np.nan
    g = run_fused(ev)
    assert g["status"][0, 0, 0] == 1 and g["status"][0, 0, 1] == 0
    assert not ({5, 9} & set(g["idx"][0, 0, 0].tolist()))
    assert len(set(g["idx"][0, 0, 0].tolist())) == 20


# ------------------------------------------------------------------ stand-alone entry points
@pytest.mark.parametrize("dtype", [synth.BF16, synth.F32])
def test_score_select_compact_chain_equals_fused(dtype):
    ev = synth.make_c3(seed=21, B=2, L=2, H=2, N=160, budget=48) if dtype == synth.BF16 else \
        synth.make_plain(2, 2, 2, 160, 128, 48, 0.5, dtype=dtype, seed=21)
    fused = run_fused(ev)
    K, V, pos, q, pref = dev(ev.K), dev(ev.V), dev(ev.pos), dev(ev.qstat), dev(ev.p_ref)
    opts = akv.Options(lam=ev.lam)
    status = torch.full((2, 2, 2), -7, dtype=torch.int32, device="cuda")
    s = akv.alpha_score(K, q, pos=pos, p_ref=pref, opts=opts, status=status)
    # the stand-alone scorer and the fused kernel may round differently in the last place
    assert np.max(np.abs(s.cpu().numpy() - fused["scores"])) < 2e-6
    # fed the very same scores, the stand-alone selection must reproduce the fused one's picks
    sel = akv.alpha_select(dev(fused["scores"]), V, ev.budget, opts)
    akv.kv_compact(K, V, pos, sel.idx_sorted)
    torch.cuda.synchronize()
    assert np.array_equal(sel.pick_order.cpu().numpy(), fused["order"])
    assert np.array_equal(sel.idx_sorted.cpu().numpy(), fused["idx"])
    # (the gains themselves may differ in the last place: the two routes sum a row's products in different orders)
    assert np.max(np.abs(sel.pick_gain.cpu().numpy() - fused["gain"])) < 1e-6
    assert np.array_equal(akv.to_host_bits(K)[..., :48, :], fused["K"][..., :48, :])
    assert np.array_equal(akv.to_host_bits(V)[..., :48, :], fused["V"][..., :48, :])
    assert np.array_equal(pos.cpu().numpy()[..., :48], fused["pos"][..., :48])
    assert int(status.abs().max()) == 0


def test_score_only_broadcast_positions_and_rotated_cache():
    ev = synth.make_plain(2, 3, 2, 70, 128, 10, 0.5, dtype=synth.BF16, seed=22)
    K, q = dev(ev.K), dev(ev.qstat)
    pos1 = dev(np.arange(70, dtype=np.int32) * 3)
    s = akv.alpha_score(K, q, pos=pos1, p_ref=dev(np.array([400, 500], dtype=np.int32)),
                        opts=akv.Options(future_window=3)).cpu().numpy()
    s0 = akv.alpha_score(K, q, pos=None).cpu().numpy()
    for b in range(2):
        for l in range(3):
            for h in range(2):
                ref = O.triattention_score(ev.K[b, l, h], np.arange(70) * 3, ev.qstat[l, h], [400, 500][b], 3)
                chk.check_scores(s[b, l, h], ref, chk.score_scale(ev.K[b, l, h], ev.qstat[l, h], 128))
                ref0 = O.triattention_score(ev.K[b, l, h], None, ev.qstat[l, h], None)
                chk.check_scores(s0[b, l, h], ref0, chk.score_scale(ev.K[b, l, h], ev.qstat[l, h], 128))


def test_select_given_scores_matches_oracle_and_duplicate_pair_closed_form():
    P, d = 40, 128
    s, V, leaders = synth.make_duplicate_pairs(P, d, 0.01, seed=2, dtype=synth.BF16)
    lam = float(s[0] - 0.01 - s[2 * (P - 1)]) + 0.05
    sc = torch.tensor(s, dtype=torch.float32, device="cuda").reshape(1, 1, 1, -1).contiguous()
    Vd = dev(V.reshape(1, 1, 1, 2 * P, d))
    for b in (1, 7, P):
        sel = akv.alpha_select(sc, Vd, b, akv.Options(lam=lam))
        assert sel.idx_sorted.cpu().numpy().ravel().tolist() == leaders[:b].tolist()
    top = akv.alpha_select(sc, Vd, 6, akv.Options(lam=0.0)).idx_sorted.cpu().numpy().ravel().tolist()
    assert top == sorted(sorted(range(2 * P), key=lambda i: (-np.float32(s[i]), i))[:6])


def test_compact_in_place_aliasing_and_negative_tail():
    ev = synth.make_plain(2, 2, 2, 64, 128, 20, 0.5, dtype=synth.BF16, seed=23)
    K, V, pos = dev(ev.K), dev(ev.V), dev(ev.pos)
    idx = np.zeros((2, 2, 2, 20), dtype=np.int32)
    idx[...] = np.arange(1, 21)                 # every destination is another row's source
    idx[1, 1, 1] = np.r_[np.arange(5, 64, 4)[:15], -1, -1, -1, -1, -1]
    akv.kv_compact(K, V, pos, dev(idx))
    torch.cuda.synchronize()
    Kn, Vn, pn = akv.to_host_bits(K), akv.to_host_bits(V), pos.cpu().numpy()
    for b in range(2):
        for l in range(2):
            for h in range(2):
                ii = idx[b, l, h]
                ii = ii[ii >= 0]
                assert np.array_equal(Kn[b, l, h, :len(ii)], ev.K[b, l, h][ii])
                assert np.array_equal(Vn[b, l, h, :len(ii)], ev.V[b, l, h][ii])
                assert np.array_equal(pn[b, l, h, :len(ii)], ev.pos[b, l, h][ii])
                assert np.array_equal(Kn[b, l, h, 21:], ev.K[b, l, h, 21:])     # untouched beyond the moved range


def test_flat_signature_eq1_and_selection_with_it():
    ev = synth.make_plain(2, 3, 2, 80, 128, 25, 0.7, dtype=synth.BF16, seed=24)
    V = dev(ev.V)
    sig = akv.alpha_signature_flat(V).cpu().numpy()
    for b in range(2):
        ref = O.signatures_flat(ev.V[b])
        assert np.max(np.abs(sig[b] - ref)) < 2e-7
    K, pos, q, pref = dev(ev.K), dev(ev.pos), dev(ev.qstat), dev(ev.p_ref)
    opts = akv.Options(lam=0.7, sig_mode=akv.SIG_FLAT)
    sel = akv.alpha_compress_event(K, V, pos, q, 25, opts, p_ref=pref, flat_sig=dev(sig), want_scores=True)
    torch.cuda.synchronize()
    Kn, Vn, pn = akv.to_host_bits(K), akv.to_host_bits(V), pos.cpu().numpy()
    for b in range(2):
        ref_sig = O.signatures_flat(ev.V[b])
        for l in range(3):
            for h in range(2):
                chk.check_event(ev.K[b, l, h], ev.V[b, l, h], ev.pos[b, l, h], ev.qstat[l, h], int(ev.p_ref[b]), 25, 0.7,
                                sel.scores[b, l, h].cpu().numpy(), sel.pick_order[b, l, h].cpu().numpy(),
                                sel.idx_sorted[b, l, h].cpu().numpy(), Kn[b, l, h], Vn[b, l, h], pn[b, l, h], sig=ref_sig)


def test_three_launch_path_for_events_that_do_not_fit_on_chip():
    """fp32 with N = 600 exceeds shared memory: score -> select -> compact with scratch scores."""
    ev = synth.make_plain(1, 2, 2, 600, 128, 50, 0.5, dtype=synth.F32, seed=25)
    K, V, pos, q, pref = dev(ev.K), dev(ev.V), dev(ev.pos), dev(ev.qstat), dev(ev.p_ref)
    sel = akv.alpha_compress_event(K, V, pos, q, 50, akv.Options(lam=0.5), p_ref=pref, want_scores=False)
    torch.cuda.synchronize()
    g = dict(K=akv.to_host_bits(K), V=akv.to_host_bits(V), pos=pos.cpu().numpy(), idx=sel.idx_sorted.cpu().numpy(),
             order=sel.pick_order.cpu().numpy(), n_kept=sel.n_kept.cpu().numpy(), status=sel.status.cpu().numpy())
    g["scores"] = akv.alpha_score(dev(ev.K), q, pos=dev(ev.pos), p_ref=pref).cpu().numpy()
    check_all(ev, g, 0.5)


def test_invalid_arguments_launch_nothing():
    ev = synth.make_plain(1, 1, 1, 32, 128, 8, 0.5, dtype=synth.BF16, seed=26)
    K, V, pos, q = dev(ev.K), dev(ev.V), dev(ev.pos), dev(ev.qstat)
    before = akv.launch_count()
    with pytest.raises(akv.AkvError) as e:
        akv.alpha_compress_event(K, V, pos, q, 33)
    assert e.value.code == 3
    with pytest.raises(akv.AkvError) as e:
        akv.alpha_compress_event(K, V, pos, q, 8, akv.Options(lam=-1.0))
    assert e.value.code == 1
    with pytest.raises(akv.AkvError) as e:
        akv.alpha_compress_event(K.view(torch.int16)[..., 1:].view(torch.bfloat16) if False else K, V, pos, q, 8,
                                 akv.Options(sig_mode=akv.SIG_FLAT))
    assert e.value.code == 1
    Kodd = torch.empty(32 * 128 + 8, dtype=torch.bfloat16, device="cuda")[4:4 + 32 * 128].view(1, 1, 1, 32, 128)
    with pytest.raises(akv.AkvError) as e:
        akv.alpha_score(Kodd, q)
    assert e.value.code == 4
    assert akv.launch_count() == before
    assert np.array_equal(akv.to_host_bits(K), ev.K)


# ------------------------------------------------------------------ events longer than the 128-row K tile
@pytest.mark.parametrize("N,budget", [(129, 48), (144, 64), (250, 33), (256, 64)])
def test_k_rows_beyond_the_tile_arrive_in_freed_slots(N, budget):
    """bf16, d = 128, budget <= 64: the kernel holds 128 K rows at a time; rows from 128 on are scored from
    the slots of the first rows. Ragged counts put the boundary inside, at and just after the tile."""
    ev = synth.make_c3(seed=N, B=4, L=2, H=2, N=N, budget=budget)
    g = run_fused(ev)
    check_all(ev, g, ev.lam)
    n_cand = [N, min(N, 129), 128, min(N, 131)]
    g = run_fused(ev, n_cand=n_cand)
    check_all(ev, g, ev.lam, n_cand=n_cand)


@pytest.mark.parametrize("page,pages_per_seq", [(64, 4), (32, 6), (256, 1)])
def test_paged_event_longer_than_the_tile(page, pages_per_seq):
    """Paged cache (page sizes are powers of two), budget 64: K pages are copied whole, a 256-slot page in two
    pieces around row 128."""
    c5 = synth.make_c5(seed=page, B=3, L=2, H=2, page=page, pages_per_seq=pages_per_seq, budget=64, rounds=1)
    L, H, N, d, b = c5.L, c5.H, c5.N, c5.d, c5.budget
    pool_K, pool_V = dev(c5.pool_K), dev(c5.pool_V)
    table, pos, q = dev(c5.block_table), dev(c5.pos), dev(c5.qstat)
    lay = akv.Layout.paged(pool_K, table)
    hostK = synth.paged_gather_dense(c5.pool_K, c5.block_table)
    hostV = synth.paged_gather_dense(c5.pool_V, c5.block_table)
    sel = akv.alpha_compress_event(pool_K, pool_V, pos, q, b, akv.Options(lam=c5.lam), layout=lay, want_scores=True)
    torch.cuda.synchronize()
    idx, order, sc = sel.idx_sorted.cpu().numpy(), sel.pick_order.cpu().numpy(), sel.scores.cpu().numpy()
    posn = pos.cpu().numpy()
    for bb in range(c5.B):
        pages = c5.block_table[bb].tolist()
        for l in range(L):
            for h in range(H):
                Kn = akv.to_host_bits(pool_K[l, pages, h]).reshape(N, d)
                Vn = akv.to_host_bits(pool_V[l, pages, h]).reshape(N, d)
                chk.check_event(hostK[bb, l, h], hostV[bb, l, h], c5.pos[bb, l, h], c5.qstat[l, h], None, b, c5.lam,
                                sc[bb, l, h], order[bb, l, h], idx[bb, l, h], Kn, Vn, posn[bb, l, h], log=[])


@pytest.mark.parametrize("maker", ["c3_192", "c2_256", "f32_96"])
def test_pool_pruning_changes_no_pick(maker):
    """The pool that Algorithm 1 runs over is pruned exactly: with pruning switched off (every candidate in the
    pool, which takes the kernels' large-pool routes) the picks, their order and the compacted rows are the same."""
    if maker == "c3_192":
        ev = synth.make_c3(seed=21, B=2, L=2, H=2, N=192, budget=64)
    elif maker == "c2_256":
        ev = synth.make_c2(seed=22, B=1, L=2, H=2)
    else:
        ev = synth.make_plain(2, 2, 2, 96, 64, 30, 0.5, dtype=synth.F32, seed=23)
    pruned = run_fused(ev)
    full = run_fused(ev, flags=akv.FLAG_NO_PRUNE)
    for k in ("order", "idx", "K", "V", "pos", "n_kept", "status"):
        assert np.array_equal(pruned[k], full[k]), k
    check_all(ev, full, ev.lam)


def test_reference_position_behind_some_keys():
    """Keys ahead of the reference position have negative distances; the fast kernel measures distances from
    the last key and turns the query statistic by the difference. Positions are sparse and large."""
    ev = synth.make_c3(seed=31, B=3, L=2, H=2, N=192, budget=64)
    rng = np.random.default_rng(31)
    ev.pos[:] = np.sort(rng.choice(3_000_000, size=192, replace=False)).astype(np.int32)
    ev.p_ref[:] = np.array([ev.pos[0, 0, 0, 100], ev.pos[0, 0, 0, 0] - 5, ev.pos[0, 0, 0, -1]], dtype=ev.p_ref.dtype)
    g = run_fused(ev)
    check_all(ev, g, ev.lam)


# ------------------------------------------------------------------ per-layer signatures, per-head budgets (Section 6)
@pytest.mark.parametrize("dtype,N,d", [(synth.BF16, 80, 128), (synth.F32, 600, 64)])
def test_per_layer_signature_mode(dtype, N, d):
    """Signatures averaged over the heads of one layer: the reduction, and the event that selects with it
    (resident kernel for the small shape, three launches for the large one)."""
    ev = synth.make_plain(2, 3, 2, N, d, 25, 0.7, dtype=dtype, seed=27)
    V = dev(ev.V)
    sig = akv.alpha_signature_layer(V).cpu().numpy()
    assert sig.shape == (2, 3, N, d)
    for b in range(2):
        for l in range(3):
            assert np.max(np.abs(sig[b, l] - O.signatures_per_layer(ev.V[b, l]))) < 2e-7
    K, pos, q, pref = dev(ev.K), dev(ev.pos), dev(ev.qstat), dev(ev.p_ref)
    opts = akv.Options(lam=0.7, sig_mode=akv.SIG_PER_LAYER)
    sel = akv.alpha_compress_event(K, V, pos, q, 25, opts, p_ref=pref, flat_sig=dev(sig), want_scores=True)
    torch.cuda.synchronize()
    Kn, Vn, pn = akv.to_host_bits(K), akv.to_host_bits(V), pos.cpu().numpy()
    for b in range(2):
        for l in range(3):
            ref_sig = O.signatures_per_layer(ev.V[b, l])
            for h in range(2):
                chk.check_event(ev.K[b, l, h], ev.V[b, l, h], ev.pos[b, l, h], ev.qstat[l, h], int(ev.p_ref[b]), 25, 0.7,
                                sel.scores[b, l, h].cpu().numpy(), sel.pick_order[b, l, h].cpu().numpy(),
                                sel.idx_sorted[b, l, h].cpu().numpy(), Kn[b, l, h], Vn[b, l, h], pn[b, l, h], sig=ref_sig)


@pytest.mark.parametrize("maker", ["c3_192", "c2_256", "f32_96", "f32_600"])
def test_per_head_budgets(maker):
    """A budget per (layer, head): every kernel family keeps budgets[l, h] rows per event, pads its index rows
    to the largest budget with -1 and reports the kept count; uniform budgets equal the scalar call."""
    if maker == "c3_192":
        ev = synth.make_c3(seed=41, B=2, L=3, H=2, N=192, budget=64)
    elif maker == "c2_256":
        ev = synth.make_c2(seed=42, B=2, L=3, H=2)
    elif maker == "f32_96":
        ev = synth.make_plain(2, 3, 2, 96, 64, 30, 0.5, dtype=synth.F32, seed=43)
    else:
        ev = synth.make_plain(2, 3, 2, 600, 128, 50, 0.5, dtype=synth.F32, seed=44)
    kmax = ev.budget
    rng = np.random.default_rng(7)
    budgets = rng.integers(1, kmax + 1, size=(3, 2)).astype(np.int32)
    budgets[0, 0], budgets[2, 1] = kmax, 1
    g = run_fused(ev, budgets=budgets)
    check_all(ev, g, ev.lam, budgets=budgets)
    assert int(g["n_kept"].sum()) == 2 * int(budgets.sum())
    scalar = run_fused(ev)
    uniform = run_fused(ev, budgets=np.full((3, 2), kmax, dtype=np.int32))
    for k in ("order", "idx", "K", "V", "pos", "n_kept", "status"):
        assert np.array_equal(scalar[k], uniform[k]), k


# ------------------------------------------------------------------ bounded waits, workspace query, large grids
@pytest.mark.parametrize("maker", ["tri_192", "tri_96", "tc_256"])
def test_bounded_wait_runs_out_and_reports_status_3(maker):
    """With the starve flag no K row is requested and the waits poll only a few times: every wait of the fused
    tensor-memory kernels runs out with nothing in flight, each event reports status 3, tensor memory is given
    back (the next, normal call runs) and K, V and positions are left as they were."""
    if maker == "tri_192":
        ev = synth.make_c3(seed=51, B=2, L=2, H=2, N=192, budget=64)
    elif maker == "tri_96":
        ev = synth.make_c3(seed=52, B=2, L=2, H=2, N=96, budget=40)
    else:
        ev = synth.make_c2(seed=53, B=2, L=2, H=2)
    g = run_fused(ev, flags=akv.FLAG_TEST_STARVE_WAIT)
    assert np.all(g["status"] == 3)
    assert np.array_equal(g["K"], ev.K) and np.array_equal(g["V"], ev.V) and np.array_equal(g["pos"], ev.pos)
    good = run_fused(ev)
    check_all(ev, good, ev.lam)


def test_workspace_query_matches_the_route():
    bf = akv.Layout(2, 2, 2, 192, 128, akv.api.AKV_BF16, (2 * 2 * 192 * 128, 2 * 192 * 128, 192 * 128, 128))
    assert akv.workspace_bytes(bf, 64) == 0                                  # on chip, one launch
    f32_small = akv.Layout(1, 1, 1, 192, 128, akv.api.AKV_F32, (192 * 128,) * 3 + (128,))
    assert akv.workspace_bytes(f32_small, 64) == 0                           # tiles resident in shared memory
    f32_big = akv.Layout(1, 2, 2, 600, 128, akv.api.AKV_F32, (4 * 600 * 128, 2 * 600 * 128, 600 * 128, 128))
    assert akv.workspace_bytes(f32_big, 50) == 1 * 2 * 2 * 600 * 4          # the scores between the launches
    bf_big = akv.Layout(1, 2, 2, 4096, 128, akv.api.AKV_BF16, (4 * 4096 * 128, 2 * 4096 * 128, 4096 * 128, 128))
    assert akv.workspace_bytes(bf_big, 128) == 0                             # streaming kernel, scores stay on chip


def test_score_with_more_events_than_a_grid_dimension_holds():
    """70 000 events: the event index is folded into grid.x, which has room for them."""
    B, N, d = 70_000, 8, 8
    rng = np.random.default_rng(61)
    K = rng.standard_normal((B, 1, 1, N, d)).astype(np.float32)
    q = rng.standard_normal((1, 1, d)).astype(np.float32)
    s = akv.alpha_score(dev(K), dev(q), pos=dev(np.arange(N, dtype=np.int32)),
                        p_ref=dev(np.full(B, N, dtype=np.int32))).cpu().numpy()
    for b in (0, 1, 65_535, 65_536, B - 1):
        ref = O.triattention_score(K[b, 0, 0], np.arange(N), q[0, 0], N)
        chk.check_scores(s[b, 0, 0], ref, chk.score_scale(K[b, 0, 0], q[0, 0], d))


# ------------------------------------------------------------------ large pools: the streaming one-launch kernel
@pytest.mark.parametrize("N,budget,lam", [(257, 40, 0.5), (300, 128, 0.0), (1000, 64, 0.5), (1000, 100, 1.5), (2050, 128, 1.0)])
def test_large_pool_stream_kernel(N, budget, lam):
    """bf16, d = 128, N > 256: K streams through a ring, scores stay on chip, pool rows of V only. Ragged
    candidate counts put the end of an event inside a ring stage, at its edge, and below the budget."""
    ev = synth.make_c3(seed=N, B=4, L=1, H=2, N=N, budget=budget)
    before = akv.launch_count()
    g = run_fused(ev, lam=lam)
    assert akv.launch_count() == before + 1                                   # one launch for the whole event
    check_all(ev, g, lam)
    n_cand = [N, N - 63, 64 * (N // 64), budget - 3]
    g = run_fused(ev, lam=lam, n_cand=n_cand)
    check_all(ev, g, lam, n_cand=n_cand)


def test_large_pool_stream_kernel_variants():
    """Same kernel: no pruning (the pool outgrows the on-chip tile, the rest of V is read in place), the greedy
    loop forced at lambda = 0, per-head budgets, irregular positions with the default reference position, every
    row scored from scratch, and the bounded waits running out."""
    ev = synth.make_c3(seed=71, B=2, L=2, H=2, N=900, budget=48)
    base = run_fused(ev)
    check_all(ev, base, ev.lam)
    full = run_fused(ev, flags=akv.FLAG_NO_PRUNE)
    for k in ("order", "idx", "K", "V", "pos"):
        assert np.array_equal(base[k], full[k]), k
    fast, loop = run_fused(ev, lam=0.0), run_fused(ev, lam=0.0, flags=akv.FLAG_FORCE_GREEDY)
    assert np.array_equal(fast["order"], loop["order"]) and np.array_equal(fast["K"], loop["K"])
    check_all(ev, fast, 0.0)
    budgets = np.array([[48, 1], [17, 30]], dtype=np.int32)
    check_all(ev, run_fused(ev, budgets=budgets), ev.lam, budgets=budgets)
    fresh = run_fused(ev, flags=akv.FLAG_NO_CHAIN)
    assert np.max(np.abs(fresh["scores"] - base["scores"])) < 2e-6
    check_all(ev, fresh, ev.lam)
    ev.pos[:] = np.sort(np.random.default_rng(72).choice(200_000, size=900, replace=False)).astype(np.int32)
    g = run_fused(ev, p_ref=False)
    check_all(ev, g, ev.lam, p_ref=False)
    starved = run_fused(ev, flags=akv.FLAG_TEST_STARVE_WAIT)
    assert np.all(starved["status"] == 3)
    assert np.array_equal(starved["K"], ev.K) and np.array_equal(starved["V"], ev.V) and np.array_equal(starved["pos"], ev.pos)


def test_large_pool_stream_kernel_paged():
    c5 = synth.make_c5(seed=73, B=2, L=2, H=2, page=64, pages_per_seq=9, budget=100, rounds=1)   # N = 576
    L, H, N, d, b = c5.L, c5.H, c5.N, c5.d, c5.budget
    pool_K, pool_V = dev(c5.pool_K), dev(c5.pool_V)
    table, pos, q = dev(c5.block_table), dev(c5.pos), dev(c5.qstat)
    lay = akv.Layout.paged(pool_K, table)
    hostK = synth.paged_gather_dense(c5.pool_K, c5.block_table)
    hostV = synth.paged_gather_dense(c5.pool_V, c5.block_table)
    sel = akv.alpha_compress_event(pool_K, pool_V, pos, q, b, akv.Options(lam=c5.lam), layout=lay, want_scores=True)
    torch.cuda.synchronize()
    idx, order, sc = sel.idx_sorted.cpu().numpy(), sel.pick_order.cpu().numpy(), sel.scores.cpu().numpy()
    posn = pos.cpu().numpy()
    for bb in range(c5.B):
        pages = c5.block_table[bb].tolist()
        for l in range(L):
            for h in range(H):
                Kn = akv.to_host_bits(pool_K[l, pages, h]).reshape(N, d)
                Vn = akv.to_host_bits(pool_V[l, pages, h]).reshape(N, d)
                chk.check_event(hostK[bb, l, h], hostV[bb, l, h], c5.pos[bb, l, h], c5.qstat[l, h], None, b, c5.lam,
                                sc[bb, l, h], order[bb, l, h], idx[bb, l, h], Kn, Vn, posn[bb, l, h], log=[])


def test_chained_and_fresh_scores_agree_on_the_tensor_memory_kernels():
    for ev in (synth.make_c3(seed=81, B=2, L=2, H=2, N=192, budget=64), synth.make_c2(seed=82, B=1, L=2, H=2)):
        a, b = run_fused(ev), run_fused(ev, flags=akv.FLAG_NO_CHAIN)
        scale = np.abs(a["scores"]).max()
        assert np.max(np.abs(a["scores"] - b["scores"])) < 1e-6 * max(scale, 1.0)
        check_all(ev, b, ev.lam)


# ------------------------------------------------------------------ shared signatures with one cosine matrix per sequence
@pytest.mark.parametrize("mode", ["flat", "layer"])
@pytest.mark.parametrize("N", [96, 256, 300])
def test_shared_cosine_matrix(mode, N):
    """Algorithm 1's cosine matrix of the shared signatures, once per sequence (Eq. 1) or per sequence and layer:
    three-part bf16 split on the tensor cores against the float64 product, with a ragged candidate count."""
    ev = synth.make_plain(2, 2, 3, N, 128, 16, 0.5, dtype=synth.BF16, seed=90 + N)
    V = dev(ev.V)
    n_cand = np.array([N, N - 37], dtype=np.int32)
    nc = dev(n_cand)
    lay = akv.Layout.dense(V)
    if mode == "flat":
        opts = akv.Options(sig_mode=akv.SIG_FLAT)
        sig = akv.alpha_signature_flat(V, n_cand=nc)
    else:
        opts = akv.Options(sig_mode=akv.SIG_PER_LAYER)
        sig = akv.alpha_signature_layer(V, n_cand=nc)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    gram = akv.alpha_gram_shared(sig, lay, opts, n_cand=nc, status=status).cpu().numpy()
    assert int(status.item()) == 0
    for b in range(2):
        n = int(n_cand[b])
        groups = [None] if mode == "flat" else range(2)
        for l in groups:
            ref_sig = O.signatures_flat(ev.V[b][:, :, :n]) if l is None else O.signatures_per_layer(ev.V[b, l][:, :n])
            got = gram[b][:n, :n] if l is None else gram[b, l][:n, :n]
            assert np.max(np.abs(got - ref_sig @ ref_sig.T)) < 5e-7
            rest = gram[b][n:] if l is None else gram[b, l][n:]
            assert np.all(rest == 0)                                  # rows beyond the candidates are left alone


@pytest.mark.parametrize("mode,N,budget", [("flat", 256, 128), ("flat", 192, 64), ("layer", 256, 100), ("flat", 130, 20)])
def test_fused_event_with_shared_cosine_matrix(mode, N, budget):
    """Shared signatures in the fused path: signature pass, one cosine matrix per sequence (and layer), then every
    event of the sequence in ONE launch that reads its cosines from that matrix. Checked against the oracle with
    the float64 signatures, and against the general route (dot products of signature rows pick by pick)."""
    ev = synth.make_c3(seed=95 + N, B=2, L=3, H=2, N=N, budget=budget)
    lam = 0.7
    K, V, pos, q, pref = dev(ev.K), dev(ev.V), dev(ev.pos), dev(ev.qstat), dev(ev.p_ref)
    lay = akv.Layout.dense(V)
    smode = akv.SIG_FLAT if mode == "flat" else akv.SIG_PER_LAYER
    sig = akv.alpha_signature_flat(V) if mode == "flat" else akv.alpha_signature_layer(V)
    gram = akv.alpha_gram_shared(sig, lay, akv.Options(sig_mode=smode))
    K2, V2, pos2 = K.clone(), V.clone(), pos.clone()
    before = akv.launch_count()
    sel = akv.alpha_compress_event(K, V, pos, q, budget, akv.Options(lam=lam, sig_mode=smode, shared_gram=gram), p_ref=pref,
                                   flat_sig=sig, want_scores=True)
    assert akv.launch_count() == before + 1
    ref = akv.alpha_compress_event(K2, V2, pos2, q, budget, akv.Options(lam=lam, sig_mode=smode), p_ref=pref, flat_sig=sig)
    torch.cuda.synchronize()
    Kn, Vn, pn = akv.to_host_bits(K), akv.to_host_bits(V), pos.cpu().numpy()
    n_same = 0
    for b in range(2):
        for l in range(3):
            ref_sig = O.signatures_flat(ev.V[b]) if mode == "flat" else O.signatures_per_layer(ev.V[b, l])
            for h in range(2):
                chk.check_event(ev.K[b, l, h], ev.V[b, l, h], ev.pos[b, l, h], ev.qstat[l, h], int(ev.p_ref[b]), budget, lam,
                                sel.scores[b, l, h].cpu().numpy(), sel.pick_order[b, l, h].cpu().numpy(),
                                sel.idx_sorted[b, l, h].cpu().numpy(), Kn[b, l, h], Vn[b, l, h], pn[b, l, h], sig=ref_sig)
                n_same += int(torch.equal(sel.pick_order[b, l, h], ref.pick_order[b, l, h]))
    assert n_same >= 11                                               # the two routes round differently: near-ties may differ
    assert int(sel.status.abs().max()) == 0 and int(sel.n_kept.min()) == budget


def _duplicated_rows(seed, lam, B=2, L=2, H=2, N=256, budget=128):
    """Every V row occurs twice (rows j and j + N/2 are bit-identical): once a row is picked its twin is
    penalised by lambda, so the picks must go far down the score order, beyond any active set."""
    ev = synth.make_plain(B, L, H, N, 128, budget, lam, dtype=synth.BF16, seed=seed)
    ev.V[..., N // 2:, :] = ev.V[..., :N // 2, :]
    return ev


@pytest.mark.parametrize("lam", [2.0, 1.5])
def test_active_set_bound_reached_and_the_loop_continues_over_the_whole_pool(lam):
    """N = 256 -> b = 128 with duplicated V rows: the one-warp loop over the best-scored rows reaches its bound;
    the picks made stand, the rest are taken over the whole pool. Every pick is checked against the oracle."""
    ev = _duplicated_rows(33, lam)
    g = run_fused(ev, lam=lam)
    log = check_all(ev, g, lam)
    # the picks did go deep: some kept row's score rank lies beyond the 180 rows an active set holds at most
    s = g["scores"][0, 0, 0]
    rank = np.argsort(np.argsort(-s))
    assert rank[g["idx"][0, 0, 0]].max() >= 181
    print("duplicated rows, lambda", lam, "near-tie divergences:", log)


def test_active_set_bound_reached_with_a_shared_cosine_matrix():
    """The same with Eq. 1 signatures and one cosine matrix per sequence (one layer, one head: the flat signature
    is the head's own), so the continuation reads its cosines from that matrix."""
    lam = 1.5
    ev = _duplicated_rows(34, lam, B=2, L=1, H=1)
    K, V, pos, q, pref = dev(ev.K), dev(ev.V), dev(ev.pos), dev(ev.qstat), dev(ev.p_ref)
    sig = akv.alpha_signature_flat(V)
    gram = akv.alpha_gram_shared(sig, akv.Layout.dense(V), akv.Options(sig_mode=akv.SIG_FLAT))
    sel = akv.alpha_compress_event(K, V, pos, q, ev.budget, akv.Options(lam=lam, sig_mode=akv.SIG_FLAT, shared_gram=gram),
                                   p_ref=pref, flat_sig=sig, want_scores=True)
    torch.cuda.synchronize()
    Kn, Vn, pn = akv.to_host_bits(K), akv.to_host_bits(V), pos.cpu().numpy()
    for b in range(2):
        chk.check_event(ev.K[b, 0, 0], ev.V[b, 0, 0], ev.pos[b, 0, 0], ev.qstat[0, 0], int(ev.p_ref[b]), ev.budget, lam,
                        sel.scores[b, 0, 0].cpu().numpy(), sel.pick_order[b, 0, 0].cpu().numpy(),
                        sel.idx_sorted[b, 0, 0].cpu().numpy(), Kn[b, 0, 0], Vn[b, 0, 0], pn[b, 0, 0],
                        sig=O.signatures_flat(ev.V[b]))
    assert int(sel.status.abs().max()) == 0 and int(sel.n_kept.min()) == ev.budget


# ------------------------------------------------------------------ grouped-query statistics
@pytest.mark.parametrize("reduce", ["mean", "max"])
@pytest.mark.parametrize("dtype,N,d", [(synth.BF16, 150, 128), (synth.F32, 600, 64)])
def test_grouped_query_statistics(reduce, dtype, N, d):
    """Several query statistics per KV head: scores are the mean or the maximum over the group (stand-alone scorer),
    and the fused call selects with them (resident kernel for the small shape, three launches for the large one)."""
    G = 4
    ev = synth.make_plain(2, 2, 2, N, d, 30, 0.5, dtype=dtype, seed=101)
    rng = np.random.default_rng(102)
    Q = rng.standard_normal((2, 2 * G, d)).astype(np.float32)            # [L, H * G, d]
    K, V, pos, pref = dev(ev.K), dev(ev.V), dev(ev.pos), dev(ev.p_ref)
    opts = akv.Options(lam=0.5, gqa_group=G, gqa_reduce=akv.GQA_MAX if reduce == "max" else akv.GQA_MEAN)
    s = akv.alpha_score(K, dev(Q), pos=pos, p_ref=pref, opts=opts).cpu().numpy()
    sel = akv.alpha_compress_event(K, V, pos, dev(Q), 30, opts, p_ref=pref, want_scores=True)
    torch.cuda.synchronize()
    Kn, Vn, pn = akv.to_host_bits(K), akv.to_host_bits(V), pos.cpu().numpy()
    for b in range(2):
        for l in range(2):
            for h in range(2):
                qs = Q[l, h * G:(h + 1) * G]
                ref = O.triattention_score_group(ev.K[b, l, h], ev.pos[b, l, h], qs, int(ev.p_ref[b]), reduce=reduce)
                scale = max(chk.score_scale(ev.K[b, l, h], q, d).max() for q in qs) * np.ones(N)
                chk.check_scores(s[b, l, h], ref, scale)
                chk.check_event(ev.K[b, l, h], ev.V[b, l, h], ev.pos[b, l, h], qs[0], int(ev.p_ref[b]), 30, 0.5,
                                None, sel.pick_order[b, l, h].cpu().numpy(), sel.idx_sorted[b, l, h].cpu().numpy(),
                                Kn[b, l, h], Vn[b, l, h], pn[b, l, h], ref_scores=ref)
                assert np.max(np.abs(sel.scores[b, l, h].cpu().numpy() - ref)) < 1e-5 * scale.max()



def test_report_worst_score_error():
    """Printed for the record (run last in this file): the worst score error of everything checked so far."""
    print("worst |err|/|s| where |s| >= 0.1 scale: %.3e; worst |err|/scale: %.3e; scores checked: %d"
          % (chk.WORST["rel_to_score"], chk.WORST["rel_to_scale"], chk.WORST["n"]))
    assert chk.WORST["rel_to_score"] <= chk.SCORE_RTOL
