"""alpha_compress_event_static: the entry point for callers that may not allocate device memory (a serving
process whose pool owns the whole device, a decode thread that cannot take cudaMalloc's synchronisation).
It keeps the intermediate scores in an array inside the library image. Checked here, through the C ABI,
against alpha_compress_event on the same inputs and against the CPU oracle, twice in a row (the array is
shared between calls and keeps the earlier call's contents), for its size limit, and for the claim itself:
the device's free memory does not move across a call that needs the whole array. Collected last on purpose."""
import numpy as np
import pytest
import torch

import __graft_entry__ as entry
import paper_2605_14292_b200 as akv
from oracle import alpha_oracle as O
from paper_2605_14292_b200 import synth

import akv_check as chk

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    entry.build()
    akv.load_library()


def _run(fn, ev, lam, **kw):
    dev = "cuda"
    K, V, pos = akv.to_device(ev.K, dev), akv.to_device(ev.V, dev), akv.to_device(ev.pos, dev)
    q, pref = akv.to_device(ev.qstat, dev), akv.to_device(ev.p_ref, dev)
    sel = fn(K, V, pos, q, ev.budget, akv.Options(lam=lam), p_ref=pref, **kw)
    torch.cuda.synchronize()
    return dict(K=akv.to_host_bits(K), V=akv.to_host_bits(V), pos=pos.cpu().numpy(), idx=sel.idx_sorted.cpu().numpy(),
                order=sel.pick_order.cpu().numpy(), gain=sel.pick_gain.cpu().numpy(), n_kept=sel.n_kept.cpu().numpy(),
                status=sel.status.cpu().numpy())


def test_static_scratch_entry_matches_the_allocating_one_twice_in_a_row():
    # two different events that do not fit on chip (fp32, N = 600 and 500): both entry points take the
    # score -> select -> compact route, so results are compared bit for bit; the second call finds the first
    # call's scores still in the shared array
    cases = [synth.make_plain(1, 2, 2, 600, 128, 50, 0.5, dtype=synth.F32, seed=31),
             synth.make_plain(2, 1, 3, 500, 128, 70, 0.5, dtype=synth.F32, seed=32)]
    for ev in cases:
        ref = _run(akv.alpha_compress_event, ev, 0.5)
        got = _run(akv.alpha_compress_event_static, ev, 0.5)
        b = ev.budget
        for k in ("idx", "order", "gain", "n_kept", "status"):
            assert np.array_equal(ref[k], got[k]), k
        assert np.array_equal(ref["K"][..., :b, :], got["K"][..., :b, :])
        assert np.array_equal(ref["V"][..., :b, :], got["V"][..., :b, :])
        assert np.array_equal(ref["pos"][..., :b], got["pos"][..., :b])
        assert int(got["n_kept"].min()) == b and int(np.abs(got["status"]).max()) == 0
        # and against the oracle: pick sequence, sorted indices and the compacted rows of every event
        B, L, H, N, d = ev.shape
        for bb in range(B):
            for l in range(L):
                for h in range(H):
                    chk.check_event(ev.K[bb, l, h], ev.V[bb, l, h], ev.pos[bb, l, h], ev.qstat[l, h], int(ev.p_ref[bb]),
                                    b, 0.5, None, got["order"][bb, l, h], got["idx"][bb, l, h], got["K"][bb, l, h],
                                    got["V"][bb, l, h], got["pos"][bb, l, h])


def test_static_scratch_entry_leaves_free_device_memory_unchanged():
    """A call whose scores fill the whole static array (the allocating entry point would need 4 MiB of scratch
    for it) with outputs allocated beforehand: free device memory is the same before and after."""
    small = synth.make_plain(1, 1, 2, 400, 8, 16, 0.5, dtype=synth.F32, seed=33)
    _run(akv.alpha_compress_event_static, small, 0.5)                      # kernels loaded, symbol address resolved
    ev = synth.make_plain(8, 4, 4, 8192, 8, 16, 0.5, dtype=synth.F32, seed=34)   # 8*4*4*8192 = 2^20 scores
    assert ev.n_events * ev.shape[3] == akv.api.STATIC_SCORES_MAX
    K, V, pos = akv.to_device(ev.K, "cuda"), akv.to_device(ev.V, "cuda"), akv.to_device(ev.pos, "cuda")
    q, pref = akv.to_device(ev.qstat, "cuda"), akv.to_device(ev.p_ref, "cuda")
    out = akv.api._alloc_sel(akv.Layout.dense(K), ev.budget, K.device, detail=True)
    opts = akv.Options(lam=0.5)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    akv.alpha_compress_event_static(K, V, pos, q, ev.budget, opts, p_ref=pref, out=out)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    assert int(out.n_kept.min()) == ev.budget and int(out.status.abs().max()) == 0
    idx, order = out.idx_sorted.cpu().numpy(), out.pick_order.cpu().numpy()
    Kn, Vn, pn = akv.to_host_bits(K), akv.to_host_bits(V), pos.cpu().numpy()
    for e in (0, 37, 127):
        bb, l, h = e // 16, (e // 4) % 4, e % 4
        chk.check_event(ev.K[bb, l, h], ev.V[bb, l, h], ev.pos[bb, l, h], ev.qstat[l, h], int(ev.p_ref[bb]), ev.budget, 0.5,
                        None, order[bb, l, h], idx[bb, l, h], Kn[bb, l, h], Vn[bb, l, h], pn[bb, l, h])


def test_static_scratch_entry_rejects_sizes_beyond_its_array():
    N = 4096
    B = akv.api.STATIC_SCORES_MAX // N + 1                     # B*L*H*N just above the limit
    K = torch.zeros((B, 1, 1, N, 8), dtype=torch.bfloat16, device="cuda")
    V = torch.zeros_like(K)
    q = torch.zeros((1, 1, 8), dtype=torch.float32, device="cuda")
    before = akv.launch_count()
    with pytest.raises(akv.AkvError) as e:
        akv.alpha_compress_event_static(K, V, None, q, 16)
    assert e.value.code == 5 and "static scratch" in str(e.value)
    assert akv.launch_count() == before
