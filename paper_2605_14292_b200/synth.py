"""Seeded synthetic inputs for the KV-cache compression event.

This module only *draws numbers and lays them out*: it holds none of the
method's arithmetic (no score, no signature, no selection). Both the CPU oracle
tests and the CUDA path take their inputs from here so that they see the very
same bits. Everything is NumPy on the host; bf16 tensors are carried as uint16
bit patterns (round-to-nearest-even from fp32, done once, here).

The shapes follow the paper's evaluated models and budgets (Section 2
"Workload", Section 4.2: DeepSeek-R1-Distill Qwen-7B / Llama-8B at budgets
b in {64, 128}); the values are N(0,1)-style stand-ins for real K/V, because
neither the model weights nor the evaluation set are available.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

F32 = 0
BF16 = 1


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even); returns the uint16 patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class EventBatch:
    """One call's worth of inputs, dense layout [B, L, H, N, d].

    K, V: fp32 arrays, or uint16 arrays holding bf16 bits (see ``dtype``).
    pos:  int32 [B, L, H, N] RoPE position of every slot (per head, because the
          fused call rewrites it in place).
    qstat: fp32 [L, H, d] per-KV-head query statistic.
    p_ref: int32 [B] reference (next query) position.
    """

    name: str
    dtype: int
    K: np.ndarray
    V: np.ndarray
    pos: np.ndarray
    qstat: np.ndarray
    p_ref: np.ndarray
    budget: int
    lam: float
    rope_base: float = 10000.0
    future_window: int = 1
    eps: float = 1e-8
    meta: dict = field(default_factory=dict)

    @property
    def shape(self):
        return self.K.shape

    @property
    def n_events(self) -> int:
        B, L, H, _, _ = self.K.shape
        return B * L * H


def _normal(rng, shape):
    return rng.standard_normal(size=shape, dtype=np.float32)


def _finish(name, dtype, K, V, qstat, budget, lam, positions=None, p_ref=None, **meta):
    B, L, H, N, d = K.shape
    if positions is None:
        positions = np.arange(N, dtype=np.int32)
    pos = np.broadcast_to(np.asarray(positions, dtype=np.int32), (B, L, H, N)).copy()
    if p_ref is None:
        p_ref = np.full((B,), int(pos.max()) + 1, dtype=np.int32)
    if dtype == BF16:
        K = f32_to_bf16_bits(K)
        V = f32_to_bf16_bits(V)
    return EventBatch(name=name, dtype=dtype, K=K, V=V, pos=pos,
                      qstat=np.ascontiguousarray(qstat, dtype=np.float32),
                      p_ref=np.asarray(p_ref, dtype=np.int32), budget=budget, lam=lam, meta=meta)


def make_plain(B, L, H, N, d, budget, lam, dtype=BF16, seed=0, name="plain") -> EventBatch:
    """K, V, q ~ N(0,1); positions 0..N-1; p_ref = N."""
    rng = np.random.default_rng(seed)
    K = _normal(rng, (B, L, H, N, d))
    V = _normal(rng, (B, L, H, N, d))
    q = _normal(rng, (L, H, d))
    return _finish(name, dtype, K, V, q, budget, lam)


def make_c1(seed=0) -> EventBatch:
    """configs[0]: a single (layer, KV head), fp32, N=192 -> b=64, lambda=0.5."""
    return make_plain(1, 1, 1, 192, 128, 64, 0.5, dtype=F32, seed=seed, name="C1-single-fp32")


def make_c2(seed=0, B=1, L=28, H=4) -> EventBatch:
    """configs[1]: Qwen-7B-shaped, bf16, per-channel scale U(0.5,2) drawn per
    (layer, head) separately for K and V, N=256 -> b=128."""
    N, d = 256, 128
    rng = np.random.default_rng(seed)
    K = _normal(rng, (B, L, H, N, d))
    V = _normal(rng, (B, L, H, N, d))
    cK = rng.uniform(0.5, 2.0, size=(1, L, H, 1, d)).astype(np.float32)
    cV = rng.uniform(0.5, 2.0, size=(1, L, H, 1, d)).astype(np.float32)
    K *= cK
    V *= cV
    q = _normal(rng, (L, H, d))
    return _finish("C2-qwen7b-shaped", BF16, K, V, q, 128, 0.5)


def make_c3(seed=0, B=16, L=32, H=8, N=192, budget=64, dup_frac=0.05, noise=0.01) -> EventBatch:
    """configs[2]: Llama-8B-shaped, bf16, batch 16, N=192 -> b=64. In every event
    round(dup_frac*N) V rows are overwritten by another row's V plus N(0, noise^2)
    before bf16 rounding (K untouched), which makes the redundancy penalty bite."""
    d = 128
    rng = np.random.default_rng(seed)
    K = _normal(rng, (B, L, H, N, d))
    V = _normal(rng, (B, L, H, N, d))
    q = _normal(rng, (L, H, d))
    n_dup = int(round(dup_frac * N))
    E = B * L * H
    Vf = V.reshape(E, N, d)
    # per event: a random permutation's first 2*n_dup entries give disjoint (dst, src) pairs
    perm = np.argsort(rng.random((E, N)), axis=1)[:, : 2 * n_dup]
    dst, src = perm[:, :n_dup], perm[:, n_dup:]
    ev = np.arange(E)[:, None]
    Vf[ev, dst] = Vf[ev, src] + noise * _normal(rng, (E, n_dup, d))
    return _finish("C3-llama8b-shaped", BF16, K, V, q, budget, 0.5, n_dup=n_dup)


def make_c4(seed=0, B=8, L=28, H=4, N=4096, lam=0.5) -> EventBatch:
    """configs[3]: large candidate pool (prefill compression), Qwen-7B shape,
    N=4096 -> b=128, lambda in {0, 0.5, 1.0} chosen by the caller."""
    return make_plain(B, L, H, N, 128, 128, lam, dtype=BF16, seed=seed, name="C4-large-pool")


@dataclass
class PagedCadence:
    """configs[4]: decode-cadence stress in a fixed-size paged KV buffer.

    pool_K / pool_V: uint16 (bf16 bits) [L, n_pages, H, page, d].
    block_table: int32 [B, pages_per_seq]; slot n of sequence b lives in page
    block_table[b, n // page] at offset n % page (same page ids in every layer).
    pos: int32 [B, L, H, N] with N = pages_per_seq * page.
    refill_K / refill_V: uint16 [R, L, H, n_new, d] blocks appended cyclically
    after each event into slots budget..N-1 (new positions continue upward).
    """

    name: str
    pool_K: np.ndarray
    pool_V: np.ndarray
    block_table: np.ndarray
    pos: np.ndarray
    qstat: np.ndarray
    refill_K: np.ndarray
    refill_V: np.ndarray
    B: int
    L: int
    H: int
    N: int
    d: int
    page: int
    budget: int
    lam: float
    rounds: int
    rope_base: float = 10000.0
    future_window: int = 1
    eps: float = 1e-8
    dtype: int = BF16


def make_c5(seed=0, B=64, L=32, H=8, page=64, pages_per_seq=4, d=128, budget=128,
            rounds=32, n_refill_blocks=2, lam=0.5) -> PagedCadence:
    N = page * pages_per_seq
    n_pages = B * pages_per_seq
    rng = np.random.default_rng(seed)
    # pages of a sequence are scattered over the pool (a fixed permutation)
    table = rng.permutation(n_pages).astype(np.int32).reshape(B, pages_per_seq)
    shape = (L, n_pages, H, page, d)
    pool_K = f32_to_bf16_bits(_normal(rng, shape))
    pool_V = f32_to_bf16_bits(_normal(rng, shape))
    pos = np.broadcast_to(np.arange(N, dtype=np.int32), (B, L, H, N)).copy()
    q = _normal(rng, (L, H, d))
    n_new = N - budget
    rK = f32_to_bf16_bits(_normal(rng, (n_refill_blocks, L, H, n_new, d)))
    rV = f32_to_bf16_bits(_normal(rng, (n_refill_blocks, L, H, n_new, d)))
    return PagedCadence(name="C5-decode-cadence", pool_K=pool_K, pool_V=pool_V, block_table=table,
                        pos=pos, qstat=q, refill_K=rK, refill_V=rV, B=B, L=L, H=H, N=N, d=d,
                        page=page, budget=budget, lam=lam, rounds=rounds)


def paged_gather_dense(pool: np.ndarray, table: np.ndarray) -> np.ndarray:
    """View a paged pool [L, n_pages, H, page, d] as dense [B, L, H, N, d] (a copy).
    Pure indexing; used by tests to hand the same bits to the oracle."""
    L, _, H, page, d = pool.shape
    B, pps = table.shape
    g = pool[:, table.reshape(-1)]                      # [L, B*pps, H, page, d]
    g = g.reshape(L, B, pps, H, page, d).transpose(1, 0, 3, 2, 4, 5)
    return np.ascontiguousarray(g).reshape(B, L, H, pps * page, d)


def make_duplicate_pairs(P, d, delta, seed=0, dtype=F32):
    """P pairs of identical V rows, orthogonal across pairs (requires P <= d).

    Returns (scores[2P], V[2P, d], leaders[P]): row 2p is the pair's leader with
    score s_p (strictly decreasing in p), row 2p+1 the follower with s_p - delta.
    The scores are *given*, not computed: this feeds selection-only tests."""
    assert P <= d
    rng = np.random.default_rng(seed)
    s_lead = np.sort(rng.uniform(1.0, 2.0, size=P))[::-1]
    scores = np.empty(2 * P, dtype=np.float64)
    scores[0::2] = s_lead
    scores[1::2] = s_lead - delta
    V = np.zeros((2 * P, d), dtype=np.float32)
    scale = rng.uniform(0.5, 2.0, size=P).astype(np.float32)
    for p in range(P):
        V[2 * p, p] = scale[p]
        V[2 * p + 1, p] = scale[p]
    if dtype == BF16:
        V = f32_to_bf16_bits(V)
    return scores, V, np.arange(0, 2 * P, 2)
