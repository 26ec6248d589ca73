"""CPU oracle for the KV-cache compression event of the alpha retainer.

TEST INFRASTRUCTURE ONLY. This is the plain, slow, float64 statement of what
the CUDA path must compute. It shares no code with the CUDA path; only tests,
the smoke check and the benchmark's CPU-baseline leg may import it. The product
never routes through it.

What is written from where:
  * selection: Section 4.1 -- Eq. 1 (V-signatures), Eq. 2 (marginal gain of a
    candidate given the chosen set), Eq. 3 (each new member maximises Eq. 2 over
    the candidates not chosen yet; the first member has the largest score) --
    which is what Algorithm 1 computes;
  * top-k baseline and the lambda = 0 case: Section 4.1 and the first branch of
    Algorithm 1;
  * compaction: the chosen rows, in slot order, become the new cache of at most
    `budget` rows (Section 1, Section 4.1);
  * score: the paper names the scorer it inherits but does not print its
    formula. The reading used here (mean RoPE attention logit of the head's
    query statistic against each pre-RoPE key, a trigonometric series in the
    position distance) is pinned only to its own closed forms and to a
    brute-force rotation-matrix evaluation:
    PARITY UNPINNED against the real TriAttention scorer.

All arithmetic is float64 on the exact input bits (bf16 inputs arrive as uint16
bit patterns and are widened exactly).
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

NEG_INF = -np.inf

STATUS_OK = 0
STATUS_NONFINITE = 1
STATUS_SHORT = 2


# --------------------------------------------------------------------------- inputs
def widen(x: np.ndarray) -> np.ndarray:
    """Exact float64 view of an input tensor: fp32 arrays widen directly, uint16
    arrays are bf16 bit patterns (sign, 8 exponent bits, 7 mantissa bits)."""
    x = np.asarray(x)
    if x.dtype == np.uint16:
        return (x.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    return x.astype(np.float64)


# --------------------------------------------------------------------------- score
def rope_frequencies(d: int, base: float) -> np.ndarray:
    """theta_f = base^(-2f/d), f = 0..d/2-1 (standard RoPE frequencies)."""
    f = np.arange(d // 2, dtype=np.float64)
    return np.power(float(base), -2.0 * f / d)


def window_coefficients(theta: np.ndarray, W: int) -> np.ndarray:
    """c_f = (1/W) * sum_{w=0}^{W-1} exp(i w theta_f): the average over the W
    future query positions p_ref .. p_ref+W-1."""
    w = np.arange(W, dtype=np.float64)[:, None]
    return np.exp(1j * w * theta[None, :]).mean(axis=0)


def triattention_score(K, pos, qstat, p_ref, W: int = 1, base: float = 10000.0) -> np.ndarray:
    """Per-token retention score s in R^n for one (sequence, layer, KV head)
    (Section 4.1 takes the scores from the TriAttention scorer it builds on;
    Section 2 describes that scorer as working from precomputed Q/K frequency
    statistics that stand in for the queries still to come).

    Reading: keys are stored pre-RoPE; RoPE pairs coordinate f with f + d/2 and
    turns the pair, seen as the complex number z(x)_f = x_f + i x_{f+d/2}, by
    the angle p * theta_f. The score of key i is the RoPE attention logit of the
    head's mean query placed at the future positions p_ref + w against key i at
    p_i, averaged over w = 0..W-1 and scaled by 1/sqrt(d):

        s_i = (1/sqrt d) Re sum_f c_f z(q)_f conj(z(k_i)_f) exp(i (p_ref - p_i) theta_f)

    ``pos is None`` means the cache is already rotated: s_i = q . k_i / sqrt d.
    """
    K = widen(K)
    q = widen(qstat)
    n, d = K.shape
    if pos is None:
        return K @ q / math.sqrt(d)
    half = d // 2
    theta = rope_frequencies(d, base)
    c = window_coefficients(theta, W)
    zq = q[:half] + 1j * q[half:]
    zk = K[:, :half] + 1j * K[:, half:]
    dist = (int(p_ref) - np.asarray(pos, dtype=np.int64)).astype(np.float64)
    turn = np.exp(1j * dist[:, None] * theta[None, :])
    terms = (c * zq)[None, :] * np.conj(zk) * turn
    return terms.real.sum(axis=1) / math.sqrt(d)


def triattention_score_group(K, pos, qstats, p_ref, W: int = 1, base: float = 10000.0, reduce: str = "mean") -> np.ndarray:
    """Grouped-query attention: the KV head serves several query heads, each with its own statistic
    (qstats: [G, d]). The key's score is the mean of the G per-head scores, or the largest of them
    ("max": a key that any query head of the group wants scores high). Each per-head score is
    triattention_score as it stands."""
    per_head = np.stack([triattention_score(K, pos, q, p_ref, W, base) for q in np.asarray(qstats)])
    if reduce == "mean":
        return per_head.mean(axis=0)
    if reduce == "max":
        return per_head.max(axis=0)
    raise ValueError(reduce)


def default_p_ref(pos) -> int:
    """When the caller gives no reference position: one past the newest slot."""
    return int(np.max(pos)) + 1


# --------------------------------------------------------------------------- signatures
def signatures_per_head(V, eps: float = 1e-8) -> np.ndarray:
    """Per-head signature mode (Section 6 names it as a variant of Eq. 1):
    v_i = V_i / (||V_i||_2 + eps) with the (layer, head) sums of Eq. 1 reduced to
    the single head at hand."""
    V = widen(V)
    nrm = np.sqrt((V * V).sum(axis=1))
    return V / (nrm + eps)[:, None]


def signatures_flat(V_all, eps: float = 1e-8) -> np.ndarray:
    """Eq. 1: u_i = (1/(L H)) sum_l sum_h V_i^(l,h);  v_i = u_i / (||u_i||_2 + eps).
    V_all is [L, H, n, d] for one sequence; slots are aligned across heads."""
    V_all = widen(V_all)
    L, H, n, d = V_all.shape
    u = V_all.sum(axis=(0, 1)) / (L * H)
    nrm = np.sqrt((u * u).sum(axis=1))
    return u / (nrm + eps)[:, None]


def signatures_per_layer(V_layer, eps: float = 1e-8) -> np.ndarray:
    """The per-layer variant Section 6 names: Eq. 1 with the sum restricted to the H KV heads
    of one layer, u_i = (1/H) sum_h V_i^(h);  v_i = u_i / (||u_i||_2 + eps).
    V_layer is [H, n, d] for one (sequence, layer)."""
    V_layer = widen(V_layer)
    H, n, d = V_layer.shape
    u = V_layer.sum(axis=0) / H
    nrm = np.sqrt((u * u).sum(axis=1))
    return u / (nrm + eps)[:, None]


# --------------------------------------------------------------------------- selection
def _argmax_lowest(a: np.ndarray, excluded: Optional[np.ndarray] = None) -> int:
    """argmax over the candidates not in ``excluded``, ties to the lowest index.
    (A candidate whose value is -inf can still be taken when nothing better is
    left, so the result is always a new index.)"""
    if excluded is None:
        return int(np.argmax(a))                      # np.argmax returns the first maximum
    cand = np.nonzero(~excluded)[0]
    return int(cand[np.argmax(a[cand])])


def sanitize_scores(s: np.ndarray):
    """Non-finite scores can never be preferred: they become -inf (flagged)."""
    s = np.array(s, dtype=np.float64, copy=True)
    bad = ~np.isfinite(s)
    s[bad] = NEG_INF
    return s, bool(bad.any())


def topk_indices(s, k: int) -> np.ndarray:
    """Modular top-k (Section 4.1; the lambda = 0 branch of Algorithm 1): the k largest scores,
    ties to the lower index, in pick order (descending score)."""
    s = np.asarray(s, dtype=np.float64)
    order = np.lexsort((np.arange(len(s)), -s))  # primary: -s ascending, then index
    return order[:k].astype(np.int64)


@dataclass
class Selection:
    order: np.ndarray      # pick order i_1 .. i_k
    gains: np.ndarray      # Delta(i_t | S_{t-1}) at the moment of the pick
    margins: np.ndarray    # best minus second-best candidate value at each pick (inf if none)
    idx_sorted: np.ndarray  # sort(S)
    status: int = STATUS_OK


def alpha_select(s, sig, k: int, lam: float, force_greedy: bool = False) -> Selection:
    """Greedy fill of the budget (Section 4.1, Eq. 2 and Eq. 3; Algorithm 1).

    State kept between picks: for every candidate i the redundancy term of Eq. 2 against the
    set chosen so far, red_i = max(0, max_{j in S} cos(v_i, v_j)), which is 0 for the empty
    set. A pick evaluates Eq. 2 for all candidates, gain_i = s_i - lam * red_i, takes the
    best candidate outside S (Eq. 3; the first pick therefore has the largest score) and
    folds the new member's cosines into red. cos(v_i, v_j) = <v_i, v_j> for the unit rows of
    Eq. 1; each one is computed when it is needed, as a plain dot product.
    s: scores [n]; sig: unit-normalised signatures [n, d]."""
    s, bad = sanitize_scores(s)
    sig = np.asarray(sig, dtype=np.float64)
    n = len(s)
    status = STATUS_NONFINITE if bad else STATUS_OK
    if n < k:
        k = n
        status = STATUS_SHORT
    if lam == 0 and not force_greedy:                     # no penalty: plain top-k of the scores
        full = topk_indices(s, n)                         # all indices, best first
        order = full[:k]
        gains = s[order]
        margins = np.full(k, np.inf)
        for t in range(k):
            if t + 1 < n and np.isfinite(s[full[t]]) and np.isfinite(s[full[t + 1]]):
                margins[t] = s[full[t]] - s[full[t + 1]]
            elif not np.isfinite(s[full[t]]):
                margins[t] = 0.0
        return Selection(order, gains, margins, np.sort(order), status)

    red = np.zeros(n)                                     # Eq. 2's max(0, max_j cos) for S = {}
    chosen = np.zeros(n, dtype=bool)
    order, gains, margins = [], [], []
    for _t in range(k):
        gain = s - lam * red                              # Eq. 2 for every candidate
        gain[chosen] = NEG_INF                            # members of S do not compete
        i = _argmax_lowest(gain, chosen)                  # Eq. 3
        others = np.delete(gain, i)
        second = others.max() if len(others) else NEG_INF
        margins.append(gain[i] - second if np.isfinite(gain[i]) and np.isfinite(second) else
                       (np.inf if np.isfinite(gain[i]) else 0.0))
        order.append(i)
        gains.append(gain[i])
        chosen[i] = True
        np.maximum(red, sig @ sig[i], out=red)            # cosines of the new member against everyone
    order = np.array(order, dtype=np.int64)
    return Selection(order, np.array(gains), np.array(margins), np.sort(order), status)


def alpha_select_from_definition(s, sig, k: int, lam: float) -> np.ndarray:
    """The same selection with nothing carried from pick to pick (tiny n only): the cosine
    matrix of all pairs is formed once, and every pick evaluates Eq. 2 for every candidate
    from its definition -- the largest cosine against the members chosen so far, floored at
    zero -- before Eq. 3 takes the best one. Returns the chosen set in ascending order."""
    s, _ = sanitize_scores(s)
    sig = np.asarray(sig, dtype=np.float64)
    n = len(s)
    k = min(k, n)
    if lam == 0:
        return np.sort(topk_indices(s, k))
    cosines = sig @ sig.T
    S: list = []
    for _t in range(k):
        gain = np.array([s[i] - (lam * max(0.0, max(cosines[i, j] for j in S)) if S else 0.0) for i in range(n)])
        member = np.zeros(n, dtype=bool)
        member[S] = True
        gain[member] = NEG_INF
        S.append(_argmax_lowest(gain, member))
    return np.sort(np.array(S, dtype=np.int64))


def marginal_gain(i: int, S: Sequence[int], s, sig, lam: float) -> float:
    """Eq. 2 from the definition, no running state:
    Delta(i | S) = s_i - lam * max(0, max_{j in S} cos(v_i, v_j))."""
    if len(S) == 0:
        return float(s[i])
    cos = max(float(np.dot(sig[i], sig[j])) for j in S)
    return float(s[i]) - lam * max(0.0, cos)


# --------------------------------------------------------------------------- compaction
def compact_rows(X: np.ndarray, idx_sorted: np.ndarray) -> np.ndarray:
    """New cache = rows idx_sorted[r] of the old one at slot r (bit copies, raw dtype)."""
    return np.ascontiguousarray(np.asarray(X)[np.asarray(idx_sorted, dtype=np.int64)])


# --------------------------------------------------------------------------- whole event
@dataclass
class EventResult:
    scores: np.ndarray
    sel: Selection
    K_new: np.ndarray
    V_new: np.ndarray
    pos_new: Optional[np.ndarray]


def compress_event(K, V, pos, qstat, p_ref, k: int, lam: float, W: int = 1, base: float = 10000.0,
                   eps: float = 1e-8, sig: Optional[np.ndarray] = None,
                   force_greedy: bool = False) -> EventResult:
    """One compression event for one (sequence, layer, KV head): score, select
    (per-head signatures unless ``sig`` is supplied, e.g. Eq. 1's flat one),
    order, compact."""
    if p_ref is None and pos is not None:
        p_ref = default_p_ref(pos)
    s = triattention_score(K, pos, qstat, p_ref, W, base)
    if sig is None:
        sig = signatures_per_head(V, eps)
    sel = alpha_select(s, sig, k, lam, force_greedy=force_greedy)
    Kn = compact_rows(K, sel.idx_sorted)
    Vn = compact_rows(V, sel.idx_sorted)
    pn = None if pos is None else compact_rows(np.asarray(pos), sel.idx_sorted)
    return EventResult(s, sel, Kn, Vn, pn)


# --------------------------------------------------------------------------- acceptance helper
@dataclass
class Replay:
    ok: bool
    n_diverged: int           # steps where the candidate's pick is not the oracle's argmax
    worst_deficit: float      # max over steps of (best value - value of candidate's pick)
    log: list                 # (step, candidate pick, oracle pick, deficit)


def replay_pick_order(s, sig, lam: float, picks: Sequence[int], tol: float = 1e-6) -> Replay:
    """Acceptance rule for a pick sequence produced elsewhere: walk the sequence,
    and at each step, with the *same* prefix S_t, evaluate Eq. 2 in float64 for
    every candidate; the pick is accepted if its value is within ``tol`` of the
    best one. Steps where it is not the float64 argmax are logged with the
    deficit (these are the sub-tolerance near-ties where two results are both
    correct)."""
    s, _ = sanitize_scores(s)
    sig = np.asarray(sig, dtype=np.float64)
    n = len(s)
    m = np.zeros(n)
    in_S = np.zeros(n, dtype=bool)
    log, worst, ok = [], 0.0, True
    for t, i in enumerate(picks):
        i = int(i)
        if i < 0 or i >= n or in_S[i]:
            return Replay(False, len(log) + 1, np.inf, log + [(t, i, -1, np.inf)])
        a = s - lam * m if t > 0 else s.copy()
        a[in_S] = NEG_INF
        best = _argmax_lowest(a, in_S)
        if best != i:
            deficit = a[best] - a[i] if np.isfinite(a[i]) else (0.0 if not np.isfinite(a[best]) else np.inf)
            log.append((t, i, best, float(deficit)))
            worst = max(worst, float(deficit))
            if deficit > tol:
                ok = False
        in_S[i] = True
        np.maximum(m, sig @ sig[i], out=m)
    return Replay(ok, len(log), worst, log)
