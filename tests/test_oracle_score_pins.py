"""Pins for the oracle's score (reading of the TriAttention 1d scorer, Section 4.1).

The formula is a reading, so it is pinned to things that do not depend on the
oracle's own complex-number form: explicit real rotation matrices (textbook
RoPE), the plain dot product special case, the d = 2 closed form, and the
invariances the construction must have.
"""
import math

import numpy as np
import pytest

from oracle import alpha_oracle as O
from oracle import c_oracle as CO
from paper_2605_14292_b200 import synth


def rope_matrix(p, d, base):
    """Textbook RoPE as a real d x d matrix: coordinates (f, f + d/2) turn by p * base^(-2f/d)."""
    h = d // 2
    R = np.zeros((d, d))
    for f in range(h):
        ang = p * base ** (-2.0 * f / d)
        c, s = math.cos(ang), math.sin(ang)
        R[f, f], R[f, f + h] = c, -s
        R[f + h, f], R[f + h, f + h] = s, c
    return R


def brute_score(K, pos, q, p_ref, W, base):
    n, d = K.shape
    out = np.zeros(n)
    for i in range(n):
        kr = rope_matrix(int(pos[i]), d, base) @ K[i]
        acc = 0.0
        for w in range(W):
            qr = rope_matrix(int(p_ref) + w, d, base) @ q
            acc += float(qr @ kr)
        out[i] = acc / W / math.sqrt(d)
    return out


@pytest.mark.parametrize("d,W,base", [(8, 1, 10000.0), (16, 3, 10000.0), (32, 5, 500.0), (4, 2, 7.0)])
def test_score_equals_rotation_matrix_bruteforce(d, W, base):
    rng = np.random.default_rng(d * 100 + W)
    n = 13
    K = rng.standard_normal((n, d)).astype(np.float32)
    q = rng.standard_normal(d).astype(np.float32)
    pos = rng.integers(0, 300, size=n).astype(np.int32)
    p_ref = 311
    want = brute_score(K.astype(np.float64), pos, q.astype(np.float64), p_ref, W, base)
    got = O.triattention_score(K, pos, q, p_ref, W, base)
    gotc = CO.score(K, pos, q, p_ref, W, base)
    assert np.max(np.abs(got - want)) < 1e-12
    assert np.max(np.abs(gotc - want)) < 1e-12


def test_score_hf_rotate_half_form():
    """Same thing in the q*cos + rotate_half(q)*sin form used by model code."""
    rng = np.random.default_rng(5)
    n, d, base = 9, 16, 10000.0
    K = rng.standard_normal((n, d))
    q = rng.standard_normal(d)
    pos = np.arange(n) * 7
    p_ref = 100
    inv = base ** (-np.arange(0, d, 2) / d)

    def rot(x, p):
        ang = np.concatenate([p * inv, p * inv])
        half = np.concatenate([-x[d // 2:], x[: d // 2]])
        return x * np.cos(ang) + half * np.sin(ang)

    want = np.array([rot(q, p_ref) @ rot(K[i], pos[i]) for i in range(n)]) / math.sqrt(d)
    got = O.triattention_score(K, pos, q, p_ref, 1, base)
    assert np.max(np.abs(got - want)) < 1e-12


def test_score_zero_distance_is_plain_dot():
    rng = np.random.default_rng(1)
    n, d = 20, 32
    K = rng.standard_normal((n, d)).astype(np.float32)
    q = rng.standard_normal(d).astype(np.float32)
    pos = np.full(n, 77, dtype=np.int32)
    want = K.astype(np.float64) @ q.astype(np.float64) / math.sqrt(d)
    for f in (O.triattention_score, CO.score):
        assert np.max(np.abs(f(K, pos, q, 77, 1, 10000.0) - want)) < 1e-13
        assert np.max(np.abs(f(K, None, q, None) - want)) < 1e-13


def test_score_shift_invariance_and_linearity():
    rng = np.random.default_rng(2)
    n, d = 17, 16
    K = rng.standard_normal((n, d)).astype(np.float32)
    K2 = rng.standard_normal((n, d)).astype(np.float32)
    q = rng.standard_normal(d).astype(np.float32)
    q2 = rng.standard_normal(d).astype(np.float32)
    pos = rng.integers(0, 1000, n).astype(np.int32)
    s = O.triattention_score(K, pos, q, 1000, 4)
    s_shift = O.triattention_score(K, pos + 12345, q, 1000 + 12345, 4)
    assert np.max(np.abs(s - s_shift)) < 1e-9
    sa = O.triattention_score(K.astype(np.float64) * 2.0 + K2, pos, q, 1000, 4)
    sb = 2.0 * s + O.triattention_score(K2, pos, q, 1000, 4)
    assert np.max(np.abs(sa - sb)) < 1e-12
    qa = O.triattention_score(K, pos, q.astype(np.float64) * 3.0 - q2, 1000, 4)
    qb = 3.0 * s - O.triattention_score(K, pos, q2, 1000, 4)
    assert np.max(np.abs(qa - qb)) < 1e-12


def test_score_d2_closed_form():
    """d = 2, W = 1: s = |q||k| cos((p_ref - p) * theta_0 + phi_q - phi_k) / sqrt 2, theta_0 = 1."""
    rng = np.random.default_rng(3)
    n = 11
    K = rng.standard_normal((n, 2))
    q = rng.standard_normal(2)
    pos = rng.integers(0, 50, n)
    p_ref = 60
    phi_q = math.atan2(q[1], q[0])
    want = np.array([
        np.hypot(*q) * np.hypot(*K[i]) * math.cos((p_ref - pos[i]) * 1.0 + phi_q - math.atan2(K[i, 1], K[i, 0]))
        for i in range(n)]) / math.sqrt(2)
    got = O.triattention_score(K, pos, q, p_ref, 1, 10000.0)
    assert np.max(np.abs(got - want)) < 1e-12


def test_score_window_is_mean_of_single_positions():
    rng = np.random.default_rng(4)
    n, d, W = 10, 8, 6
    K = rng.standard_normal((n, d))
    q = rng.standard_normal(d)
    pos = np.arange(n)
    each = [O.triattention_score(K, pos, q, 40 + w, 1) for w in range(W)]
    assert np.max(np.abs(O.triattention_score(K, pos, q, 40, W) - np.mean(each, axis=0))) < 1e-12


def test_score_c_matches_numpy_on_bf16_bits():
    ev = synth.make_plain(1, 2, 2, 50, 128, 10, 0.5, dtype=synth.BF16, seed=11)
    for l in range(2):
        for h in range(2):
            a = O.triattention_score(ev.K[0, l, h], ev.pos[0, l, h], ev.qstat[l, h], ev.p_ref[0], 3)
            b = CO.score(ev.K[0, l, h], ev.pos[0, l, h], ev.qstat[l, h], ev.p_ref[0], 3)
            assert np.max(np.abs(a - b)) < 1e-12


def test_bf16_round_trip_and_rounding():
    x = np.array([1.0, 1.00390625, 1.005859375, -2.5, 3.1415927, 0.0, 1e-30], dtype=np.float32)
    bits = synth.f32_to_bf16_bits(x)
    back = synth.bf16_bits_to_f32(bits)
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7: round to even -> 1.0
    assert back[0] == 1.0 and back[1] == 1.0
    # 1 + 2^-8 + 2^-9 rounds up to 1 + 2^-7
    assert back[2] == np.float32(1.0078125)
    assert back[3] == np.float32(-2.5)
    assert abs(back[4] - 3.140625) < 1e-7
    assert np.array_equal(O.widen(bits), back.astype(np.float64))


def test_group_score_reduces_to_the_plain_score_and_to_linearity():
    """Grouped queries: one member is the plain score; the mean over members is the score of the mean statistic
    (the score is linear in it); the maximum is reached by a member at every key and does not depend on the
    members' order."""
    rng = np.random.default_rng(20)
    n, d, G = 23, 16, 4
    K = rng.standard_normal((n, d)).astype(np.float32)
    Q = rng.standard_normal((G, d)).astype(np.float32)
    pos = np.sort(rng.choice(500, size=n, replace=False))
    one = O.triattention_score_group(K, pos, Q[:1], 600, 2)
    assert np.array_equal(one, O.triattention_score(K, pos, Q[0], 600, 2))
    mean = O.triattention_score_group(K, pos, Q, 600, 2, reduce="mean")
    assert np.max(np.abs(mean - O.triattention_score(K, pos, Q.astype(np.float64).mean(axis=0), 600, 2))) < 1e-12
    mx = O.triattention_score_group(K, pos, Q, 600, 2, reduce="max")
    each = np.stack([O.triattention_score(K, pos, q, 600, 2) for q in Q])
    assert np.all(mx >= each - 0) and np.all(np.isin(mx, each))
    assert np.array_equal(mx, O.triattention_score_group(K, pos, Q[::-1], 600, 2, reduce="max"))
    assert np.all(mx >= mean - 1e-12)
