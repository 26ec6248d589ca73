"""ctypes access to the C oracle (alpha_oracle.c) -- TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg import this.
``build()`` compiles the C file with gcc next to its source; nothing here is
used by, or shared with, the CUDA path.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "alpha_oracle.c")
_SO = os.path.join(_HERE, "liborc.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fPIC", "-shared", "-o", _SO, _SRC, "-lm"])
    return _SO


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_select.restype = C.c_int
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _dtype_code(x: np.ndarray) -> int:
    if x.dtype == np.uint16:
        return 1
    if x.dtype == np.float32:
        return 0
    raise TypeError("K/V must be float32 or uint16 (bf16 bits)")


def score(K, pos, qstat, p_ref, W=1, base=10000.0):
    K = np.ascontiguousarray(K)
    n, d = K.shape
    q = np.ascontiguousarray(qstat, dtype=np.float32)
    s = np.empty(n, dtype=np.float64)
    pp = None if pos is None else np.ascontiguousarray(pos, dtype=np.int32)
    lib().orc_score(_p(K), C.c_int(_dtype_code(K)), C.c_int(n), C.c_int(d), _p(pp), _p(q),
                    C.c_int64(0 if p_ref is None else int(p_ref)), C.c_int(W), C.c_double(base), _p(s))
    return s


def signature(V, eps=1e-8):
    V = np.ascontiguousarray(V)
    n, d = V.shape
    sig = np.empty((n, d), dtype=np.float64)
    lib().orc_signature(_p(V), C.c_int(_dtype_code(V)), C.c_int(n), C.c_int(d), C.c_double(eps), _p(sig))
    return sig


def select(s, sig, k, lam, force_greedy=False):
    s = np.ascontiguousarray(s, dtype=np.float64)
    sig = np.ascontiguousarray(sig, dtype=np.float64)
    n, d = sig.shape
    order = np.full(k, -1, dtype=np.int64)
    gain = np.zeros(k)
    margin = np.zeros(k)
    st = C.c_int(0)
    kk = lib().orc_select(_p(s), _p(sig), C.c_int(n), C.c_int(d), C.c_int(k), C.c_double(lam),
                          C.c_int(int(force_greedy)), _p(order), _p(gain), _p(margin), C.byref(st))
    return order[:kk], gain[:kk], margin[:kk], st.value


def event_batch(K, V, pos, qstat, p_ref, k, lam, W=1, base=10000.0, eps=1e-8, force_greedy=False,
                events=None, threads=1, want_rows=True, want_scores=True, budgets=None):
    """Run whole events over a dense batch [B, L, H, n, d]; returns a dict of
    arrays shaped [B, L, H, ...]. ``events`` = (e0, e1) range in flattened
    (b, l, h) order (default all); outside it outputs are left untouched (zeros). ``budgets``: optional int32
    [L, H] per-(layer, head) budgets (each <= k; k stays the row length of the outputs)."""
    K = np.ascontiguousarray(K)
    V = np.ascontiguousarray(V)
    B, L, H, n, d = K.shape
    E = B * L * H
    e0, e1 = (0, E) if events is None else events
    dt = _dtype_code(K)
    pp = None if pos is None else np.ascontiguousarray(pos, dtype=np.int32).reshape(E, n)
    q = np.ascontiguousarray(qstat, dtype=np.float32)
    pr = None if p_ref is None else np.ascontiguousarray(p_ref, dtype=np.int32)
    bud = None if budgets is None else np.ascontiguousarray(budgets, dtype=np.int32).reshape(L * H)
    out = {
        "scores": np.zeros((B, L, H, n), dtype=np.float64) if want_scores else None,
        "idx_sorted": np.full((B, L, H, k), -1, dtype=np.int32),
        "order": np.full((B, L, H, k), -1, dtype=np.int32),
        "K": np.zeros((B, L, H, k, d), dtype=K.dtype) if want_rows else None,
        "V": np.zeros((B, L, H, k, d), dtype=V.dtype) if want_rows else None,
        "pos": np.zeros((B, L, H, k), dtype=np.int32) if (want_rows and pp is not None) else None,
        "status": np.zeros((B, L, H), dtype=np.int32),
    }

    def run(lo, hi):
        lib().orc_event_batch(_p(K), _p(V), C.c_int(dt), C.c_int(B), C.c_int(L), C.c_int(H), C.c_int(n),
                              C.c_int(d), _p(pp), _p(q), _p(pr), C.c_int(W), C.c_double(base),
                              C.c_double(eps), C.c_int(k), C.c_double(lam), C.c_int(int(force_greedy)),
                              C.c_int(lo), C.c_int(hi), _p(out["scores"]), _p(out["idx_sorted"]),
                              _p(out["order"]), _p(out["K"]), _p(out["V"]), _p(out["pos"]), _p(out["status"]), _p(bud))

    threads = max(1, int(threads))
    if threads == 1 or e1 - e0 < 2:
        run(e0, e1)
    else:
        cuts = np.linspace(e0, e1, min(threads, e1 - e0) + 1).astype(int)
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(lambda ab: run(int(ab[0]), int(ab[1])), zip(cuts[:-1], cuts[1:])))
    return out
