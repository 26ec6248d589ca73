"""Thin Python binding of the alphakv C ABI (include/alphakv.h).

Argument marshalling only: every step of the compression event (score, greedy
selection of Section 4.1 / Algorithm 1, ordering, compaction) runs in the CUDA
kernels behind the C entry points of the same names. PyTorch supplies device
memory and streams. There is no CPU fallback: if the compiled library is missing
the import fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_PKG, "libalphakv.so")

AKV_F32, AKV_BF16 = 0, 1
SIG_PER_HEAD, SIG_FLAT, SIG_PER_LAYER = 0, 1, 2
FLAG_FORCE_GREEDY = 1
FLAG_NO_PRUNE = 2
FLAG_TEST_STARVE_WAIT = 4
FLAG_NO_CHAIN = 8
GQA_MEAN, GQA_MAX = 0, 1

EXPORTS = ("akv_default_options", "akv_create", "akv_destroy", "akv_last_error", "akv_status_string",
           "akv_launch_count", "akv_workspace_bytes", "alpha_score", "alpha_select", "alpha_signature_flat",
           "alpha_signature_layer", "alpha_gram_shared", "kv_compact", "alpha_compress_event",
           "alpha_compress_event_static")


class AkvError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"alphakv error {code}: {msg}")
        self.code = code


class _Layout(C.Structure):
    _fields_ = [("B", C.c_int32), ("L", C.c_int32), ("H", C.c_int32), ("N", C.c_int32), ("d", C.c_int32),
                ("dtype", C.c_int), ("stride_b", C.c_int64), ("stride_l", C.c_int64), ("stride_h", C.c_int64),
                ("stride_n", C.c_int64), ("page_size", C.c_int32), ("block_table", C.c_void_p),
                ("pages_per_seq", C.c_int32), ("stride_page", C.c_int64), ("stride_page_h", C.c_int64),
                ("stride_page_n", C.c_int64)]


class _Options(C.Structure):
    _fields_ = [("lam", C.c_float), ("eps", C.c_float), ("rope_base", C.c_float), ("future_window", C.c_int32),
                ("sig_mode", C.c_int), ("flags", C.c_uint32), ("head_budgets", C.c_void_p), ("shared_gram", C.c_void_p), ("gqa_group", C.c_int32), ("gqa_reduce", C.c_int32)]


_lib = None


def load_library(path: Optional[str] = None):
    """dlopen the compiled library; raises if it has not been built (python -m paper_2605_14292_b200.build)."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or _SO
    if not os.path.exists(p):
        raise ImportError(f"{p} is missing: build it with `python {os.path.join(_PKG, 'build.py')}` "
                          "(there is no CPU fallback)")
    lib = C.CDLL(p)
    lib.akv_last_error.restype = C.c_char_p
    lib.akv_last_error.argtypes = [C.c_void_p]
    lib.akv_status_string.restype = C.c_char_p
    lib.akv_launch_count.restype = C.c_uint64
    lib.akv_create.argtypes = [C.POINTER(C.c_void_p), C.c_int]
    lib.akv_destroy.argtypes = [C.c_void_p]
    vp, i64, i32 = C.c_void_p, C.c_int64, C.c_int32
    lib.alpha_score.argtypes = [vp, C.POINTER(_Layout), vp, vp, i64, i64, i64, vp, vp, vp, C.POINTER(_Options), vp, vp, vp]
    lib.alpha_select.argtypes = [vp, C.POINTER(_Layout), vp, vp, vp, vp, i32, C.POINTER(_Options), vp, vp, vp, vp, vp, vp]
    lib.alpha_signature_flat.argtypes = [vp, C.POINTER(_Layout), vp, vp, C.POINTER(_Options), vp, vp]
    lib.alpha_signature_layer.argtypes = [vp, C.POINTER(_Layout), vp, vp, C.POINTER(_Options), vp, vp]
    lib.alpha_gram_shared.argtypes = [vp, C.POINTER(_Layout), vp, vp, C.POINTER(_Options), vp, vp, vp]
    lib.akv_workspace_bytes.argtypes = [C.POINTER(_Layout), i32, C.POINTER(_Options), C.POINTER(C.c_size_t)]
    lib.kv_compact.argtypes = [vp, C.POINTER(_Layout), vp, vp, vp, i64, i64, i64, vp, i32, vp]
    lib.alpha_compress_event.argtypes = [vp, C.POINTER(_Layout), vp, vp, vp, i64, i64, i64, vp, vp, vp, vp, i32,
                                         C.POINTER(_Options), vp, vp, vp, vp, vp, vp, vp]
    lib.alpha_compress_event_static.argtypes = [vp, C.POINTER(_Layout), vp, vp, vp, i64, i64, i64, vp, vp, vp, vp, i32,
                                                C.POINTER(_Options), vp, vp, vp, vp, vp, vp]
    if path is None:
        _lib = lib
    return lib


_handles = {}


def _handle(device: torch.device):
    idx = device.index if device.index is not None else torch.cuda.current_device()
    if idx not in _handles:
        h = C.c_void_p()
        _check(load_library().akv_create(C.byref(h), idx))
        _handles[idx] = h
    return _handles[idx]


def _check(code: int):
    if code != 0:
        raise AkvError(code, load_library().akv_last_error(None).decode())


def launch_count() -> int:
    return int(load_library().akv_launch_count())


@dataclass
class Options:
    lam: float = 0.5
    eps: float = 1e-8
    rope_base: float = 10000.0
    future_window: int = 1
    sig_mode: int = SIG_PER_HEAD
    flags: int = 0
    head_budgets: Optional[torch.Tensor] = None   # device int32 [L, H]: per-(layer, head) budgets, or None
    shared_gram: Optional[torch.Tensor] = None    # device fp32 [B, N, N] / [B, L, N, N]: cosine matrix of shared signatures
    gqa_group: int = 1                            # query statistics per KV head: qstat is [L, H * gqa_group, d]
    gqa_reduce: int = 0                           # 0: mean over the group, 1: maximum

    def c(self) -> _Options:
        hb = self.head_budgets
        if hb is not None and (hb.dtype != torch.int32 or not hb.is_cuda or not hb.is_contiguous()):
            raise ValueError("head_budgets must be a contiguous int32 CUDA tensor [L, H]")
        sg = self.shared_gram
        if sg is not None and (sg.dtype != torch.float32 or not sg.is_cuda or not sg.is_contiguous()):
            raise ValueError("shared_gram must be a contiguous float32 CUDA tensor")
        return _Options(self.lam, self.eps, self.rope_base, self.future_window, self.sig_mode, self.flags,
                        None if hb is None else hb.data_ptr(), None if sg is None else sg.data_ptr(), self.gqa_group,
                        self.gqa_reduce)


@dataclass
class Layout:
    """How K and V are addressed: dense [B, L, H, N, d] (strides of the tensor) or paged
    (pool [L, n_pages, H, page, d] plus an int32 block table [B, pages_per_seq])."""
    B: int
    L: int
    H: int
    N: int
    d: int
    dtype: int
    strides: tuple = (0, 0, 0, 0)
    page_size: int = 0
    block_table: Optional[torch.Tensor] = None
    page_strides: tuple = (0, 0, 0)   # (page, head, slot) in elements; layer stride is strides[1]

    @staticmethod
    def dense(x: torch.Tensor) -> "Layout":
        if x.dim() != 5 or x.stride(4) != 1:
            raise ValueError("expected [B, L, H, N, d] with contiguous d")
        B, L, H, N, d = x.shape
        return Layout(B, L, H, N, d, _dtype_code(x), tuple(int(s) for s in x.stride()[:4]))

    @staticmethod
    def paged(pool: torch.Tensor, block_table: torch.Tensor, N: Optional[int] = None) -> "Layout":
        if pool.dim() != 5 or pool.stride(4) != 1:
            raise ValueError("expected pool [L, n_pages, H, page, d] with contiguous d")
        L, _, H, page, d = pool.shape
        B, pps = block_table.shape
        if block_table.dtype != torch.int32 or not block_table.is_contiguous():
            raise ValueError("block_table must be contiguous int32")
        sl, sp, sh, sn, _ = (int(s) for s in pool.stride())
        return Layout(B, L, H, N if N is not None else pps * page, d, _dtype_code(pool), (0, sl, 0, 0), page,
                      block_table, (sp, sh, sn))

    def c(self) -> _Layout:
        y = _Layout()
        y.B, y.L, y.H, y.N, y.d, y.dtype = self.B, self.L, self.H, self.N, self.d, self.dtype
        y.stride_b, y.stride_l, y.stride_h, y.stride_n = self.strides
        y.page_size = self.page_size
        y.block_table = _ptr(self.block_table)
        y.pages_per_seq = 0 if self.block_table is None else int(self.block_table.shape[1])
        y.stride_page, y.stride_page_h, y.stride_page_n = self.page_strides
        return y

    @property
    def n_events(self) -> int:
        return self.B * self.L * self.H


def _dtype_code(x: torch.Tensor) -> int:
    if x.dtype == torch.bfloat16:
        return AKV_BF16
    if x.dtype == torch.float32:
        return AKV_F32
    raise TypeError(f"K/V must be float32 or bfloat16, got {x.dtype}")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _need(t: Optional[torch.Tensor], dtype, name: str, cuda=True):
    if t is None:
        return
    if t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    if cuda and not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")


def _pos_strides(pos: Optional[torch.Tensor], lay: Layout):
    """pos may be [N], [B, N] or [B, L, H, N] (int32, last dim contiguous); returns (b, l, h) strides."""
    if pos is None:
        return 0, 0, 0
    if pos.dtype != torch.int32 or pos.stride(-1) != 1 or pos.shape[-1] < lay.N:
        raise ValueError("pos must be int32 with a contiguous last dimension of at least N slots")
    if pos.dim() == 1:
        return 0, 0, 0
    if pos.dim() == 2:
        return int(pos.stride(0)), 0, 0
    if pos.dim() == 4:
        return int(pos.stride(0)), int(pos.stride(1)), int(pos.stride(2))
    raise ValueError("pos must have 1, 2 or 4 dimensions")


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _lay(x: torch.Tensor, layout: Optional[Layout]) -> Layout:
    return layout if layout is not None else Layout.dense(x)


# --------------------------------------------------------------------------------------------- entry points
def alpha_score(K, qstat, pos=None, p_ref=None, n_cand=None, opts: Optional[Options] = None,
                layout: Optional[Layout] = None, out=None, status=None):
    """Retention scores s [B, L, H, N] (fp32) -- C entry point ``alpha_score``."""
    lay = _lay(K, layout)
    opts = opts or Options()
    _need(qstat, torch.float32, "qstat"); _need(p_ref, torch.int32, "p_ref"); _need(n_cand, torch.int32, "n_cand")
    if out is None:
        out = torch.zeros((lay.B, lay.L, lay.H, lay.N), dtype=torch.float32, device=K.device)
    _need(out, torch.float32, "out"); _need(status, torch.int32, "status")
    sb, sl, sh = _pos_strides(pos, lay)
    with torch.cuda.device(K.device):
        _check(load_library().alpha_score(_handle(K.device), C.byref(lay.c()), _ptr(K), _ptr(pos), sb, sl, sh,
                                          _ptr(n_cand), _ptr(qstat), _ptr(p_ref), C.byref(opts.c()), _ptr(out),
                                          _ptr(status), _stream()))
    return out


@dataclass
class Selection:
    idx_sorted: torch.Tensor
    pick_order: Optional[torch.Tensor] = None
    pick_gain: Optional[torch.Tensor] = None
    n_kept: Optional[torch.Tensor] = None
    status: Optional[torch.Tensor] = None
    scores: Optional[torch.Tensor] = None


def _alloc_sel(lay: Layout, budget: int, device, detail: bool) -> Selection:
    shp = (lay.B, lay.L, lay.H, budget)
    sel = Selection(torch.empty(shp, dtype=torch.int32, device=device))
    if detail:
        sel.pick_order = torch.empty(shp, dtype=torch.int32, device=device)
        sel.pick_gain = torch.empty(shp, dtype=torch.float32, device=device)
        sel.n_kept = torch.empty(shp[:3], dtype=torch.int32, device=device)
        sel.status = torch.empty(shp[:3], dtype=torch.int32, device=device)
    return sel


def alpha_select(scores, V, budget: int, opts: Optional[Options] = None, flat_sig=None, n_cand=None,
                 layout: Optional[Layout] = None, detail: bool = True, out: Optional[Selection] = None) -> Selection:
    """Greedy set-conditioned selection (Algorithm 1) -- C entry point ``alpha_select``."""
    opts = opts or Options()
    if layout is None:
        if V is not None:
            layout = Layout.dense(V)
        else:
            B, L, H, N = scores.shape
            layout = Layout(B, L, H, N, int(flat_sig.shape[-1]), AKV_F32, (L * H * N * 8, H * N * 8, N * 8, 8))
    lay = layout
    _need(scores, torch.float32, "scores"); _need(flat_sig, torch.float32, "flat_sig"); _need(n_cand, torch.int32, "n_cand")
    sel = out or _alloc_sel(lay, budget, scores.device, detail)
    with torch.cuda.device(scores.device):
        _check(load_library().alpha_select(_handle(scores.device), C.byref(lay.c()), _ptr(scores), _ptr(V),
                                           _ptr(flat_sig), _ptr(n_cand), budget, C.byref(opts.c()),
                                           _ptr(sel.idx_sorted), _ptr(sel.pick_order), _ptr(sel.pick_gain),
                                           _ptr(sel.n_kept), _ptr(sel.status), _stream()))
    return sel


def alpha_signature_flat(V, opts: Optional[Options] = None, n_cand=None, layout: Optional[Layout] = None, out=None):
    """Eq. 1 signatures [B, N, d] (fp32) -- C entry point ``alpha_signature_flat``."""
    lay = _lay(V, layout)
    opts = opts or Options()
    if out is None:
        out = torch.zeros((lay.B, lay.N, lay.d), dtype=torch.float32, device=V.device)
    _need(out, torch.float32, "out")
    with torch.cuda.device(V.device):
        _check(load_library().alpha_signature_flat(_handle(V.device), C.byref(lay.c()), _ptr(V), _ptr(n_cand),
                                                   C.byref(opts.c()), _ptr(out), _stream()))
    return out


def alpha_signature_layer(V, opts: Optional[Options] = None, n_cand=None, layout: Optional[Layout] = None, out=None):
    """Per-layer signatures [B, L, N, d] (fp32), Eq. 1 summed over one layer's heads -- C entry point
    ``alpha_signature_layer``."""
    lay = _lay(V, layout)
    opts = opts or Options()
    if out is None:
        out = torch.zeros((lay.B, lay.L, lay.N, lay.d), dtype=torch.float32, device=V.device)
    _need(out, torch.float32, "out")
    with torch.cuda.device(V.device):
        _check(load_library().alpha_signature_layer(_handle(V.device), C.byref(lay.c()), _ptr(V), _ptr(n_cand),
                                                    C.byref(opts.c()), _ptr(out), _stream()))
    return out


def alpha_gram_shared(sig, layout: Layout, opts: Options, n_cand=None, out=None, status=None):
    """Cosine matrix of shared signatures, [B, N, N] (flat) or [B, L, N, N] (per layer), fp32 -- C entry point
    ``alpha_gram_shared``. ``opts.sig_mode`` says which; ``layout`` gives B, L, N, d."""
    _need(sig, torch.float32, "sig"); _need(n_cand, torch.int32, "n_cand"); _need(status, torch.int32, "status")
    lay = layout
    if out is None:
        shape = (lay.B, lay.N, lay.N) if opts.sig_mode == SIG_FLAT else (lay.B, lay.L, lay.N, lay.N)
        out = torch.zeros(shape, dtype=torch.float32, device=sig.device)
    _need(out, torch.float32, "out")
    with torch.cuda.device(sig.device):
        _check(load_library().alpha_gram_shared(_handle(sig.device), C.byref(lay.c()), _ptr(sig), _ptr(n_cand),
                                                C.byref(opts.c()), _ptr(out), _ptr(status), _stream()))
    return out


def workspace_bytes(layout: Layout, budget: int, opts: Optional[Options] = None) -> int:
    """Scratch bytes the fused call would allocate for this shape -- C entry point ``akv_workspace_bytes``."""
    out = C.c_size_t(0)
    _check(load_library().akv_workspace_bytes(C.byref(layout.c()), budget, C.byref((opts or Options()).c()), C.byref(out)))
    return int(out.value)


def kv_compact(K, V, pos, idx_sorted, layout: Optional[Layout] = None):
    """In-place move of the kept rows to slots 0..budget-1 -- C entry point ``kv_compact``."""
    ref = K if K is not None else V
    lay = _lay(ref, layout)
    _need(idx_sorted, torch.int32, "idx_sorted")
    budget = int(idx_sorted.shape[-1])
    sb, sl, sh = _pos_strides(pos, lay)
    with torch.cuda.device(ref.device):
        _check(load_library().kv_compact(_handle(ref.device), C.byref(lay.c()), _ptr(K), _ptr(V), _ptr(pos), sb, sl, sh,
                                         _ptr(idx_sorted), budget, _stream()))


def alpha_compress_event(K, V, pos, qstat, budget: int, opts: Optional[Options] = None, p_ref=None, n_cand=None,
                         flat_sig=None, layout: Optional[Layout] = None, detail: bool = True,
                         want_scores: bool = False, out: Optional[Selection] = None) -> Selection:
    """Score + select + order + compact in one call -- C entry point ``alpha_compress_event``.
    K, V and pos are rewritten in place."""
    lay = _lay(K, layout)
    opts = opts or Options()
    _need(qstat, torch.float32, "qstat"); _need(p_ref, torch.int32, "p_ref"); _need(n_cand, torch.int32, "n_cand")
    _need(flat_sig, torch.float32, "flat_sig")
    sel = out or _alloc_sel(lay, budget, K.device, detail)
    if want_scores and sel.scores is None:
        sel.scores = torch.zeros((lay.B, lay.L, lay.H, lay.N), dtype=torch.float32, device=K.device)
    sb, sl, sh = _pos_strides(pos, lay)
    with torch.cuda.device(K.device):
        _check(load_library().alpha_compress_event(
            _handle(K.device), C.byref(lay.c()), _ptr(K), _ptr(V), _ptr(pos), sb, sl, sh, _ptr(n_cand), _ptr(qstat),
            _ptr(p_ref), _ptr(flat_sig), budget, C.byref(opts.c()), _ptr(sel.idx_sorted), _ptr(sel.pick_order),
            _ptr(sel.pick_gain), _ptr(sel.scores), _ptr(sel.n_kept), _ptr(sel.status), _stream()))
    return sel


STATIC_SCORES_MAX = 1 << 20


def alpha_compress_event_static(K, V, pos, qstat, budget: int, opts: Optional[Options] = None, p_ref=None, n_cand=None,
                                flat_sig=None, layout: Optional[Layout] = None, detail: bool = True,
                                out: Optional[Selection] = None) -> Selection:
    """The compression event for callers that must not allocate device memory -- C entry point
    ``alpha_compress_event_static``. Scores are kept in a 4 MiB array inside the library image instead of
    cudaMalloc'ed scratch, so B*L*H*N may not exceed STATIC_SCORES_MAX; calls on one device share that array
    and must not overlap on the GPU. Pass ``out`` (pre-allocated outputs) to keep torch from allocating too.
    K, V and pos are rewritten in place."""
    lay = _lay(K, layout)
    opts = opts or Options()
    _need(qstat, torch.float32, "qstat"); _need(p_ref, torch.int32, "p_ref"); _need(n_cand, torch.int32, "n_cand")
    _need(flat_sig, torch.float32, "flat_sig")
    sel = out or _alloc_sel(lay, budget, K.device, detail)
    sb, sl, sh = _pos_strides(pos, lay)
    with torch.cuda.device(K.device):
        _check(load_library().alpha_compress_event_static(
            _handle(K.device), C.byref(lay.c()), _ptr(K), _ptr(V), _ptr(pos), sb, sl, sh, _ptr(n_cand), _ptr(qstat),
            _ptr(p_ref), _ptr(flat_sig), budget, C.byref(opts.c()), _ptr(sel.idx_sorted), _ptr(sel.pick_order),
            _ptr(sel.pick_gain), _ptr(sel.n_kept), _ptr(sel.status), _stream()))
    return sel


# --------------------------------------------------------------------------------------------- host <-> torch helpers
def to_device(x, device="cuda"):
    """NumPy array from the input generators -> torch tensor on `device` (uint16 arrays are bf16 bits)."""
    import numpy as np
    if isinstance(x, np.ndarray) and x.dtype == np.uint16:
        return torch.from_numpy(x.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(x).to(device)


def to_host_bits(t: torch.Tensor):
    """Torch tensor -> NumPy; bf16 comes back as uint16 bit patterns."""
    import numpy as np
    if t.dtype == torch.bfloat16:
        return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()
