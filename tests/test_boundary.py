"""The C-ABI library builds, loads and exports every symbol include/alphakv.h declares (no GPU needed),
and the host-side validation returns error codes without launching anything."""
import ctypes as C
import os
import re

import pytest

import __graft_entry__ as entry
from paper_2605_14292_b200 import api

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    entry.build()
    return api.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "alphakv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(?:akv_status_t|void|uint64_t|const char\*)\s+(\w+)\s*\(", text)
    return sorted(set(names))


def test_header_symbols_are_exported(lib):
    syms = declared_symbols()
    assert {"alpha_score", "alpha_select", "kv_compact", "alpha_compress_event", "alpha_signature_flat",
            "alpha_signature_layer", "akv_create", "akv_destroy", "akv_last_error", "akv_workspace_bytes"} <= set(syms)
    for s in syms:
        assert hasattr(lib, s), f"{s} declared in alphakv.h but not exported"
    assert set(api.EXPORTS) <= set(syms)


def test_default_options(lib):
    o = api._Options()
    lib.akv_default_options(C.byref(o))
    assert abs(o.lam - 0.5) < 1e-7 and o.future_window == 1 and abs(o.rope_base - 10000.0) < 1e-3
    assert o.sig_mode == api.SIG_PER_HEAD and o.flags == 0


def test_null_handle_and_bad_arguments_return_codes(lib):
    lay = api.Layout(1, 1, 1, 16, 128, api.AKV_BF16, (2048, 2048, 2048, 128)).c()
    opt = api.Options().c()
    # null handle is rejected before anything else
    launches = lib.akv_launch_count()
    rc = lib.alpha_score(None, C.byref(lay), None, None, 0, 0, 0, None, None, None, C.byref(opt), None, None, None)
    assert rc == 1 and b"handle" in lib.akv_last_error(None)
    rc = lib.kv_compact(None, C.byref(lay), None, None, None, 0, 0, 0, None, 4, None)
    assert rc == 1
    assert lib.akv_status_string(3) == b"budget out of range"
    assert lib.akv_launch_count() == launches           # a refused call launches nothing


def test_workspace_query_validates_before_it_touches_the_device(lib):
    lay = api.Layout(1, 1, 1, 16, 128, api.AKV_BF16, (2048, 2048, 2048, 128)).c()
    opt = api.Options().c()
    out = C.c_size_t(77)
    assert lib.akv_workspace_bytes(C.byref(lay), 4, C.byref(opt), None) == 1
    assert lib.akv_workspace_bytes(C.byref(lay), 17, C.byref(opt), C.byref(out)) == 3 and out.value == 0
    assert b"budget" in lib.akv_last_error(None)
    assert lib.akv_workspace_bytes(None, 4, C.byref(opt), C.byref(out)) == 1
