"""Builds the CUDA library in-tree: csrc/alphakv.cu -> paper_2605_14292_b200/libalphakv.so (sm_100a)."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG, "csrc")
SO = os.path.join(PKG, "libalphakv.so")

SO_PHASE = os.path.join(PKG, "libalphakv_phase.so")   # profiling build with per-phase cycle stamps

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC", "-shared",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def stale() -> bool:
    if not os.path.exists(SO):
        return True
    t = os.path.getmtime(SO)
    deps = glob.glob(os.path.join(CSRC, "*")) + [os.path.join(os.path.dirname(PKG), "include", "alphakv.h")]
    return any(os.path.getmtime(p) > t for p in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not stale():
        return SO
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", SO] + sources()
    subprocess.check_call(cmd)
    return SO


def build_phase_clocks() -> str:
    """The same sources with -DAKV_PHASE_CLOCKS: kernels stamp clock64() at their phase boundaries into a
    buffer registered through akv_debug_phase_buffer(). Only profiling scripts load this file."""
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    subprocess.check_call([nvcc] + NVCC_FLAGS + ["-DAKV_PHASE_CLOCKS", "-o", SO_PHASE] + sources())
    return SO_PHASE


if __name__ == "__main__":
    if "--phase-clocks" in sys.argv:
        print(build_phase_clocks())
    else:
        print(build(force=True, verbose="-v" in sys.argv))
