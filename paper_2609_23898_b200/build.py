"""Builds libcerar.so (the C-ABI library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "libcerar.so")
CHECKED_LIB_PATH = os.path.join(PKG_DIR, "libcerar_checked.so")   # the same sources with -DCERAR_BOUNDS_CHECK
SOURCES = ["api.cu", "kernels.cu", "contract_tc.cu", "fused.cu", "ring.cu", "ring_fused.cu", "ring_fp8.cu", "static_ws.cu", "plan.cpp"]
HEADERS = ["kernels.cuh", "ptx.cuh", "tc_common.cuh", "plan.hpp", "linalg.hpp", os.path.join("..", "..", "include", "cerar.h")]


def _nvcc() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the CERAR library cannot be built")


def is_stale(path: str = LIB_PATH) -> bool:
    if not os.path.exists(path):
        return True
    t = os.path.getmtime(path)
    files = [os.path.join(CSRC, f) for f in SOURCES + HEADERS]
    return any(os.path.getmtime(f) > t for f in files if os.path.exists(f))


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Compile every CUDA/C++ source into libcerar.so (checked=True: into libcerar_checked.so, whose
    kernels compare every address they form with the extent of its buffer); returns its path."""
    out = CHECKED_LIB_PATH if checked else LIB_PATH
    if not force and not is_stale(out):
        return out
    cmd = [
        _nvcc(), "-shared", "-Xcompiler", "-fPIC", "-O3", "-std=c++17", "-lineinfo", "--threads", "4",
        "-gencode", "arch=compute_100a,code=sm_100a",
        "-o", out,
    ] + (["-DCERAR_BOUNDS_CHECK"] if checked else []) + [os.path.join(CSRC, f) for f in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        print(res.stdout + res.stderr)
    return out


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
