"""Builds libqlinear.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libqlinear.so")
SOURCES = ["qlinear.cu", "pack.cpp"]
DEPS = SOURCES + ["layout.h", "dequant.cuh", "sm100_ptx.cuh", "embed.cuh", "gemv.cuh", "gemv_rows.cuh", "gemv_a8.cuh", "kv.cuh", "gemv_stream.cuh", "gemm.cuh", "gemm_pair.cuh", "gemm_pair_ta.cuh", "norm.cuh", "rope.cuh", os.path.join("..", "..", "include", "qlinear.h")]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(os.path.join(CSRC, d)) > t for d in DEPS)


def build(force: bool = False, verbose: bool = False) -> str:
    if not (force or _stale()):
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
           "-Xcompiler", "-fPIC,-O3,-fopenmp", "-shared", "-cudart", "static",
           "-o", LIB] + [os.path.join(CSRC, s) for s in SOURCES] + ["-lgomp"]
    cmd[1:1] = os.environ.get("QL_EXTRA_NVCC_FLAGS", "").split()   # extra compiler flags, e.g. -DNAME for an experiment build
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.check_call(cmd)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
