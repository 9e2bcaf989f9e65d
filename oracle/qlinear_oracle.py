"""CPU oracle for the weight-only quantised linear layer -- TEST INFRASTRUCTURE ONLY.

Nothing in the product package imports this module; only tests, the smoke
check and the benchmark's cpu_baseline leg do.  It shares no code with the
CUDA library (own unpack, own dequantisation, own fp16 handling through numpy).

The result has a plain definition, so the oracle is that definition written
out with numpy in fp64 (paper Section 4.2 for the quantisation schemes and the
FP16 activations, Section 3.7 for dequantisation inside the linear operator,
Section 3.1 for the O x I weight orientation; group size 32 along K for int4 is
the benchmark's choice, the "sub-channel quantisation" of Section 5):

    w[n,k]   = fp16(s[n, k // G]) * q[n,k]                    (exact in fp64)
    y64[m,n] = sum_k fp16(x[m,k]) * w[n,k]                    (fp64)
    A[m,n]   = sum_k |fp16(x[m,k]) * w[n,k]|                  (tolerance denominator)
    y16[m,n] = round-to-nearest-even fp16 of y64[m,n]

`linear` uses numpy's fp64 matmul as the contraction step (summation order is
the library's; fp64 round-off is ~1e-13 relative to A, far below the 1e-3
tolerances).  `linear_loops` calls the C oracle beside this file, which writes
the three loops out with ascending k; the tests require the two to agree.

Parity pins: tests/test_oracle_pins.py (worked examples stored under
tests/golden/, brute force over all byte values, one-hot / zero / closed-form
cases, power-of-two and negation invariants, a double-rounding trap).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_C_SRC = os.path.join(_HERE, "qlinear_oracle.c")
_C_LIB = os.path.join(_HERE, "liboracle.so")


# ----------------------------------------------------------------------------- integer forms
def pack_nibbles(q: np.ndarray) -> np.ndarray:
    """int8 [N, K] in [-8, 7] -> canonical nibble bytes uint8 [N, K/2]:
    byte j = (q[2j] & 0xF) | ((q[2j+1] & 0xF) << 4), two's complement."""
    q = np.asarray(q, dtype=np.int8)
    if q.min(initial=0) < -8 or q.max(initial=0) > 7:
        raise ValueError("int4 value outside [-8, 7]")
    u = q.astype(np.uint8) & 0xF
    return (u[..., 0::2] | (u[..., 1::2] << 4)).astype(np.uint8)


def unpack_nibbles(b: np.ndarray) -> np.ndarray:
    """Inverse of pack_nibbles, by the arithmetic definition v < 8 ? v : v - 16."""
    b = np.asarray(b, dtype=np.uint8)
    lo = (b & 0xF).astype(np.int16)
    hi = (b >> 4).astype(np.int16)
    out = np.empty(b.shape[:-1] + (b.shape[-1] * 2,), dtype=np.int8)
    out[..., 0::2] = np.where(lo < 8, lo, lo - 16)
    out[..., 1::2] = np.where(hi < 8, hi, hi - 16)
    return out


# ----------------------------------------------------------------------------- the definition
def dequantize(q: np.ndarray, s: np.ndarray, group: int) -> np.ndarray:
    """w[n,k] = fp16(s[n, k // G]) * q[n,k] as fp64 [N, K]; group == 0 means G = K."""
    q = np.asarray(q, dtype=np.int8)
    N, K = q.shape
    G = K if group == 0 else group
    if K % G:
        raise ValueError("group must divide K")
    s = np.asarray(s, dtype=np.float16).reshape(N, K // G)
    return np.repeat(s.astype(np.float64), G, axis=1) * q.astype(np.float64)


def linear(x: np.ndarray, q: np.ndarray, s: np.ndarray, group: int):
    """(y64, A, y16) for x fp16 [M, K], q int8 [N, K], s fp16 [N, K/G]."""
    x64 = np.asarray(x, dtype=np.float16).astype(np.float64)
    w = dequantize(q, s, group)
    y64 = x64 @ w.T
    A = np.abs(x64) @ np.abs(w).T
    with np.errstate(over="ignore"):
        y16 = y64.astype(np.float16)  # numpy rounds fp64 -> fp16 once, nearest-even
    return y64, A, y16


def linear_from_nibbles(x, nibble_bytes, s, group):
    """Same, taking int4 weights in the canonical nibble-byte interchange form."""
    return linear(x, unpack_nibbles(nibble_bytes), s, group)


# ----------------------------------------------------------------------------- acceptance
REL_L2_TOL = 1e-3      # ||y - y64||_2 / ||y64||_2 over the whole output
ELEM_TOL = 5e-3        # |y - y64| <= ELEM_TOL * A per element


def check_against(y_test: np.ndarray, y64: np.ndarray, A: np.ndarray):
    """Returns (ok, rel_l2, worst per-element ratio |y - y64| / A)."""
    d = np.asarray(y_test).astype(np.float64) - y64
    den = np.linalg.norm(y64)
    rel = float(np.linalg.norm(d) / den) if den > 0 else float(np.linalg.norm(d))
    with np.errstate(divide="ignore", invalid="ignore"):
        ratio = np.where(A > 0, np.abs(d) / A, np.where(d == 0, 0.0, np.inf))
    worst = float(ratio.max(initial=0.0))
    return (rel <= REL_L2_TOL and worst <= ELEM_TOL), rel, worst


# ----------------------------------------------------------------------------- C oracle
def build_c(force: bool = False) -> str:
    """Compile the C oracle beside this file (gcc, OpenMP) and return the library path."""
    if force or not os.path.exists(_C_LIB) or os.path.getmtime(_C_LIB) < os.path.getmtime(_C_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", _C_LIB, _C_SRC, "-lm"])
    return _C_LIB


_lib = None


def c_lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build_c())
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
        L.oracle_unpack_nibbles.argtypes = [vp, i64, vp]
        L.oracle_unpack_nibbles.restype = None
        L.oracle_fp16_to_double.argtypes = [ctypes.c_uint16]
        L.oracle_fp16_to_double.restype = ctypes.c_double
        L.oracle_double_to_fp16.argtypes = [ctypes.c_double]
        L.oracle_double_to_fp16.restype = ctypes.c_uint16
        L.oracle_dequantize.argtypes = [vp, vp, i32, i32, i32, vp]
        L.oracle_dequantize.restype = None
        L.oracle_linear.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp]
        L.oracle_linear.restype = None
        L.oracle_threads.restype = i32
        L.oracle_set_threads.argtypes = [i32]
        _lib = L
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def unpack_nibbles_loops(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint8)
    out = np.empty(b.shape[:-1] + (b.shape[-1] * 2,), dtype=np.int8)
    c_lib().oracle_unpack_nibbles(_ptr(b), b.size, _ptr(out))
    return out


def dequantize_loops(q: np.ndarray, s: np.ndarray, group: int) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.int8)
    s = np.ascontiguousarray(s, dtype=np.float16)
    N, K = q.shape
    w = np.empty((N, K), dtype=np.float64)
    c_lib().oracle_dequantize(_ptr(q), _ptr(s.view(np.uint16)), N, K, group, _ptr(w))
    return w


def linear_loops(x: np.ndarray, q: np.ndarray, s: np.ndarray, group: int, threads: int = 0):
    """(y64, A, y16) by the C triple loop (ascending k); threads = 0 keeps OpenMP's default."""
    x = np.ascontiguousarray(x, dtype=np.float16)
    M, K = x.shape
    N = q.shape[0]
    if threads:
        c_lib().oracle_set_threads(threads)
    w = dequantize_loops(q, s, group)
    y64 = np.empty((M, N), dtype=np.float64)
    A = np.empty((M, N), dtype=np.float64)
    y16 = np.empty((M, N), dtype=np.uint16)
    c_lib().oracle_linear(_ptr(x.view(np.uint16)), _ptr(w), M, N, K, _ptr(y64), _ptr(A), _ptr(y16))
    return y64, A, y16.view(np.float16)


def threads() -> int:
    return int(c_lib().oracle_threads())


if __name__ == "__main__":
    print(build_c(force=True))
