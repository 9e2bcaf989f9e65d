"""Seeded synthetic tensors for the quantised linear layer.

This module serves both the CPU oracle's tests and the CUDA path's tests and
bench.  It holds none of the linear layer's arithmetic (no unpacking, no
dequantisation, no matmul): it only draws integers, scales and activations.

Every value is a pure function of (seed, tensor_id, element index) through a
counter-based splitmix64 generator, so results do not depend on the torch or
numpy version, on the order tensors are drawn in, or on how a tensor is split.

Distributions (they stand in for the Gemma2-2B / Llama3.1-8B checkpoints the
paper evaluates, Section 4.2, which are not available offline):
  * integer weights: uniform over [lo, hi], unbiased (rejection on the
    multiply-shift range reduction);
  * scales: uniform in [1e-3, 1e-2] drawn in fp64, rounded to nearest-even fp16;
  * activations: Box-Muller N(0, 1) in fp64, rounded to nearest-even fp16.
"""
from __future__ import annotations

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_CHUNK = 1 << 18  # elements per vectorised block (keeps temporaries cache-sized)


def _mix(z: np.ndarray) -> np.ndarray:
    """splitmix64 output function on an array of uint64 counters."""
    with np.errstate(over="ignore"):
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        return z ^ (z >> np.uint64(31))


def _stream_key(seed: int, tensor_id: int, lane: int = 0) -> np.uint64:
    """One 64-bit key per (seed, tensor, lane); lanes give independent draws per element."""
    k = np.array([(seed * 0x9E3779B97F4A7C15 + 0x632BE59BD9B4E019) & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64)
    k = _mix(k)
    k = _mix(k ^ np.uint64((tensor_id * 0xD1342543DE82EF95 + 1) & 0xFFFFFFFFFFFFFFFF))
    k = _mix(k ^ np.uint64((lane * 0xA0761D6478BD642F + 2) & 0xFFFFFFFFFFFFFFFF))
    return k[0]


def raw_u64(seed: int, tensor_id: int, start: int, count: int, lane: int = 0) -> np.ndarray:
    """Elements [start, start+count) of stream (seed, tensor_id, lane) as uint64."""
    key = _stream_key(seed, tensor_id, lane)
    idx = np.arange(start, start + count, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return _mix(key + (idx + np.uint64(1)) * _GOLDEN)


def uniform_ints(seed: int, tensor_id: int, shape, lo: int, hi: int) -> np.ndarray:
    """int8 array of `shape`, uniform over the closed range [lo, hi]."""
    assert -128 <= lo <= hi <= 127
    n = int(np.prod(shape))
    r = hi - lo + 1
    out = np.empty(n, dtype=np.int8)
    reject_below = np.uint64((1 << 32) % r)
    for s in range(0, n, _CHUNK):
        c = min(_CHUNK, n - s)
        prod = (raw_u64(seed, tensor_id, s, c, 0) >> np.uint64(32)) * np.uint64(r)
        vals = (prod >> np.uint64(32)).astype(np.int64) + lo
        todo = np.nonzero((prod & np.uint64(0xFFFFFFFF)) < reject_below)[0]
        lane = 1
        while todo.size:  # rare: probability r / 2^32 per element
            prod = (raw_u64(seed, tensor_id, s, c, lane)[todo] >> np.uint64(32)) * np.uint64(r)
            ok = (prod & np.uint64(0xFFFFFFFF)) >= reject_below
            vals[todo[ok]] = (prod[ok] >> np.uint64(32)).astype(np.int64) + lo
            todo = todo[~ok]
            lane += 1
        out[s:s + c] = vals.astype(np.int8)
    return out.reshape(shape)


def _unit(z: np.ndarray) -> np.ndarray:
    """uint64 -> fp64 in [0, 1) with 53 random bits."""
    return (z >> np.uint64(11)).astype(np.float64) * (1.0 / (1 << 53))


def uniform_scales_fp16(seed: int, tensor_id: int, shape, lo: float = 1e-3, hi: float = 1e-2) -> np.ndarray:
    """fp16 array of `shape`: uniform in [lo, hi] in fp64, then rounded to nearest-even fp16."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.float16)
    for s in range(0, n, _CHUNK):
        c = min(_CHUNK, n - s)
        u = _unit(raw_u64(seed, tensor_id, s, c))
        out[s:s + c] = (lo + u * (hi - lo)).astype(np.float16)
    return out.reshape(shape)


def normal_fp16(seed: int, tensor_id: int, shape) -> np.ndarray:
    """fp16 array of `shape`: Box-Muller N(0,1) in fp64, rounded to nearest-even fp16."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.float16)
    for s in range(0, n, _CHUNK):
        c = min(_CHUNK, n - s)
        u1 = 1.0 - _unit(raw_u64(seed, tensor_id, s, c, lane=0))  # (0, 1]
        u2 = _unit(raw_u64(seed, tensor_id, s, c, lane=1))
        out[s:s + c] = (np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)).astype(np.float16)
    return out.reshape(shape)
