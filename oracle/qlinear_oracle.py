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
cases, power-of-two and negation invariants, a double-rounding trap) and
tests/test_oracle_pins_next.py for the three extensions further down (fused
gating, residual + RMS normalisation and rotary embedding + QKV layout, Section 3.6; int8 activation
quantisation, Section 3.7; the KV cache as weights, Section 3.8).  No function
here is unpinned.
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


# ----------------------------------------------------------------------------- fused gating (paper Section 3.6)
# The paper's operator fusion merges "element-wise operators from two branches with a fully connected
# operator" (Section 3.6, the left example of its fusion figure): in the feed-forward block the gate and up
# projections read the same x and meet in an element-wise product, y = act(W_gate x) * (W_up x).  The paper
# names no activation; the model families it evaluates use SiLU (Llama) and the tanh form of GELU (Gemma).
# Reading: both projections stay unrounded until the product (the fused kernel keeps them in fp32
# accumulators), and the product is rounded to fp16 once.
_SQRT_2_OVER_PI = 0.7978845608028654  # sqrt(2 / pi)


def activation(g: np.ndarray, act: str) -> np.ndarray:
    """fp64 activation by its textbook formula: 'identity', 'silu' (g * sigmoid(g)), 'gelu_tanh'."""
    g = np.asarray(g, dtype=np.float64)
    if act == "identity":
        return g.copy()
    if act == "silu":
        return g / (1.0 + np.exp(-g))
    if act == "gelu_tanh":
        return 0.5 * g * (1.0 + np.tanh(_SQRT_2_OVER_PI * (g + 0.044715 * g * g * g)))
    raise ValueError(act)


# Largest slope of the activation (bounds how an error in the gate projection reaches the product).
ACT_LIPSCHITZ = {"identity": 1.0, "silu": 1.0999, "gelu_tanh": 1.1290}


def gated_linear(x, q_gate, s_gate, q_up, s_up, group: int, act: str):
    """(y64, bound, y16): y64 = act(gate64) * up64 with gate64 / up64 the two `linear` results.
    bound[m,n] is the per-element acceptance bound that follows from the linear layer's own
    (|d gate| <= ELEM_TOL * A_gate, |d up| <= ELEM_TOL * A_up), first order, plus one fp16 rounding:
        ELEM_TOL * (L_act * |up64| * A_gate + |act(gate64)| * A_up) + 2^-10 * |y64|."""
    g64, A_g, _ = linear(x, q_gate, s_gate, group)
    u64, A_u, _ = linear(x, q_up, s_up, group)
    a = activation(g64, act)
    y64 = a * u64
    bound = ELEM_TOL * (ACT_LIPSCHITZ[act] * np.abs(u64) * A_g + np.abs(a) * A_u) + 2.0 ** -10 * np.abs(y64)
    with np.errstate(over="ignore"):
        y16 = y64.astype(np.float16)
    return y64, bound, y16


def check_gated(y_test, y64, bound):
    """Returns (ok, rel_l2, worst |y - y64| / bound): rel-L2 <= REL_L2_TOL over the whole output, every element inside its bound."""
    d = np.asarray(y_test).astype(np.float64) - y64
    den = np.linalg.norm(y64)
    rel = float(np.linalg.norm(d) / den) if den > 0 else float(np.linalg.norm(d))
    with np.errstate(divide="ignore", invalid="ignore"):
        ratio = np.where(bound > 0, np.abs(d) / bound, np.where(d == 0, 0.0, np.inf))
    worst = float(ratio.max(initial=0.0))
    return (rel <= REL_L2_TOL and worst <= 1.0), rel, worst


# ----------------------------------------------------------------------------- activation quantisation (paper Section 3.7)
# The method the paper describes for operators with external weights quantises the ACTIVATIONS too: a
# quantisation kernel "converts the floating-point input activations to 8-bit integers and computes the
# requisite quantization parameters", a second kernel multiplies them with the pre-quantised weights using
# integer instructions and "perform[s] dequantization on the output activations" (prefill); in decode the
# quantisation happens inside the fully-connected kernel.  The steps below follow that order.  The paper
# gives neither the granularity nor the rounding; the readings taken (recorded in the design notes):
#   * one scale per token (row of x), symmetric, zero-point 0:  scale_x[m] = amax_m / 127,  amax_m = max_k |x[m,k]|
#   * a floating-point value decides an integer here, so the decision is taken in ONE stated precision, fp32,
#     with these IEEE operations:  r = 127 / amax (division),  v = x * r (multiplication),
#     xq = round-half-to-even(v) clamped to [-127, 127];  a row of zeros gets scale 1 and xq = 0
#   * the integer dot products are exact (accumulated in int64 here), one per scale group of the weights
#   * output dequantisation  y = scale_x[m] * sum_g s[n,g] * acc[m,n,g],  in fp64 here from the fp32 scale_x
#     and the fp16 weight scales, then one rounding to fp16.


def quantize_activations(x: np.ndarray):
    """x fp16 [M, K] -> (xq int8 [M, K], scale_x float32 [M]) by the fp32 steps stated above."""
    x32 = np.asarray(x, dtype=np.float16).astype(np.float32)
    amax = np.abs(x32).max(axis=1)
    live = amax > 0
    safe = np.where(live, amax, np.float32(1.0)).astype(np.float32)
    r = (np.float32(127.0) / safe).astype(np.float32)                    # one IEEE fp32 division per token
    v = (x32 * r[:, None]).astype(np.float32)                            # one IEEE fp32 multiplication per element
    xq = np.clip(np.rint(v), -127, 127).astype(np.int8)                  # rint = round half to even
    scale = np.where(live, (safe / np.float32(127.0)).astype(np.float32), np.float32(1.0)).astype(np.float32)
    return xq, scale


def linear_int8_activations(x, q, s, group: int):
    """(y64, acc, xq, scale_x, y16): the linear layer with per-token int8 activations.
    acc int64 [M, N, K/G] are the exact integer dot products per scale group."""
    q = np.asarray(q, dtype=np.int8)
    N, K = q.shape
    G = K if group == 0 else group
    xq, scale_x = quantize_activations(x)
    M = xq.shape[0]
    # exact integers through the fp64 matmul: every product is below 2^14 and a sum over K <= 2^24 terms stays far
    # below 2^53, so fp64 represents every partial sum exactly whatever the summation order
    xg, qg = xq.astype(np.float64).reshape(M, K // G, G), q.astype(np.float64).reshape(N, K // G, G)
    acc = np.rint(np.stack([xg[:, g, :] @ qg[:, g, :].T for g in range(K // G)], axis=2)).astype(np.int64)
    s64 = np.asarray(s, dtype=np.float16).reshape(N, K // G).astype(np.float64)
    y64 = scale_x.astype(np.float64)[:, None] * np.einsum("mng,ng->mn", acc.astype(np.float64), s64)
    with np.errstate(over="ignore"):
        y16 = y64.astype(np.float16)
    return y64, acc, xq, scale_x, y16


# ----------------------------------------------------------------------------- KV cache as weights (paper Section 3.8)
# The attention matmuls are run as operators with weights: the K cache is stored O x I with O = cache
# positions and I = head dimension (it "represent[s] K^T for the QK^T computation"), the V cache O x I with
# O = head dimension and I = cache positions, so that the second product comes out as [query rows, d_h].
# Both are then the linear layer above; only the meaning of the axes differs.  The caches are held in the
# int8 per-output-channel format of Section 4.2 (one scale per cached key for K; one scale per head
# dimension for V), the reading recorded in the design notes: the paper does not say how its cache is stored.


def kv_quantize_rows(a: np.ndarray):
    """fp16 [T, d] -> (int8 [T, d], fp16 scale [T]): one scale per row (per cached token),
    s = fp16(amax / 127) with the division in fp32, q = round-half-even(a / s) in fp32 clamped to [-127, 127];
    a row whose scale rounds to zero (all zeros, or below fp16's range) is stored as zeros with scale 1."""
    a32 = np.asarray(a, dtype=np.float16).astype(np.float32)
    amax = np.abs(a32).max(axis=1)
    s16 = (amax / np.float32(127.0)).astype(np.float32).astype(np.float16)
    dead = s16.astype(np.float32) == 0
    sf = np.where(dead, np.float32(1.0), s16.astype(np.float32)).astype(np.float32)
    with np.errstate(over="ignore"):
        v = (a32 / sf[:, None]).astype(np.float32)
    q = np.clip(np.rint(v), -127, 127).astype(np.int8)
    q[dead] = 0
    return q, np.where(dead, np.float16(1.0), s16).astype(np.float16)


def kv_attention(qry, k, v, prob):
    """The two attention products over a cache built from fp16 keys k [T, d] and values v [T, d]:
    returns (scores64 [R, T], A_scores, out64 [R, d], A_out).  The value scales are per token, i.e. per INPUT
    channel of the V layer, so they are folded into the probabilities first: x' = fp16(prob * s_v) (the product of
    two fp16 numbers is exact in fp32; one rounding to fp16), out = x' . q_v with unit channel scales."""
    k_q, k_s = kv_quantize_rows(k)
    v_q, v_s = kv_quantize_rows(v)
    sc64, A_sc, _ = kv_scores(qry, k_q, k_s)
    xp = (np.asarray(prob, np.float16).astype(np.float32) * v_s.astype(np.float32)[None, :]).astype(np.float16)
    out64, A_out, _ = kv_output(xp, np.ascontiguousarray(v_q.T), np.ones(v_q.shape[1], np.float16))
    return sc64, A_sc, out64, A_out


def kv_scores(qry, k_q, k_s):
    """scores64 [R, T] = qry [R, d_h] . Kcache^T, K cache k_q int8 [T, d_h] (O = T, I = d_h), k_s fp16 [T]."""
    return linear(qry, k_q, k_s, 0)


def kv_output(prob, v_q, v_s):
    """out64 [R, d_h] = prob [R, T] . V, V cache v_q int8 [d_h, T] (O = d_h, I = T), v_s fp16 [d_h]."""
    return linear(prob, v_q, v_s, 0)


# ----------------------------------------------------------------------------- residual + RMS normalisation (paper Section 3.6)
# The paper's second fusion example merges "residual connection and element-wise operations with a manually optimized
# RMS normalization operator": the operator that produces the linear layer's input.  The paper gives no formulas; the
# readings taken (recorded in the design notes) are the ones the paper's models use:
#   h[m,k]  = x[m,k] + r[m,k]                                   residual connection (the sum of two fp16 values, exact)
#   ms[m]   = (1/K) * sum_k h[m,k]^2                            mean square over the hidden dimension
#   y[m,k]  = h[m,k] / sqrt(ms[m] + eps) * (offset + g[k])      RMS normalisation with its element-wise scale
#             (offset = 0: Llama; offset = 1: Gemma stores the scale as g - 1)
# The normalisation is computed from the UNROUNDED sum h (a merged operator has it in registers); the operator also
# returns fp16(h), the residual stream for the next block.  Everything in fp64 here, one rounding to fp16 per output.
def residual_rmsnorm(x, r, g, eps: float, offset: float = 0.0):
    """x, r fp16 [M, K] (r may be None: no residual), g fp16 [K] -> (h64, h16, y64, y16)."""
    h = np.asarray(x, dtype=np.float16).astype(np.float64)
    if r is not None:
        h = h + np.asarray(r, dtype=np.float16).astype(np.float64)
    ms = np.mean(h * h, axis=1, keepdims=True)
    y = h / np.sqrt(ms + float(eps)) * (float(offset) + np.asarray(g, dtype=np.float16).astype(np.float64))[None, :]
    with np.errstate(over="ignore"):
        return h, h.astype(np.float16), y, y.astype(np.float16)


def residual_rmsnorm_bound(h64, y64, K: int):
    """Acceptance bounds (|dh|, |dy|) for an fp32 implementation: h is exact before its rounding (2^-11 relative, or
    2^-25 absolute among the fp16 subnormals); y carries that rounding plus the fp32 arithmetic: a sum of K squares
    kept in at least 128 partial sums that are then added pairwise (K / 128 + 7 additions deep), the square root, the
    division and two multiplications, half an fp32 ulp (2^-24) each, first order."""
    bh = 2.0 ** -11 * np.abs(h64) + 2.0 ** -25
    by = (2.0 ** -11 + (K / 128.0 + 7 + 5) * 2.0 ** -24) * np.abs(y64) + 2.0 ** -25
    return bh, by


# ----------------------------------------------------------------------------- rotary embedding + QKV layout (paper Section 3.6)
# The paper's hand-written attention-block kernel "combine[s] rotary embedding with the layout transformations of query
# (Q), key (K), and value (V) projections", the query going from (B, 1, S, h_q * d_h) to (B * h_kv, S * h_q / h_kv, d_h).
# What the paper leaves open, and the readings taken (recorded in the design notes):
#   * rotary convention: the rotate-half form of the paper's models (Llama, Gemma): element i < d_h / 2 pairs with
#     element i + d_h / 2;  out_i = x_i * cos - x_{i+d/2} * sin,  out_{i+d/2} = x_{i+d/2} * cos + x_i * sin
#   * the angles come as tables cos[p, i], sin[p, i] (fp32, one row per position p, i < d_h / 2) and a position per token,
#     so that any frequency schedule can be used and no trigonometry is left to the kernel
#   * order inside the merged query dimension: the source is (B, S, h_kv, g, d_h) with g = h_q / h_kv; the kernel swaps
#     the S and h_kv axes, so row s * g + j of KV head hk holds query head hk * g + j of token s
#   * K (rotated) and V (not rotated) go to (B * h_kv, S, d_h): one contiguous [S, d_h] block per KV head, the rows
#     the KV cache of Section 3.8 takes in.
def rope_qkv(q, k, v, pos, cos, sin, B: int, S: int, h_q: int, h_kv: int, d_h: int):
    """q fp16 [B*S, h_q*d_h], k, v fp16 [B*S, h_kv*d_h], pos int [B*S], cos / sin fp32 [n_pos, d_h/2]
    -> (q_out64 [B*h_kv, S*g, d_h], k_out64 [B*h_kv, S, d_h], v_out64 [B*h_kv, S, d_h], amp_q, amp_k) in fp64;
    amp = |x_i| + |x_{i+d/2}| per output element (the tolerance denominator of the rotation)."""
    g, half = h_q // h_kv, d_h // 2
    assert h_q == g * h_kv and d_h == 2 * half
    c = np.asarray(cos, dtype=np.float32).astype(np.float64)[np.asarray(pos)]           # [B*S, half]
    s_ = np.asarray(sin, dtype=np.float32).astype(np.float64)[np.asarray(pos)]

    def rotate(t, heads):
        t = np.asarray(t, dtype=np.float16).astype(np.float64).reshape(B * S, heads, d_h)
        lo, hi = t[:, :, :half], t[:, :, half:]
        out = np.concatenate([lo * c[:, None, :] - hi * s_[:, None, :], hi * c[:, None, :] + lo * s_[:, None, :]], axis=2)
        amp = np.concatenate([np.abs(lo) + np.abs(hi)] * 2, axis=2)
        return out, amp

    def to_heads(t, heads):                                              # [B*S, heads, d_h] -> [B, h_kv, S, heads / h_kv, d_h]
        return t.reshape(B, S, h_kv, heads // h_kv, d_h).transpose(0, 2, 1, 3, 4)

    rq, aq = rotate(q, h_q)
    rk, ak = rotate(k, h_kv)
    vv = np.asarray(v, dtype=np.float16).astype(np.float64).reshape(B * S, h_kv, d_h)
    q_out = to_heads(rq, h_q).reshape(B * h_kv, S * g, d_h)
    k_out = to_heads(rk, h_kv).reshape(B * h_kv, S, d_h)
    v_out = to_heads(vv, h_kv).reshape(B * h_kv, S, d_h)
    return q_out, k_out, v_out, to_heads(aq, h_q).reshape(B * h_kv, S * g, d_h), to_heads(ak, h_kv).reshape(B * h_kv, S, d_h)


def rope_bound(y64, amp):
    """|dy| allowed for an fp32 implementation: the fp16 rounding of the result (2^-11 relative, 2^-25 among the
    subnormals) plus two products and one sum in fp32 (half an ulp of 2^-24 each, on terms no larger than amp)."""
    return 2.0 ** -11 * np.abs(y64) + 3 * 2.0 ** -24 * amp + 2.0 ** -25


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
