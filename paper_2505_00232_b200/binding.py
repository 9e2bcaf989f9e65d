"""Thin ctypes binding over libqlinear.so (see include/qlinear.h): argument marshalling only.

Every arithmetic step runs inside the library's CUDA kernels (or, for pack/unpack, its host
packer).  torch is used for device memory and streams.  There is no CPU fallback: if the shared
library has not been built, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqlinear.so")

QL_OK = 0
QL_ERR_INVALID_ARG, QL_ERR_UNSUPPORTED, QL_ERR_ALLOC, QL_ERR_CUDA, QL_ERR_DEVICE_TIMEOUT, QL_ERR_ARCH = 1, 2, 3, 4, 5, 6
QL_PATH_GEMV, QL_PATH_GEMM = 1, 2
QL_ACT_IDENTITY, QL_ACT_SILU, QL_ACT_GELU_TANH = 0, 1, 2
ACTIVATIONS = {"identity": QL_ACT_IDENTITY, "silu": QL_ACT_SILU, "gelu_tanh": QL_ACT_GELU_TANH}

EXPORTS = (
    "qlinear_packed_size", "qlinear_pack", "qlinear_unpack", "qlinear_create", "qlinear_forward", "qlinear_forward_group", "qlinear_forward_batch", "qlinear_forward_gated", "qlinear_forward_a8", "qlinear_quantize_activations", "qlinear_kv_append", "qlinear_kv_scores", "qlinear_kv_output", "qlinear_kv_append_heads", "qlinear_kv_scores_heads", "qlinear_kv_output_heads", "qlinear_embed", "qlinear_residual_rmsnorm", "qlinear_rope_qkv",
    "qlinear_path_for", "qlinear_debug_unpack_device", "qlinear_debug_expire_wait", "qlinear_debug_null_launch", "qlinear_device_status", "qlinear_decode_static", "qlinear_destroy",
    "qlinear_status_string", "qlinear_version", "qlinear_debug_plan", "qlinear_debug_config_reads",
)


class QLinearError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (ql_status {status})")


class qlinear_desc(ctypes.Structure):
    _fields_ = [("N", ctypes.c_int32), ("K", ctypes.c_int32), ("bits", ctypes.c_int32), ("group", ctypes.c_int32)]


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2505_00232_b200.build` "
            "(nvcc, sm_100a). There is no fallback path.")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32 = ctypes.c_void_p, ctypes.c_int32
    dp = ctypes.POINTER(qlinear_desc)
    lib.qlinear_packed_size.argtypes = [dp]
    lib.qlinear_packed_size.restype = ctypes.c_size_t
    lib.qlinear_pack.argtypes = [dp, vp, vp, vp, ctypes.c_size_t]
    lib.qlinear_pack.restype = ctypes.c_int
    lib.qlinear_unpack.argtypes = [dp, vp, vp, vp]
    lib.qlinear_unpack.restype = ctypes.c_int
    lib.qlinear_create.argtypes = [dp, vp, ctypes.c_int, ctypes.POINTER(vp)]
    lib.qlinear_create.restype = ctypes.c_int
    lib.qlinear_forward.argtypes = [vp, vp, vp, i32, vp]
    lib.qlinear_forward.restype = ctypes.c_int
    lib.qlinear_path_for.argtypes = [vp, i32]
    lib.qlinear_path_for.restype = i32
    lib.qlinear_debug_unpack_device.argtypes = [vp, vp, vp]
    lib.qlinear_debug_unpack_device.restype = ctypes.c_int
    lib.qlinear_forward_group.argtypes = [ctypes.POINTER(vp), ctypes.c_int32, vp, ctypes.POINTER(vp), ctypes.c_int32, vp]
    lib.qlinear_forward_group.restype = ctypes.c_int
    lib.qlinear_forward_batch.argtypes = [ctypes.POINTER(vp), ctypes.c_int32, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.c_int32, vp]
    lib.qlinear_forward_batch.restype = ctypes.c_int
    lib.qlinear_forward_gated.argtypes = [vp, vp, vp, vp, i32, i32, vp]
    lib.qlinear_forward_gated.restype = ctypes.c_int
    lib.qlinear_forward_a8.argtypes = [vp, vp, vp, i32, vp]
    lib.qlinear_forward_a8.restype = ctypes.c_int
    lib.qlinear_quantize_activations.argtypes = [vp, vp, vp, i32, i32, ctypes.c_int, vp]
    lib.qlinear_quantize_activations.restype = ctypes.c_int
    lib.qlinear_kv_append.argtypes = [vp, vp, vp, vp, vp, i32, i32, vp]
    lib.qlinear_kv_append.restype = ctypes.c_int
    lib.qlinear_kv_scores.argtypes = [vp, vp, vp, i32, vp]
    lib.qlinear_kv_scores.restype = ctypes.c_int
    lib.qlinear_kv_output.argtypes = [vp, vp, vp, vp, vp, i32, vp]
    lib.qlinear_kv_output.restype = ctypes.c_int
    lib.qlinear_embed.argtypes = [vp, vp, ctypes.c_int32, vp, vp]
    lib.qlinear_embed.restype = ctypes.c_int
    lib.qlinear_residual_rmsnorm.argtypes = [vp, vp, vp, ctypes.c_float, ctypes.c_float, vp, vp, i32, i32, ctypes.c_int, vp]
    lib.qlinear_residual_rmsnorm.restype = ctypes.c_int
    lib.qlinear_rope_qkv.argtypes = [vp, vp, vp, vp, vp, vp, i32, vp, vp, vp, i32, i32, i32, i32, i32, ctypes.c_int, vp]
    lib.qlinear_rope_qkv.restype = ctypes.c_int
    lib.qlinear_debug_expire_wait.argtypes = [vp, vp]
    lib.qlinear_debug_expire_wait.restype = ctypes.c_int
    lib.qlinear_debug_null_launch.argtypes = [vp, ctypes.c_int32, ctypes.c_int32, vp]
    lib.qlinear_debug_null_launch.restype = ctypes.c_int
    pvp = ctypes.POINTER(ctypes.c_void_p)
    lib.qlinear_kv_append_heads.argtypes = [pvp, pvp, ctypes.c_int32, vp, vp, ctypes.c_int64, ctypes.c_int64, pvp, ctypes.c_int32, ctypes.c_int32, vp]
    lib.qlinear_kv_append_heads.restype = ctypes.c_int
    lib.qlinear_kv_scores_heads.argtypes = [pvp, ctypes.c_int32, vp, vp, ctypes.c_int32, vp]
    lib.qlinear_kv_scores_heads.restype = ctypes.c_int
    lib.qlinear_kv_output_heads.argtypes = [pvp, ctypes.c_int32, vp, pvp, vp, ctypes.c_int32, vp]
    lib.qlinear_kv_output_heads.restype = ctypes.c_int
    lib.qlinear_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32)]
    lib.qlinear_device_status.restype = ctypes.c_int
    lib.qlinear_decode_static.argtypes = [dp, vp, vp, vp, i32, ctypes.c_int, vp]
    lib.qlinear_decode_static.restype = ctypes.c_int
    lib.qlinear_destroy.argtypes = [vp]
    lib.qlinear_destroy.restype = ctypes.c_int
    lib.qlinear_status_string.argtypes = [ctypes.c_int]
    lib.qlinear_status_string.restype = ctypes.c_char_p
    lib.qlinear_version.restype = ctypes.c_uint32
    lib.qlinear_debug_plan.argtypes = [vp, i32, ctypes.POINTER(i32), i32]
    lib.qlinear_debug_plan.restype = i32
    lib.qlinear_debug_config_reads.restype = ctypes.c_uint32
    return lib


lib = _load()


def status_string(status: int) -> str:
    return lib.qlinear_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != QL_OK:
        raise QLinearError(status, where)


def _np_ptr(a: np.ndarray) -> ctypes.c_void_p:
    return a.ctypes.data_as(ctypes.c_void_p)


@dataclass(frozen=True)
class Desc:
    N: int
    K: int
    bits: int
    group: int = 0

    def c(self) -> qlinear_desc:
        return qlinear_desc(self.N, self.K, self.bits, self.group)

    @property
    def n_groups(self) -> int:
        return 1 if self.group == 0 else self.K // self.group


# ---------------------------------------------------------------------------- host calls
def qlinear_packed_size(desc: Desc) -> int:
    return int(lib.qlinear_packed_size(ctypes.byref(desc.c())))


def qlinear_pack(desc: Desc, q: np.ndarray, s: np.ndarray) -> np.ndarray:
    """q int8 [N, K] (one integer per byte), s fp16 [N] or [N, K/group] -> packed blob (uint8 array)."""
    q = np.ascontiguousarray(q, dtype=np.int8)
    s = np.ascontiguousarray(s, dtype=np.float16)
    size = qlinear_packed_size(desc)
    if size == 0:
        raise QLinearError(QL_ERR_UNSUPPORTED, "qlinear_packed_size")
    if q.shape != (desc.N, desc.K) or s.size != desc.N * desc.n_groups:
        raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_pack (shape)")
    out = np.empty(size, dtype=np.uint8)
    _check(lib.qlinear_pack(ctypes.byref(desc.c()), _np_ptr(q), _np_ptr(s), _np_ptr(out), size), "qlinear_pack")
    return out


def qlinear_unpack(desc: Desc, packed: np.ndarray):
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    if packed.size < qlinear_packed_size(desc) or qlinear_packed_size(desc) == 0:
        raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_unpack (size)")
    q = np.empty((desc.N, desc.K), dtype=np.int8)
    s = np.empty((desc.N, desc.n_groups), dtype=np.float16)
    _check(lib.qlinear_unpack(ctypes.byref(desc.c()), _np_ptr(packed), _np_ptr(q), _np_ptr(s)), "qlinear_unpack")
    return q, s


# ---------------------------------------------------------------------------- device calls
def _stream_ptr(stream) -> ctypes.c_void_p:
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def qlinear_decode_static(desc: Desc, packed, x, out=None, stream=None):
    """Decode (M <= 8) without a handle and without any allocation inside the library: the caller passes the
    packed device tensor, x and (optionally) the output tensor; see include/qlinear.h."""
    import torch
    if (x.dim() != 2 or x.shape[1] != desc.K or x.dtype != torch.float16 or not x.is_cuda or not x.is_contiguous()):
        raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_decode_static (x must be contiguous fp16 CUDA [M, K])")
    if (not packed.is_cuda or packed.dtype != torch.uint8 or not packed.is_contiguous()
            or packed.numel() < qlinear_packed_size(desc) or packed.device != x.device):
        raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_decode_static (packed must be a contiguous uint8 CUDA tensor of the packed size)")
    M = x.shape[0]
    if out is None:
        out = torch.empty((M, desc.N), dtype=torch.float16, device=x.device)
    elif out.shape != (M, desc.N) or out.dtype != torch.float16 or not out.is_contiguous() or out.device != x.device:
        raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_decode_static (bad out tensor)")
    _check(lib.qlinear_decode_static(ctypes.byref(desc.c()), ctypes.c_void_p(packed.data_ptr()),
                                     ctypes.c_void_p(x.data_ptr()), ctypes.c_void_p(out.data_ptr()), M,
                                     x.device.index or 0, _stream_ptr(stream)), "qlinear_decode_static")
    return out


def qlinear_forward_group_raw(lins, x_ptr: int, y_ptrs, M: int, stream=None) -> None:
    """qlinear_forward_group on raw device pointers: the layers `lins` applied to one x."""
    n = len(lins)
    hs = (ctypes.c_void_p * n)(*[l._h for l in lins])
    ys = (ctypes.c_void_p * n)(*[ctypes.c_void_p(int(p)) for p in y_ptrs])
    _check(lib.qlinear_forward_group(hs, n, ctypes.c_void_p(x_ptr), ys, M, _stream_ptr(stream)), "qlinear_forward_group")


def qlinear_forward_batch_raw(lins, x_ptrs, y_ptrs, M: int, stream=None) -> None:
    """qlinear_forward_batch on raw device pointers: layer i applied to its own input x_ptrs[i]."""
    n = len(lins)
    hs = (ctypes.c_void_p * n)(*[l._h for l in lins])
    xs = (ctypes.c_void_p * n)(*[ctypes.c_void_p(int(p)) for p in x_ptrs])
    ys = (ctypes.c_void_p * n)(*[ctypes.c_void_p(int(p)) for p in y_ptrs])
    _check(lib.qlinear_forward_batch(hs, n, xs, ys, M, _stream_ptr(stream)), "qlinear_forward_batch")


def qlinear_forward_batch(lins, xs, outs=None, stream=None):
    """xs: one fp16 CUDA tensor [M, K] per layer -> list of fp16 [M, N_i] (one launch for M <= 8: up to 4 layers, 8 if they are int8)."""
    import torch
    K, M = lins[0].desc.K, xs[0].shape[0]
    if len(xs) != len(lins):
        raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_forward_batch (one input per layer)")
    for x in xs:
        if x.dim() != 2 or tuple(x.shape) != (M, K) or x.dtype != torch.float16 or not x.is_cuda or not x.is_contiguous():
            raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_forward_batch (every x must be contiguous fp16 CUDA [M, K])")
    if outs is None:
        outs = [torch.empty((M, l.desc.N), dtype=torch.float16, device=xs[0].device) for l in lins]
    for l, o in zip(lins, outs):
        if o.shape != (M, l.desc.N) or o.dtype != torch.float16 or not o.is_contiguous():
            raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_forward_batch (bad out tensor)")
    qlinear_forward_batch_raw(lins, [x.data_ptr() for x in xs], [o.data_ptr() for o in outs], M, stream)
    return outs


def kv_scores_batch(caches, q_rows, stream=None):
    """The score product of up to 8 KV heads in one launch: caches[i].scores(q_rows[i]) for every i (paper Section 3.8)."""
    return qlinear_forward_batch([c.k for c in caches], q_rows, stream=stream)


def qlinear_forward_group(lins, x, outs=None, stream=None):
    """x: fp16 CUDA tensor [M, K] -> list of fp16 [M, N_i], one per layer (one launch for M <= 8)."""
    import torch
    K = lins[0].desc.K
    if x.dim() != 2 or x.shape[1] != K or x.dtype != torch.float16 or not x.is_cuda or not x.is_contiguous():
        raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_forward_group (x must be contiguous fp16 CUDA [M, K])")
    M = x.shape[0]
    if outs is None:
        outs = [torch.empty((M, l.desc.N), dtype=torch.float16, device=x.device) for l in lins]
    for l, o in zip(lins, outs):
        if o.shape != (M, l.desc.N) or o.dtype != torch.float16 or not o.is_contiguous():
            raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_forward_group (bad out tensor)")
    qlinear_forward_group_raw(lins, x.data_ptr(), [o.data_ptr() for o in outs], M, stream)
    return outs


def qlinear_forward_gated_raw(gate, up, x_ptr: int, y_ptr: int, M: int, act: str, stream=None) -> None:
    _check(lib.qlinear_forward_gated(gate._h, up._h, ctypes.c_void_p(x_ptr), ctypes.c_void_p(y_ptr), M, ACTIVATIONS[act],
                                     _stream_ptr(stream)), "qlinear_forward_gated")


def qlinear_forward_gated(gate, up, x, act: str = "silu", out=None, stream=None):
    """y = act(x . W_gate^T) * (x . W_up^T) as fp16 [M, N], from one fused launch where the shape allows."""
    import torch
    K, N = gate.desc.K, gate.desc.N
    if x.dim() != 2 or x.shape[1] != K or x.dtype != torch.float16 or not x.is_cuda or not x.is_contiguous():
        raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_forward_gated (x must be contiguous fp16 CUDA [M, K])")
    if act not in ACTIVATIONS:
        raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_forward_gated (unknown activation)")
    M = x.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=torch.float16, device=x.device)
    elif out.shape != (M, N) or out.dtype != torch.float16 or not out.is_contiguous():
        raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_forward_gated (bad out tensor)")
    qlinear_forward_gated_raw(gate, up, x.data_ptr(), out.data_ptr(), M, act, stream)
    return out


def qlinear_quantize_activations(x, stream=None):
    """x fp16 CUDA [M, K] -> (xq int8 [M, K], scale fp32 [M]): the prefill stage's quantisation kernel."""
    import torch
    if x.dim() != 2 or x.dtype != torch.float16 or not x.is_cuda or not x.is_contiguous() or x.shape[1] % 32:
        raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_quantize_activations (x must be contiguous fp16 CUDA [M, K], K % 32 == 0)")
    M, K = x.shape
    xq = torch.empty((M, K), dtype=torch.int8, device=x.device)
    scale = torch.empty((M,), dtype=torch.float32, device=x.device)
    _check(lib.qlinear_quantize_activations(ctypes.c_void_p(x.data_ptr()), ctypes.c_void_p(xq.data_ptr()), ctypes.c_void_p(scale.data_ptr()),
                                            M, K, x.device.index or 0, _stream_ptr(stream)), "qlinear_quantize_activations")
    return xq, scale


def qlinear_residual_rmsnorm(x, residual, gamma, eps: float, gamma_offset: float = 0.0, h_out=None, y_out=None, want_h=True, stream=None):
    """x, residual (or None) fp16 CUDA [M, K], gamma fp16 [K] -> (h, y): h = x + residual, y = rmsnorm(h) * (gamma_offset + gamma).
    h_out / y_out may be given (h_out may be x or residual: in place); want_h=False skips the h output (h is then None)."""
    import torch
    def ok(t, shape):
        return t.dtype == torch.float16 and t.is_cuda and t.is_contiguous() and tuple(t.shape) == shape and t.device == x.device
    if x.dim() != 2 or not ok(x, tuple(x.shape)) or x.shape[1] % 8 or x.shape[1] < 8:
        raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_residual_rmsnorm (x must be contiguous fp16 CUDA [M, K], K % 8 == 0)")
    M, K = x.shape
    if (residual is not None and not ok(residual, (M, K))) or not ok(gamma, (K,)):
        raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_residual_rmsnorm (residual [M, K] / gamma [K] fp16 on x's device)")
    if y_out is None:
        y_out = torch.empty_like(x)
    if h_out is None and want_h:
        h_out = torch.empty_like(x)
    if not ok(y_out, (M, K)) or (h_out is not None and not ok(h_out, (M, K))):
        raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_residual_rmsnorm (bad output tensor)")
    _check(lib.qlinear_residual_rmsnorm(ctypes.c_void_p(x.data_ptr()), ctypes.c_void_p(residual.data_ptr() if residual is not None else None),
                                        ctypes.c_void_p(gamma.data_ptr()), float(eps), float(gamma_offset),
                                        ctypes.c_void_p(h_out.data_ptr() if h_out is not None else None), ctypes.c_void_p(y_out.data_ptr()),
                                        M, K, x.device.index or 0, _stream_ptr(stream)), "qlinear_residual_rmsnorm")
    return h_out, y_out


def qlinear_rope_qkv(q, k, v, pos, cos, sin, B: int, S: int, h_q: int, h_kv: int, d_h: int, stream=None):
    """q fp16 CUDA [B*S, h_q*d_h], k, v [B*S, h_kv*d_h], pos int32 [B*S], cos / sin fp32 [n_pos, d_h/2]
    -> (q_out [B*h_kv, S*h_q/h_kv, d_h], k_out [B*h_kv, S, d_h], v_out [B*h_kv, S, d_h]): rotary embedding + layout change."""
    import torch
    T = B * S
    def ok(t, dtype, shape):
        return t.dtype == dtype and t.is_cuda and t.is_contiguous() and tuple(t.shape) == shape and t.device == q.device
    if h_kv < 1 or h_q % h_kv or d_h % 16 or not ok(q, torch.float16, (T, h_q * d_h)) or not ok(k, torch.float16, (T, h_kv * d_h)) \
            or not ok(v, torch.float16, (T, h_kv * d_h)) or not ok(pos, torch.int32, (T,)) or cos.dim() != 2 \
            or not ok(cos, torch.float32, (cos.shape[0], d_h // 2)) or not ok(sin, torch.float32, tuple(cos.shape)):
        raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_rope_qkv (shapes / dtypes: see the header)")
    g = h_q // h_kv
    q_out = torch.empty((B * h_kv, S * g, d_h), dtype=torch.float16, device=q.device)
    k_out = torch.empty((B * h_kv, S, d_h), dtype=torch.float16, device=q.device)
    v_out = torch.empty((B * h_kv, S, d_h), dtype=torch.float16, device=q.device)
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    _check(lib.qlinear_rope_qkv(p(q), p(k), p(v), p(pos), p(cos), p(sin), cos.shape[0], p(q_out), p(k_out), p(v_out), B, S, h_q, h_kv, d_h,
                                q.device.index or 0, _stream_ptr(stream)), "qlinear_rope_qkv")
    return q_out, k_out, v_out


class QLinear:
    """One quantised linear layer resident on a GPU: owns the packed device tensor and the handle."""

    def __init__(self, desc: Desc, packed, device=None):
        import torch
        self.desc = desc
        if isinstance(packed, np.ndarray):
            dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
            packed = torch.from_numpy(np.ascontiguousarray(packed, dtype=np.uint8)).to(dev)
        if not packed.is_cuda or packed.dtype != torch.uint8 or not packed.is_contiguous():
            raise QLinearError(QL_ERR_INVALID_ARG, "QLinear (packed must be a contiguous uint8 CUDA tensor)")
        if packed.numel() < qlinear_packed_size(desc):
            raise QLinearError(QL_ERR_INVALID_ARG, "QLinear (packed blob too small)")
        self.packed = packed                      # keeps the device memory alive
        self.device = packed.device
        h = ctypes.c_void_p()
        _check(lib.qlinear_create(ctypes.byref(desc.c()), ctypes.c_void_p(packed.data_ptr()),
                                  self.device.index or 0, ctypes.byref(h)), "qlinear_create")
        self._h = h

    @classmethod
    def from_weights(cls, q: np.ndarray, s: np.ndarray, bits: int, group: int = 0, device=None) -> "QLinear":
        desc = Desc(int(q.shape[0]), int(q.shape[1]), bits, group)
        return cls(desc, qlinear_pack(desc, q, s), device)

    def forward(self, x, out=None, stream=None):
        """x: fp16 CUDA tensor [M, K] -> y fp16 [M, N] (qlinear_forward on the current stream)."""
        import torch
        if x.dim() != 2 or x.shape[1] != self.desc.K or x.dtype != torch.float16 or not x.is_cuda or not x.is_contiguous():
            raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_forward (x must be contiguous fp16 CUDA [M, K])")
        M = x.shape[0]
        if out is None:
            out = torch.empty((M, self.desc.N), dtype=torch.float16, device=x.device)
        elif out.shape != (M, self.desc.N) or out.dtype != torch.float16 or not out.is_contiguous():
            raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_forward (bad out tensor)")
        self.forward_raw(x.data_ptr(), out.data_ptr(), M, stream)
        return out

    def forward_a8(self, x, out=None, stream=None):
        """The decode call with int8 activations quantised inside the kernel (qlinear_forward_a8), M <= 8."""
        import torch
        if x.dim() != 2 or x.shape[1] != self.desc.K or x.dtype != torch.float16 or not x.is_cuda or not x.is_contiguous():
            raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_forward_a8 (x must be contiguous fp16 CUDA [M, K])")
        M = x.shape[0]
        if out is None:
            out = torch.empty((M, self.desc.N), dtype=torch.float16, device=x.device)
        elif out.shape != (M, self.desc.N) or out.dtype != torch.float16 or not out.is_contiguous():
            raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_forward_a8 (bad out tensor)")
        _check(lib.qlinear_forward_a8(self._h, ctypes.c_void_p(x.data_ptr()), ctypes.c_void_p(out.data_ptr()), M, _stream_ptr(stream)),
               "qlinear_forward_a8")
        return out

    def forward_a8_raw(self, x_ptr: int, y_ptr: int, M: int, stream=None) -> None:
        _check(lib.qlinear_forward_a8(self._h, ctypes.c_void_p(x_ptr), ctypes.c_void_p(y_ptr), M, _stream_ptr(stream)), "qlinear_forward_a8")

    def forward_raw(self, x_ptr: int, y_ptr: int, M: int, stream=None) -> None:
        _check(lib.qlinear_forward(self._h, ctypes.c_void_p(x_ptr), ctypes.c_void_p(y_ptr), M, _stream_ptr(stream)),
               "qlinear_forward")

    def embed(self, ids, out=None, stream=None):
        """ids: int32 CUDA tensor [n] -> fp16 [n, K], the dequantised rows ids of the table (qlinear_embed)."""
        import torch
        if ids.dim() != 1 or ids.dtype != torch.int32 or not ids.is_cuda or not ids.is_contiguous():
            raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_embed (ids must be a contiguous int32 CUDA vector)")
        n = ids.shape[0]
        if out is None:
            out = torch.empty((n, self.desc.K), dtype=torch.float16, device=ids.device)
        elif out.shape != (n, self.desc.K) or out.dtype != torch.float16 or not out.is_contiguous():
            raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_embed (bad out tensor)")
        _check(lib.qlinear_embed(self._h, ctypes.c_void_p(ids.data_ptr()), n, ctypes.c_void_p(out.data_ptr()),
                                 _stream_ptr(stream)), "qlinear_embed")
        return out

    def path_for(self, M: int) -> int:
        return int(lib.qlinear_path_for(self._h, M))

    def debug_unpack(self, stream=None):
        import torch
        q = torch.empty((self.desc.N, self.desc.K), dtype=torch.int8, device=self.device)
        _check(lib.qlinear_debug_unpack_device(self._h, ctypes.c_void_p(q.data_ptr()), _stream_ptr(stream)),
               "qlinear_debug_unpack_device")
        return q

    def debug_expire_wait(self, stream=None) -> None:
        """Runs the kernels' bounded wait on a barrier nothing completes (about a second); see device_status."""
        _check(lib.qlinear_debug_expire_wait(self._h, _stream_ptr(stream)), "qlinear_debug_expire_wait")

    def debug_null_launch(self, grid: int = 1, block: int = 32, stream=None) -> None:
        """Launches a kernel that does nothing (what a dependent launch costs on this machine)."""
        _check(lib.qlinear_debug_null_launch(self._h, grid, block, _stream_ptr(stream)), "qlinear_debug_null_launch")

    def device_status(self):
        detail = ctypes.c_uint32(0)
        st = lib.qlinear_device_status(self._h, ctypes.byref(detail))
        return int(st), int(detail.value)

    def close(self) -> None:
        if getattr(self, "_h", None):
            lib.qlinear_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class KVCache:
    """One KV head's cache held as two int8 weight blobs (see include/qlinear.h, qlinear_kv_append): argument
    marshalling only -- the blobs start as the packed form of zero weights, every later byte is written by the library."""

    def __init__(self, cache_size: int, d_h: int, device="cuda:0"):
        import torch
        self.cache_size, self.d_h, self.length = cache_size, d_h, 0
        kd, vd = Desc(cache_size, d_h, 8, 0), Desc(d_h, cache_size, 8, 0)
        self.k = QLinear(kd, qlinear_pack(kd, np.zeros((cache_size, d_h), np.int8), np.zeros((cache_size, 1), np.float16)), device)
        self.v = QLinear(vd, qlinear_pack(vd, np.zeros((d_h, cache_size), np.int8), np.ones((d_h, 1), np.float16)), device)
        self.v_scale = torch.zeros((cache_size,), dtype=torch.float16, device=device)

    def append(self, k_new, v_new, stream=None):
        """k_new, v_new: fp16 CUDA [n_new, d_h], written to positions length .. length + n_new - 1."""
        import torch
        for t in (k_new, v_new):
            if t.dim() != 2 or t.shape[1] != self.d_h or t.dtype != torch.float16 or not t.is_cuda or not t.is_contiguous():
                raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_kv_append (k_new, v_new must be contiguous fp16 CUDA [n, d_h])")
        n = k_new.shape[0]
        if v_new.shape[0] != n:
            raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_kv_append (k_new and v_new differ in length)")
        _check(lib.qlinear_kv_append(self.k._h, self.v._h, ctypes.c_void_p(k_new.data_ptr()), ctypes.c_void_p(v_new.data_ptr()),
                                     ctypes.c_void_p(self.v_scale.data_ptr()), self.length, n, _stream_ptr(stream)), "qlinear_kv_append")
        self.length += n

    def scores(self, q_rows, stream=None):
        """q_rows fp16 [R, d_h] -> fp16 [R, cache_size] (positions beyond `length` score 0)."""
        import torch
        if q_rows.dim() != 2 or q_rows.shape[1] != self.d_h or q_rows.dtype != torch.float16 or not q_rows.is_cuda or not q_rows.is_contiguous():
            raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_kv_scores (q_rows must be contiguous fp16 CUDA [R, d_h])")
        out = torch.empty((q_rows.shape[0], self.cache_size), dtype=torch.float16, device=q_rows.device)
        _check(lib.qlinear_kv_scores(self.k._h, ctypes.c_void_p(q_rows.data_ptr()), ctypes.c_void_p(out.data_ptr()), q_rows.shape[0],
                                     _stream_ptr(stream)), "qlinear_kv_scores")
        return out

    def output(self, prob, stream=None):
        """prob fp16 [R, cache_size] -> fp16 [R, d_h]."""
        import torch
        if prob.dim() != 2 or prob.shape[1] != self.cache_size or prob.dtype != torch.float16 or not prob.is_cuda or not prob.is_contiguous():
            raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_kv_output (prob must be contiguous fp16 CUDA [R, cache_size])")
        tmp = torch.empty_like(prob)
        out = torch.empty((prob.shape[0], self.d_h), dtype=torch.float16, device=prob.device)
        _check(lib.qlinear_kv_output(self.v._h, ctypes.c_void_p(prob.data_ptr()), ctypes.c_void_p(self.v_scale.data_ptr()),
                                     ctypes.c_void_p(tmp.data_ptr()), ctypes.c_void_p(out.data_ptr()), prob.shape[0], _stream_ptr(stream)),
               "qlinear_kv_output")
        return out


class KVHeads:
    """The caches of all KV heads of one attention layer (n_heads <= 16 KVCache objects of equal shape), driven through
    the calls that serve every head in one launch (qlinear_kv_*_heads in include/qlinear.h): argument marshalling only."""

    def __init__(self, n_heads: int, cache_size: int, d_h: int, device="cuda:0"):
        self.heads = [KVCache(cache_size, d_h, device) for _ in range(n_heads)]
        self.n, self.cache_size, self.d_h, self.length = n_heads, cache_size, d_h, 0
        arr = ctypes.c_void_p * n_heads
        self._hk = arr(*[c.k._h for c in self.heads])
        self._hv = arr(*[c.v._h for c in self.heads])
        self._vs = arr(*[ctypes.c_void_p(c.v_scale.data_ptr()) for c in self.heads])

    def append_raw(self, k_ptr: int, v_ptr: int, head_stride: int, token_stride: int, n_new: int, stream=None) -> None:
        _check(lib.qlinear_kv_append_heads(self._hk, self._hv, self.n, ctypes.c_void_p(k_ptr), ctypes.c_void_p(v_ptr), head_stride, token_stride,
                                           self._vs, self.length, n_new, _stream_ptr(stream)), "qlinear_kv_append_heads")
        self.length += n_new
        for c in self.heads:
            c.length = self.length

    def append(self, k_new, v_new, stream=None):
        """k_new, v_new: fp16 CUDA [n_heads, n_new, d_h] (the k_out / v_out of qlinear_rope_qkv)."""
        import torch
        for t in (k_new, v_new):
            if t.dim() != 3 or t.shape[0] != self.n or t.shape[2] != self.d_h or t.dtype != torch.float16 or not t.is_cuda or not t.is_contiguous():
                raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_kv_append_heads (k_new, v_new must be contiguous fp16 CUDA [n_heads, n_new, d_h])")
        if k_new.shape != v_new.shape:
            raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_kv_append_heads (k_new and v_new differ in shape)")
        n_new = k_new.shape[1]
        self.append_raw(k_new.data_ptr(), v_new.data_ptr(), n_new * self.d_h, self.d_h, n_new, stream)

    def scores_raw(self, q_ptr: int, out_ptr: int, R: int, stream=None) -> None:
        _check(lib.qlinear_kv_scores_heads(self._hk, self.n, ctypes.c_void_p(q_ptr), ctypes.c_void_p(out_ptr), R, _stream_ptr(stream)),
               "qlinear_kv_scores_heads")

    def scores(self, q_rows, stream=None):
        """q_rows fp16 [n_heads, R, d_h] -> fp16 [n_heads, R, cache_size]."""
        import torch
        if q_rows.dim() != 3 or q_rows.shape[0] != self.n or q_rows.shape[2] != self.d_h or q_rows.dtype != torch.float16 or not q_rows.is_cuda or not q_rows.is_contiguous():
            raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_kv_scores_heads (q_rows must be contiguous fp16 CUDA [n_heads, R, d_h])")
        out = torch.empty((self.n, q_rows.shape[1], self.cache_size), dtype=torch.float16, device=q_rows.device)
        self.scores_raw(q_rows.data_ptr(), out.data_ptr(), q_rows.shape[1], stream)
        return out

    def output_raw(self, prob_ptr: int, out_ptr: int, R: int, stream=None) -> None:
        _check(lib.qlinear_kv_output_heads(self._hv, self.n, ctypes.c_void_p(prob_ptr), self._vs, ctypes.c_void_p(out_ptr), R, _stream_ptr(stream)),
               "qlinear_kv_output_heads")

    def output(self, prob, stream=None):
        """prob fp16 [n_heads, R, cache_size] -> fp16 [n_heads, R, d_h]."""
        import torch
        if prob.dim() != 3 or prob.shape[0] != self.n or prob.shape[2] != self.cache_size or prob.dtype != torch.float16 or not prob.is_cuda or not prob.is_contiguous():
            raise QLinearError(QL_ERR_INVALID_ARG, "qlinear_kv_output_heads (prob must be contiguous fp16 CUDA [n_heads, R, cache_size])")
        out = torch.empty((self.n, prob.shape[1], self.d_h), dtype=torch.float16, device=prob.device)
        self.output_raw(prob.data_ptr(), out.data_ptr(), prob.shape[1], stream)
        return out
