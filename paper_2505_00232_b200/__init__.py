"""B200-native weight-only quantised linear layer (decode GEMV + prefill GEMM) behind a C ABI."""
from .binding import (Desc, QLinear, KVCache, KVHeads, QLinearError, qlinear_decode_static, qlinear_forward_group, qlinear_forward_group_raw, qlinear_forward_batch, qlinear_forward_batch_raw, kv_scores_batch, qlinear_forward_gated, qlinear_forward_gated_raw, qlinear_quantize_activations, qlinear_residual_rmsnorm, qlinear_rope_qkv, qlinear_pack, qlinear_packed_size, qlinear_unpack,  # noqa: F401
                      status_string, lib, LIB_PATH, EXPORTS, QL_PATH_GEMM, QL_PATH_GEMV,
                      QL_OK, QL_ERR_INVALID_ARG, QL_ERR_UNSUPPORTED, QL_ERR_ALLOC, QL_ERR_CUDA, QL_ERR_DEVICE_TIMEOUT, QL_ERR_ARCH)
