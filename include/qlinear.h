/*
 * qlinear -- weight-only quantised linear layer for NVIDIA B200 (sm_100a).
 *
 *     y[m,n] = fp16( sum_k x[m,k] * s[n, k/G] * q[n,k] )        fp32 accumulation
 *
 * W = s*q is N x K (output channels x input channels: the O x I weight
 * orientation of the paper's Section 3.1), q are int8 or int4 integers, s are
 * fp16 scales (one per output channel, or one per group of G consecutive k),
 * x is M x K fp16 row-major, y is M x N fp16 row-major.
 *
 * The calls follow the life cycle the paper describes for operators with
 * external weights: the weights are converted once, at initialisation, into the
 * memory layout the kernels read (Section 3.4, "weights conversion"; Section
 * 3.1, weight layouts); every forward call then picks the kernel for its stage
 * from the shape of the input (Section 3.7: a memory-bound fully-connected
 * kernel for decode, a compute-bound matrix-multiply kernel for prefill), both
 * reading the same resident weights.  Quantisation schemes: Section 4.2 (q8 =
 * int8 per channel; 8/4/4 = int8 attention, int4 feed-forward/embedding).
 *
 * Threads and streams.  A handle is immutable after qlinear_create, so any
 * number of host threads may call the forward functions on it.  The kernels of
 * two calls may overlap on the GPU (different streams) unless one of them is a
 * prefill call the library splits along K (a layer, or group of layers, with
 * fewer 256 x 256 output tiles than half the SM count): those calls meet in one
 * per-device scratch area and must be ordered against each other by the caller
 * (same stream, or events).  qlinear_decode_static has its own rule, stated
 * there.
 *
 * Device memory.  The caller owns the packed weights, x and y.  The library
 * owns one small set of buffers PER DEVICE, allocated when the first handle on
 * that device is created and kept until the process exits: 40 MB of scratch
 * (fp32 partial tiles of the K-split prefill case, the int8 activations of the
 * integer prefill form, the two projections of the unfused gating route) plus
 * arrival counters, and one word of pinned host memory through which kernels
 * report an expired wait.  A handle
 * itself owns host memory only.
 *
 * Environment.  Every QLINEAR_* variable is read once per process, at the
 * first call that creates a handle; later changes are not seen.
 *
 * No function falls back to the CPU: without an sm_100 device qlinear_create
 * fails with QL_ERR_ARCH.
 */
#ifndef QLINEAR_H
#define QLINEAR_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct qlinear_s* qlinear_t;

typedef enum {
    QL_OK = 0,
    QL_ERR_INVALID_ARG = 1,     /* null pointer, misaligned pointer, bad size, value out of range   */
    QL_ERR_UNSUPPORTED = 2,     /* shape / bits / group combination the library does not implement   */
    QL_ERR_ALLOC = 3,           /* host allocation failed                                            */
    QL_ERR_CUDA = 4,            /* a CUDA runtime / driver call failed (launch errors included)      */
    QL_ERR_DEVICE_TIMEOUT = 5,  /* a bounded wait inside a kernel expired; the output is invalid     */
    QL_ERR_ARCH = 6             /* the device is not compute capability 10.x                         */
} ql_status;

/* Shape and quantisation scheme of one layer (Section 4.2).
 *   N, K   output / input channels.  K must be a multiple of 32, N a multiple of 8.
 *   bits   8 or 4.
 *   group  0 = one scale per output channel; for bits == 4 also 32, 64 or 128 = scales per group of
 *          that many consecutive k (must divide K).  bits == 8 supports group == 0 only. */
typedef struct {
    int32_t N, K, bits, group;
} qlinear_desc;

/* Which kernel a forward call with M tokens runs (Section 3.7, stage-aware selection). */
typedef enum { QL_PATH_GEMV = 1, QL_PATH_GEMM = 2 } ql_path;

/* Bytes of the packed blob for this layer; 0 if the descriptor is invalid or unsupported. */
size_t qlinear_packed_size(const qlinear_desc* desc);

/* Weights conversion (Section 3.4; layouts: Section 3.1).  HOST function, pure, calls no CUDA.
 *   q        host, N*K int8, row-major, one integer per byte: [-128,127] for bits 8, [-8,7] for bits 4.
 *   s_fp16   host, fp16 bit patterns, row-major [N] (group 0) or [N, K/group].
 *   packed   host, out, packed_bytes >= qlinear_packed_size(desc).  Opaque, position-independent,
 *            starts with a versioned header; the caller copies it to device memory unchanged.
 * Errors: QL_ERR_INVALID_ARG (null, short buffer, integer outside the range of `bits`),
 *         QL_ERR_UNSUPPORTED (descriptor). Nothing is written on error. */
ql_status qlinear_pack(const qlinear_desc* desc, const int8_t* q, const uint16_t* s_fp16,
                       void* packed, size_t packed_bytes);

/* Host inverse of qlinear_pack (for tests and for re-exporting weights): fills q_out [N*K] and
 * s_out [N] or [N, K/group].  Checks the header against desc (QL_ERR_INVALID_ARG on mismatch). */
ql_status qlinear_unpack(const qlinear_desc* desc, const void* packed, int8_t* q_out, uint16_t* s_out);

/* Binds a packed blob that already lives in DEVICE memory to a handle (Section 3.4: the converted
 * weights stay resident in GPU memory and serve both stages, Section 3.7).
 *   packed_dev  device pointer, 256-byte aligned, qlinear_packed_size(desc) bytes, owned by the caller,
 *               must stay alive and unchanged until qlinear_destroy (the KV-cache calls below are the one exception:
 *               they write into their blobs).
 *   device      CUDA device ordinal that owns packed_dev.
 * The handle owns host memory only (shape, kernel plans); the first handle on a device also creates that
 * device's shared buffers (see "Device memory" above), so the first create on a device should come before
 * any stream capture.
 * Errors: QL_ERR_INVALID_ARG, QL_ERR_UNSUPPORTED (descriptor, or a shape no decode plan fits), QL_ERR_ARCH
 * (device is not sm_100), QL_ERR_CUDA, QL_ERR_ALLOC. */
ql_status qlinear_create(const qlinear_desc* desc, const void* packed_dev, int device, qlinear_t* out);

/* y = x . W^T for M >= 1 tokens, enqueued on `cuda_stream` (a cudaStream_t; NULL = default stream).
 *   x_dev  device, fp16 [M, K] row-major contiguous, 16-byte aligned, read-only during the call.
 *   y_dev  device, fp16 [M, N] row-major contiguous, 16-byte aligned, must not overlap x_dev.
 * Asynchronous: returns after the launch; allocates nothing; never synchronises.  M <= 8 runs the
 * decode kernel, larger M the prefill kernel (Section 3.7); see qlinear_path_for.
 * Errors: QL_ERR_INVALID_ARG (null / misaligned pointers, M < 1, M*K or M*N beyond 2^31-1 elements),
 * QL_ERR_CUDA (launch failure, reported synchronously), QL_ERR_DEVICE_TIMEOUT (an earlier kernel of this
 * library on the handle's DEVICE gave up a bounded wait: its output is invalid; nothing is launched, and every
 * forward call on that device keeps returning this code until qlinear_device_status has cleared it.  The
 * code reaches the host through pinned memory, so this check costs no synchronisation). */
ql_status qlinear_forward(qlinear_t h, const void* x_dev, void* y_dev, int32_t M, void* cuda_stream);

/* The same result as n calls of qlinear_forward with one x: ys_dev[i] = x . W_i^T for the n layers hs[i]
 * (1 <= n <= 4), which must live on one device and agree in K, bits and group (q/k/v projections; gate
 * and up projections).  For M <= 8 all n layers run in ONE decode kernel launch: their output channels
 * are numbered one after the other and spread over the grid together, so short layers do not each pay
 * a launch of their own (the paper's operator fusion, Section 3 "Operator Fusion", merges kernels for
 * the same reason: launch overhead and memory-bound work).  Every output is bit-identical to what
 * qlinear_forward gives for that layer only if the K split chosen for the group equals the layer's own;
 * it always meets the same tolerance, and is run-to-run deterministic.  For larger M the layers share
 * one launch of the prefill kernel when every layer qualifies for its
 * CTA-pair form (a multiple of 256 output channels after padding to 128); the tiles of all layers then
 * fill the persistent grid together.  Otherwise they run one after the other.
 *   hs      host array of n handles; ys_dev host array of n device pointers (fp16 [M, N_i], 16-byte
 *           aligned, not overlapping x_dev or one another); x_dev as in qlinear_forward.
 * Asynchronous, allocates nothing; the plan of the group is made per call and nothing is written to a handle.
 * Errors: as qlinear_forward; QL_ERR_INVALID_ARG also for n outside 1..4 or layers that do not agree. */
ql_status qlinear_forward_group(const qlinear_t* hs, int32_t n, const void* x_dev, void* const* ys_dev,
                                int32_t M, void* cuda_stream);

/* Layers with DIFFERENT inputs in one launch: ys[i] = xs[i] . W_i^T for i < n (1 <= n <= 8), all with the same M.  The
 * case in mind is the attention products over the KV cache held as weights (paper Section 3.8): every KV head has its
 * own cache handle and its own query rows, and a launch per head and product is launch-bound.  Same requirements on the
 * handles as qlinear_forward_group (one device, equal K, bits and group).  For M <= 8 and K a whole number of chunks the
 * call is one decode launch (more than 4 layers: int8 layers only); otherwise it is n calls of qlinear_forward, in
 * order.  Pointers as for qlinear_forward. */
ql_status qlinear_forward_batch(const qlinear_t* handles, int32_t n, const void* const* xs_dev, void* const* ys_dev, int32_t M, void* cuda_stream);

/* Activation of the gate branch in qlinear_forward_gated. */
typedef enum { QL_ACT_IDENTITY = 0, QL_ACT_SILU = 1, QL_ACT_GELU_TANH = 2 } ql_act;

/* Fused gating of the feed-forward block (Section 3.6, "Operator Fusion": element-wise operators of two
 * branches fused with a fully connected operator):
 *     y[m,n] = fp16( act(gate[m,n]) * up[m,n] ),   gate = x . W_gate^T,  up = x . W_up^T   (both in fp32)
 * with act = identity, SiLU g / (1 + exp(-g)) (the Llama family) or the tanh form of GELU (the Gemma family);
 * the paper names no activation.  Neither projection is written to memory: for M <= 8 one decode launch
 * holds both branches of every output channel in the same CTA; for M > 128 (and layers of a multiple of 256
 * channels after padding to 128) the CTA-pair prefill kernel keeps the two projections of a tile in its two
 * tensor-memory accumulators and the epilogue writes only their product, which halves the write-back.
 * Shapes outside those two cases (9 <= M <= 128, other channel counts, K not a multiple of the decode chunk)
 * run the two projections into the device's shared scratch and a small element-wise kernel after them: same
 * result, no saving; such calls must be ordered against K-split prefill calls like those among themselves.
 *   h_gate, h_up  two layers on one device with the same N, K, bits and group
 *   x_dev, y_dev  as in qlinear_forward; y_dev is fp16 [M, N]
 * Asynchronous, allocates nothing.  Errors: as qlinear_forward; QL_ERR_INVALID_ARG also for layers that do
 * not agree or an unknown activation; QL_ERR_UNSUPPORTED if the unfused case needs more scratch than the
 * device's shared buffer holds (2 * M * N fp16 beyond about 19 MB). */
ql_status qlinear_forward_gated(qlinear_t h_gate, qlinear_t h_up, const void* x_dev, void* y_dev, int32_t M,
                                int32_t act, void* cuda_stream);

/* The linear layer with int8 ACTIVATIONS, decode stage (Section 3.7, "Stage-Aware Optimizations": in the
 * memory-bound decode stage the quantisation of the input activations is integrated into the fully-connected
 * kernel, the products with the pre-quantised weights use integer instructions, and the dequantisation is
 * applied to the output).  Per token m:  amax = max_k |x[m,k]|,  xq = round-half-to-even(x * (127 / amax))
 * clamped to [-127, 127] (IEEE fp32, one rounding per operation; a row of zeros quantises to zeros with scale 1),
 *     y[m,n] = fp16( (amax / 127) * sum_g s[n,g] * sum_{k in g} xq[m,k] * q[n,k] )
 * with the inner sums exact (integer tensor-core instructions).  The paper gives neither the granularity of the
 * activation scale nor the rounding; one scale per token, symmetric, is the reading taken here.
 *   h, x_dev, y_dev, cuda_stream as in qlinear_forward.
 * M <= 8, every scheme: one decode launch with the quantisation inside it.
 * M > 128, the paper's own per-channel schemes (group 0: q8 and per-channel int4), K a multiple of 128 and a
 * multiple of 256 output channels after padding to 128: the prefill form of the same section -- the quantisation
 * kernel (qlinear_quantize_activations, into the device's shared scratch), then the CTA-pair prefill kernel in its
 * integer form: the stored weight integers go to the tensor cores unconverted (tcgen05.mma kind::i8, u8 x s8 -> s32
 * in tensor memory), and the epilogue removes the storage offset and applies both scales.  Such calls use the shared
 * scratch and must be ordered against each other and against K-split prefill calls.
 * Anything else (grouped scales with M > 8, 9 <= M <= 128, other shapes): QL_ERR_UNSUPPORTED.
 * Asynchronous, allocates nothing.  The result differs from qlinear_forward's by the quantisation noise of x
 * (about 1 % relative for Gaussian x); it equals it to fp32 round-off when x already lies on the int8 grid. */
ql_status qlinear_forward_a8(qlinear_t h, const void* x_dev, void* y_dev, int32_t M, void* cuda_stream);

/* The activation-quantisation kernel of the prefill stage (Section 3.7): x_dev fp16 [M, K] -> xq_dev int8 [M, K]
 * and scale_dev fp32 [M], by the per-token steps stated at qlinear_forward_a8.  K a multiple of 32; x_dev and
 * xq_dev 16-byte aligned; all three buffers on `device`, caller-owned.  Asynchronous on `cuda_stream`.
 * Errors: QL_ERR_INVALID_ARG, QL_ERR_CUDA. */
ql_status qlinear_quantize_activations(const void* x_dev, int8_t* xq_dev, float* scale_dev, int32_t M, int32_t K,
                                       int device, void* cuda_stream);

/* The KV cache held as weights (Section 3.8, "GPU-Optimized KV Cache Layout"): the K cache is a layer with
 * O = cache positions and I = head dimension d_h (it stands for K^T in Q K^T), the V cache a layer with O = d_h and
 * I = cache positions, so that both attention products are calls of the linear kernels and the second comes out as
 * [query rows, d_h], the layout the paper's QKV transformation wants (rows = S * h_q / h_kv per KV head).
 * The paper does not say how its cache is stored; here both caches are int8 blobs (Section 4.2's 8-bit format)
 * with one scale per cached TOKEN:  s = fp16(max|v| / 127),  q = round-half-to-even(v / s) clamped to +-127, IEEE
 * fp32 operations (a vector whose scale rounds to zero is stored as zeros with scale 1).
 *
 * A cache pair is two ordinary handles over caller-owned blobs that the caller packed from ZERO weights:
 *   h_k  desc {N = cache positions, K = d_h, bits 8, group 0}, channel scales 0 (an empty position scores 0)
 *   h_v  desc {N = d_h, K = cache positions, bits 8, group 0}, channel scales 1
 * qlinear_kv_append quantises n_new key and value vectors (k_new_dev, v_new_dev: fp16 [n_new, d_h]) and writes them
 * to positions pos .. pos + n_new - 1: the key integers and their scales into the K blob (a token is an output
 * channel there), the value integers into the V blob and their scales into v_scale_dev (fp16 [cache positions],
 * caller-owned): in the V cache a token is an INPUT channel, so its scale is folded into the probabilities instead,
 *     out[r, d] = sum_t (prob[r, t] * s_v[t]) * q_v[t, d].
 * These are the only calls that write to a blob; they must be ordered against forward calls on the same handles.
 * qlinear_kv_scores:  scores_dev [R, cache positions] = q_rows_dev [R, d_h] . K^T   (= qlinear_forward on h_k).
 * qlinear_kv_output:  out_dev [R, d_h] from prob_dev fp16 [R, cache positions]; tmp_dev is caller-owned scratch of
 *                     the same shape as prob_dev (it receives prob * s_v rounded to fp16 where that product needs a
 *                     pass of its own: R > 8, or a cache length that is not a multiple of 32).
 * k_new_dev, v_new_dev, v_scale_dev, prob_dev, tmp_dev, out_dev: 16-byte aligned.
 * Masking and the softmax between the two are the caller's.  Asynchronous, allocate nothing.
 * Errors: QL_ERR_INVALID_ARG (null / misaligned pointers, handles that are not an int8 cache pair of matching
 * shape, pos + n_new beyond the cache, d_h > 1024), otherwise as qlinear_forward. */
ql_status qlinear_kv_append(qlinear_t h_k, qlinear_t h_v, const void* k_new_dev, const void* v_new_dev, void* v_scale_dev,
                            int32_t pos, int32_t n_new, void* cuda_stream);
ql_status qlinear_kv_scores(qlinear_t h_k, const void* q_rows_dev, void* scores_dev, int32_t R, void* cuda_stream);
ql_status qlinear_kv_output(qlinear_t h_v, const void* prob_dev, const void* v_scale_dev, void* tmp_dev, void* out_dev,
                            int32_t R, void* cuda_stream);

/* The same three steps for ALL KV heads of an attention layer at once (n_heads <= 16 cache pairs of equal shape, arrays
 * of handles h_k[i], h_v[i] and of their scale arrays v_scale_dev[i], all host arrays of device pointers): one launch per
 * step for up to 8 heads instead of one (or two) per head -- at decode every one of these products is a few hundred
 * KB and bound by the launch, not by the bytes.  The buffers have the layout the rotary / layout kernel writes:
 *   qlinear_kv_append_heads: element (head i, new token t, dimension j) of k_new_dev / v_new_dev at
 *                            i * head_stride + t * token_stride + j (strides in elements, multiples of 8;
 *                            k_out / v_out of qlinear_rope_qkv: head_stride = S * d_h, token_stride = d_h)
 *   qlinear_kv_scores_heads: q_rows_dev fp16 [n_heads, R, d_h] -> scores_dev fp16 [n_heads, R, cache positions]
 *   qlinear_kv_output_heads: prob_dev fp16 [n_heads, R, cache positions] -> out_dev fp16 [n_heads, R, d_h]; R <= 8 and
 *                            a cache length that is a multiple of 32: the product prob * s_v (rounded to fp16, as in
 *                            qlinear_kv_output) is formed inside the decode kernel on the way to the tensor core, so
 *                            there is no scratch buffer and no pass of its own.  Other shapes: QL_ERR_UNSUPPORTED
 *                            (use qlinear_kv_output per head).
 * All device pointers 16-byte aligned, R * d_h and R * cache positions multiples of 8.  Results are bit-identical to
 * the per-head calls wherever those take K undivided (d_h <= 128) and meet the same tolerance everywhere.  Score
 * products of more than four row super-blocks per SM (long caches; R <= 8, d_h = 64, 128 or 256) run on a persistent
 * kernel of their own (csrc/gemv_rows.cuh).  Asynchronous, allocate nothing.  Errors as above. */
ql_status qlinear_kv_append_heads(const qlinear_t* h_k, const qlinear_t* h_v, int32_t n_heads, const void* k_new_dev,
                                  const void* v_new_dev, int64_t head_stride, int64_t token_stride, void* const* v_scale_dev,
                                  int32_t pos, int32_t n_new, void* cuda_stream);
ql_status qlinear_kv_scores_heads(const qlinear_t* h_k, int32_t n_heads, const void* q_rows_dev, void* scores_dev, int32_t R,
                                  void* cuda_stream);
ql_status qlinear_kv_output_heads(const qlinear_t* h_v, int32_t n_heads, const void* prob_dev, const void* const* v_scale_dev,
                                  void* out_dev, int32_t R, void* cuda_stream);

/* Embedding lookup from a quantised table (Section 4.2: the mixed 8/4/4 scheme keeps the embedding table
 * in int4 like the feed-forward weights).  The handle's layer is read as a table of N rows of K values:
 *   y_dev[t, k] = fp16( s[ids[t], k / group] * q[ids[t], k] )      for t in [0, n), k in [0, K)
 * the correctly rounded product (one rounding), i.e. the dequantised row, bit for bit.  The same blob can
 * serve as LM head through qlinear_forward.
 *   ids_dev  device, int32 [n], 4-byte aligned; a row number outside [0, N) gives a row of zeros
 *   y_dev    device, fp16 [n, K] row-major contiguous, 16-byte aligned
 * Asynchronous on `cuda_stream`, allocates nothing.  n == 0 is a no-op (the pointers are not looked at).
 * Errors: QL_ERR_INVALID_ARG (null / misaligned pointers, n < 0), QL_ERR_CUDA (launch failure). */
ql_status qlinear_embed(qlinear_t h, const int32_t* ids_dev, int32_t n, void* y_dev, void* cuda_stream);

/* Residual connection + RMS normalisation: the operator that PRODUCES the linear layer's input (paper Section 3.6,
 * second fusion example: the residual connection and the element-wise operations merged with the RMS normalisation
 * operator).  Per token m (row of K values):
 *     h[m,k] = x[m,k] + residual[m,k]                               (fp32; residual may be NULL: h = x)
 *     y[m,k] = h[m,k] / sqrt(mean_k h[m,k]^2 + eps) * (gamma_offset + gamma[k])
 * h_out (may be NULL) receives fp16(h), the residual stream of the next block; y_out receives fp16(y).  The paper gives
 * no formulas; these are the ones of the models it runs (gamma_offset = 0: Llama; 1: Gemma, which stores gamma - 1).
 * x_dev, residual_dev, h_out_dev, y_out_dev: fp16 [M, K] row-major, device memory of `device`, 16-byte aligned;
 * gamma_dev: fp16 [K].  K a multiple of 8; M >= 0 (0: nothing is done); eps >= 0.  h_out_dev may be x_dev or
 * residual_dev (in place), y_out_dev may be x_dev; h_out_dev and y_out_dev must differ.  No handle, no library-owned
 * memory; asynchronous on cuda_stream.  Returns QL_ERR_INVALID_ARG for null / misaligned pointers or a bad shape,
 * QL_ERR_CUDA if the launch fails. */
/* Rotary embedding combined with the layout transformation of the Q, K and V projections (paper Section 3.6: the
 * hand-written kernel of the attention block; query from (B, 1, S, h_q * d_h) to (B * h_kv, S * h_q / h_kv, d_h)).
 * Inputs (what the q / k / v projections wrote, token t = b * S + s): q_dev fp16 [B*S, h_q*d_h], k_dev and v_dev fp16
 * [B*S, h_kv*d_h]; pos_dev int32 [B*S], the position of every token; cos_dev / sin_dev fp32 [n_pos, d_h/2], the angle
 * tables (row = position), so that any frequency schedule can be used.  The paper fixes neither the rotary convention
 * nor the order inside the merged query dimension; the readings taken: rotate-half pairs (element i < d_h/2 with
 * element i + d_h/2:  out_i = x_i cos - x_{i+d/2} sin,  out_{i+d/2} = x_{i+d/2} cos + x_i sin), and, with g = h_q / h_kv,
 *     q_out[b*h_kv + hk, s*g + j, :] = rot(q[t, (hk*g + j)*d_h ...]),   k_out[b*h_kv + hk, s, :] = rot(k[t, hk*d_h ...]),
 *     v_out[b*h_kv + hk, s, :] = v[t, hk*d_h ...]   (not rotated),
 * i.e. one contiguous [rows, d_h] block per KV head: the rows qlinear_kv_append and qlinear_kv_scores take.
 * q_out_dev fp16 [B*h_kv, S*g, d_h], k_out_dev and v_out_dev fp16 [B*h_kv, S, d_h]; all pointers device memory of
 * `device`, 16-byte aligned (pos 4); outputs must not be the inputs.  h_q a multiple of h_kv, d_h a multiple of 16;
 * positions must lie in [0, n_pos) (the kernel clamps them rather than read outside the tables).  No handle, no
 * library-owned memory; asynchronous on cuda_stream.  QL_ERR_INVALID_ARG for null / misaligned pointers or bad shapes. */
ql_status qlinear_rope_qkv(const void* q_dev, const void* k_dev, const void* v_dev, const int32_t* pos_dev, const float* cos_dev,
                           const float* sin_dev, int32_t n_pos, void* q_out_dev, void* k_out_dev, void* v_out_dev, int32_t B, int32_t S,
                           int32_t h_q, int32_t h_kv, int32_t d_h, int32_t device, void* cuda_stream);

ql_status qlinear_residual_rmsnorm(const void* x_dev, const void* residual_dev, const void* gamma_dev, float eps, float gamma_offset,
                                   void* h_out_dev, void* y_out_dev, int32_t M, int32_t K, int32_t device, void* cuda_stream);

/* The kernel qlinear_forward uses for M tokens on this handle (0 if h is NULL or M < 1). */
int32_t qlinear_path_for(qlinear_t h, int32_t M);

/* Runs, on the device, the same unpack routine the forward kernels use and writes the integers
 * q_dev_out [N*K] int8 row-major (device memory, caller-owned).  Used to prove that the device sees
 * exactly the integers that were packed.  Asynchronous on `cuda_stream`. */
ql_status qlinear_debug_unpack_device(qlinear_t h, int8_t* q_dev_out, void* cuda_stream);

/* Test aid for the failure path: launches a one-warp kernel that runs the kernels' bounded wait on a
 * barrier nothing ever completes.  The wait gives up after about a second, records its code (0x9A0) and
 * the kernel returns normally; the next qlinear_device_status reports QL_ERR_DEVICE_TIMEOUT with that code
 * and the device stays usable.  Asynchronous on `cuda_stream`. */
ql_status qlinear_debug_expire_wait(qlinear_t h, void* cuda_stream);

/* Measurement aid: launches, the way every kernel of this library is launched (programmatic dependent launch unless
 * the environment switched it off), a kernel of `grid` blocks of `block` threads that does nothing.  Chained in a
 * stream or a CUDA graph it gives the cost of a dependent launch on the machine, the floor under every small layer.
 * Asynchronous on `cuda_stream`. */
ql_status qlinear_debug_null_launch(qlinear_t h, int32_t grid, int32_t block, void* cuda_stream);

/* Synchronises the handle's device and reports whether any kernel of this library on that device gave up a
 * bounded wait (QL_ERR_DEVICE_TIMEOUT), else QL_OK.  `detail`, if not NULL, receives a code that
 * identifies the wait.  Clears the condition (the flag the forward calls look at, and the arrival counters
 * an abandoned K-split launch may have left behind), after which the device's handles work again.
 * A wait only counts time after the kernel's own stream dependency has resolved: a long-running earlier
 * kernel in the stream does not expire the waits of the kernel queued behind it. */
ql_status qlinear_device_status(qlinear_t h, uint32_t* detail);

/* Decode call for callers that cannot allocate device memory.  (The paper has no counterpart: this is
 * a deployment variant of the decode stage of Section 3.7, not a new operation.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a latency-critical serving loop
 * whose memory was carved up front, under a memory pool that owns every byte of the device, or in a
 * plugin that is only handed input and output buffers.  qlinear_create allocates a small device scratch
 * for the streaming decode kernel; this call takes no handle and allocates nothing, neither on the device
 * nor through any library: the kernel's partial-sum slots and arrival counters live in one static device
 * array of 2,752,512 bytes (2.5 MiB of slots for at most 320 CTAs + 128 KiB of counters) that every GPU
 * loading the library holds until the process exits.
 *
 *   desc, packed_dev   as for qlinear_create (the blob already in device memory, 256-byte aligned)
 *   x_dev, y_dev, M    as for qlinear_forward, with 1 <= M <= 8 (decode only)
 *   device             ordinal that owns the buffers; cuda_stream as for qlinear_forward
 *
 * Computes exactly what qlinear_forward computes for M <= 8 (same packed weights, same tolerance; the
 * summation order differs from the default decode kernel, so results may differ in the last bit).
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress) and sets a kernel
 * attribute; make that first call outside any stream capture.  Every call shares the one array, which keeps
 * the previous call's contents: the counters are cleared on the stream before each launch, the slots are
 * overwritten before they are read.  Two calls that overlap on the GPU (different streams, or different
 * host threads without stream ordering between them) race on it -- serialise them.
 * Errors: QL_ERR_INVALID_ARG (null / misaligned pointers, M outside 1..8), QL_ERR_UNSUPPORTED (descriptor
 * not supported, more than 4096 row super-blocks i.e. N > 524288, or int4 with K not a multiple of 64),
 * QL_ERR_ARCH, QL_ERR_CUDA. */
ql_status qlinear_decode_static(const qlinear_desc* desc, const void* packed_dev, const void* x_dev, void* y_dev,
                                int32_t M, int device, void* cuda_stream);

/* Frees the handle's host memory.  Does not touch the packed blob or the device's shared buffers.  NULL is allowed. */
ql_status qlinear_destroy(qlinear_t h);

/* Static, NUL-terminated description of a status code. */
const char* qlinear_status_string(ql_status s);

/* Library ABI version (major << 16 | minor). */
uint32_t qlinear_version(void);

/* Test aids (no paper counterpart).  qlinear_debug_plan writes up to n_out of the decode plan's numbers for M
 * tokens {kernel (1 cluster, 3 streaming), grid CTAs, CTAs per cluster, K slices per CTA, chunks per slice,
 * 1000 x (work of the busiest SM / mean), row-blocks, chunks along K} and returns how many it wrote (0 on bad
 * arguments).  qlinear_debug_config_reads returns how many times the QLINEAR_* environment has been read by
 * this process (1 after the first call, for good). */
int32_t qlinear_debug_plan(qlinear_t h, int32_t M, int32_t* out, int32_t n_out);
uint32_t qlinear_debug_config_reads(void);

#ifdef __cplusplus
}
#endif
#endif /* QLINEAR_H */
