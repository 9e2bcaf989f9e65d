// The KV cache held as weights (paper Section 3.8, "GPU-Optimized KV Cache Layout"): the K cache is a layer with
// O = cache positions and I = head dimension (it stands for K^T in Q K^T), the V cache a layer with O = head
// dimension and I = cache positions, so that both attention products are calls of the linear kernels and the
// second one comes out as [query rows, d_h].  Both caches are int8 blobs in the layout of layout.h.
//
// This kernel appends tokens: it quantises each new key and value vector with one scale per TOKEN,
//     s = fp16(amax / 127)  (fp32 division, rounded to fp16),   q = round-half-even(v / s) clamped to [-127, 127]
// (a vector whose scale rounds to zero is stored as zeros with scale 1), and writes the integers to the places the
// layout gives them.  For K a token is an output channel, so s is that channel's scale in the blob.  For V a token
// is an INPUT channel; its scale cannot live in the blob (a channel scale there would span all tokens), so it goes
// to a side array and is folded into the attention probabilities before the product:
//     out[r, d] = sum_t (prob[r, t] * s_v[t]) * q_v[t, d].
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "layout.h"

namespace ql {

// Byte offset, from the start of the body, of int8 weight (row, k) of a layer with n_kc chunks of 32.
__host__ __device__ __forceinline__ int64_t int8_weight_offset(int row, int k, int n_kc)
{
    const int rsb = row >> 7, rb = (row & 127) >> 4, g = row & 7, upper = (row >> 3) & 1;
    const int kc = k >> 5, c = (k & 31) >> 3, r8 = k & 7;
    const int w = ((r8 >> 2) << 1) | ((r8 >> 1) & 1), b = (r8 & 1) | (upper << 1);
    return ((int64_t)rsb * n_kc + kc) * kWeightBlockBytes + rb * 512 + ((g << 2) | c) * 16 + w * 4 + b;
}

constexpr int kKvMaxHeads = 16;          // KV heads (cache pairs of equal shape) that one append launch serves

struct KvAppendParams {
    // per head (blockIdx.y)
    uint8_t* k_body[kKvMaxHeads];        // K cache: N = cache positions, K = d_h
    __half* k_scales[kKvMaxHeads];       // its per-channel (= per-token) scales
    uint8_t* v_body[kKvMaxHeads];        // V cache: N = d_h, K = cache positions
    __half* v_scale[kKvMaxHeads];        // [cache positions] per-token scales of V (side array)
    const __half* k_new;                 // element (head h, new token i, dimension j) at h * head_stride + i * token_stride + j
    const __half* v_new;
    int64_t head_stride, token_stride;
    int32_t d_h, cache_size, pos, n_new;
    int32_t k_n_kc, v_n_kc;
};

// One CTA (128 threads) per new token and head; d_h <= 1024.
__global__ void __launch_bounds__(128) kv_append_kernel(const KvAppendParams p)
{
    __shared__ float wmax[2][4];
    __shared__ float sc[2];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int i = blockIdx.x, t = p.pos + i, hd = blockIdx.y;
    const int64_t src = hd * p.head_stride + i * p.token_stride;
    const __half* kv[2] = {p.k_new + src, p.v_new + src};
    float am[2] = {0.f, 0.f};
    for (int j = threadIdx.x; j < p.d_h; j += 128) {
        am[0] = fmaxf(am[0], fabsf(__half2float(kv[0][j])));
        am[1] = fmaxf(am[1], fabsf(__half2float(kv[1][j])));
    }
#pragma unroll
    for (int s = 0; s < 2; ++s) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) am[s] = fmaxf(am[s], __shfl_xor_sync(0xffffffffu, am[s], o));
        if ((threadIdx.x & 31) == 0) wmax[s][threadIdx.x >> 5] = am[s];
    }
    __syncthreads();
    if (threadIdx.x < 2) {
        const int s = threadIdx.x;
        const float a = fmaxf(fmaxf(wmax[s][0], wmax[s][1]), fmaxf(wmax[s][2], wmax[s][3]));
        const __half h0 = __float2half_rn(__fdiv_rn(a, 127.f));
        const bool dead = __half2float(h0) == 0.f;                       // a zero vector, or a scale below fp16's range
        sc[s] = dead ? 0.f : __half2float(h0);                           // 0 marks "store zeros"
        const __half h = dead ? __float2half_rn(1.f) : h0;
        if (s == 0) p.k_scales[hd][t] = h; else p.v_scale[hd][t] = h;
    }
    __syncthreads();
    for (int j = threadIdx.x; j < p.d_h; j += 128) {
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            int q = 0;
            if (sc[s] != 0.f) q = max(-127, min(127, __float2int_rn(__fdiv_rn(__half2float(kv[s][j]), sc[s]))));
            const uint8_t stored = (uint8_t)(q + 128);
            if (s == 0) p.k_body[hd][int8_weight_offset(t, j, p.k_n_kc)] = stored;  // K: row = token, k = dimension
            else p.v_body[hd][int8_weight_offset(j, t, p.v_n_kc)] = stored;         // V: row = dimension, k = token
        }
    }
}

// x'[r, t] = fp16(prob[r, t] * s_v[t]): the per-token scales of V folded into the probabilities.
__global__ void __launch_bounds__(256) kv_scale_probs_kernel(const __half* prob, const __half* v_scale, __half* out, int64_t n, int T)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n; i += (int64_t)gridDim.x * 256)
        out[i] = __float2half_rn(__half2float(prob[i]) * __half2float(v_scale[i % T]));
}

}  // namespace ql
