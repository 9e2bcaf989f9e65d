// Residual connection + RMS normalisation, the operator that produces the linear layer's input (paper Section 3.6:
// "merging residual connection and element-wise operations with a manually optimized RMS normalization operator").
//
//   h[m,k] = x[m,k] + r[m,k]                                 (fp32: the sum of two fp16 values is exact)
//   y[m,k] = h[m,k] / sqrt(mean_k h[m,k]^2 + eps) * (offset + g[k])
//
// One CTA per token.  Pass 1 adds the squares (each thread keeps its own partial sum, 256 of them per token, which
// are then added pairwise: warp shuffles, then one more tree over the 8 warp sums); pass 2 writes fp16(h), the
// residual stream of the next block, and fp16(y), from the sums kept in registers (K <= 16384) or from a second read
// of x and r.  Bound: HBM (reads 2 * M * K * 2 bytes, writes the same).
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ql {

constexpr int kNormThreads = 256;

struct NormParams {
    const __half* x;
    const __half* r;             // may be null: no residual
    const __half* g;
    __half* h_out;               // may be null
    __half* y_out;
    float eps, offset;
    int32_t M, K;
};

__device__ __forceinline__ void norm_load8(const __half* p, float v[8])
{
    const uint4 u = *reinterpret_cast<const uint4*>(p);
    const __half2* h = reinterpret_cast<const __half2*>(&u);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(h[i]);
        v[2 * i] = f.x;
        v[2 * i + 1] = f.y;
    }
}
__device__ __forceinline__ void norm_store8(__half* p, const float v[8])
{
    uint4 u;
    __half2* h = reinterpret_cast<__half2*>(&u);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2half2_rn(v[2 * i], v[2 * i + 1]);
    *reinterpret_cast<uint4*>(p) = u;
}

// VPT: 8-value vectors per thread kept in registers between the two passes (K <= 2048 * VPT); VPT = 0: any K, the
// second pass reads x and r again (they are still in L1 / L2).
template <int VPT>
__global__ void __launch_bounds__(kNormThreads) residual_rmsnorm_kernel(const NormParams p)
{
    __shared__ float warp_sum[kNormThreads / 32];
    __shared__ float rstd_s;
    const int m = blockIdx.x;
    const int64_t row = (int64_t)m * p.K;
    const int n_vec = p.K >> 3;
    constexpr int NV = VPT > 0 ? VPT : 1;
    float keep[NV][8];
    // programmatic dependent launch: the next kernel may start its own set-up now; x and r may come from the previous
    // one, the weights g do not: they are requested before the wait, so that their latency is not added to the chain
    // "previous kernel done -> x -> sum -> y" (one token: 2.05 -> 1.6 us)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    uint4 gk[NV];
    if (VPT > 0) {
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            const int v = threadIdx.x + j * kNormThreads;
            gk[j] = v < n_vec ? *reinterpret_cast<const uint4*>(p.g + 8 * v) : make_uint4(0, 0, 0, 0);
        }
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");

    auto load_h = [&](int v, float a[8]) {
        norm_load8(p.x + row + 8 * v, a);
        if (p.r) {
            float b[8];
            norm_load8(p.r + row + 8 * v, b);
#pragma unroll
            for (int i = 0; i < 8; ++i) a[i] += b[i];
        }
    };
    auto squares = [](const float a[8]) {                                // the 8 squares of a vector, added pairwise
        const float s01 = a[0] * a[0] + a[1] * a[1], s23 = a[2] * a[2] + a[3] * a[3];
        const float s45 = a[4] * a[4] + a[5] * a[5], s67 = a[6] * a[6] + a[7] * a[7];
        return (s01 + s23) + (s45 + s67);
    };

    float ss = 0.f;
    if (VPT > 0) {
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            const int v = threadIdx.x + j * kNormThreads;
            if (v < n_vec) { load_h(v, keep[j]); ss += squares(keep[j]); }
        }
    } else {
        for (int v = threadIdx.x; v < n_vec; v += kNormThreads) {
            float a[8];
            load_h(v, a);
            ss += squares(a);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((threadIdx.x & 31) == 0) warp_sum[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x == 0) {
        const float t = ((warp_sum[0] + warp_sum[1]) + (warp_sum[2] + warp_sum[3])) + ((warp_sum[4] + warp_sum[5]) + (warp_sum[6] + warp_sum[7]));
        rstd_s = 1.0f / sqrtf(t / (float)p.K + p.eps);                   // IEEE division and square root
    }
    __syncthreads();
    const float rstd = rstd_s;

    auto finish = [&](int v, float a[8], const uint4* gv) {
        float g[8];
        if (gv) {
            const __half2* h2 = reinterpret_cast<const __half2*>(gv);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f = __half22float2(h2[i]);
                g[2 * i] = f.x;
                g[2 * i + 1] = f.y;
            }
        } else norm_load8(p.g + 8 * v, g);
        if (p.h_out) norm_store8(p.h_out + row + 8 * v, a);
#pragma unroll
        for (int i = 0; i < 8; ++i) a[i] = (a[i] * rstd) * (p.offset + g[i]);
        norm_store8(p.y_out + row + 8 * v, a);
    };
    if (VPT > 0) {
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            const int v = threadIdx.x + j * kNormThreads;
            if (v < n_vec) finish(v, keep[j], &gk[j]);
        }
    } else {
        for (int v = threadIdx.x; v < n_vec; v += kNormThreads) {
            float a[8];
            load_h(v, a);
            finish(v, a, nullptr);
        }
    }
}

}  // namespace ql
