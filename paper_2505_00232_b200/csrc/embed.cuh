// Embedding lookup from a quantised table (paper Section 4.2: in the mixed 8/4/4 scheme the embedding
// table is stored with int4 weights, like the feed-forward layers): y[t, :] = fp16(s * q[ids[t], :]).
//
// The table is an ordinary packed layer (N = vocabulary, K = hidden size), so the LM head and the
// embedding can share one blob.  A CTA serves one token: its threads walk the 16-byte pieces of the
// token's row (one piece = the row's weights of one lane column in one K chunk), unpack them with the
// same routine the decode and prefill kernels use, multiply by the scale in fp32 (exact: an 11-bit by a
// 4- or 8-bit factor) and round once to fp16, which is the correctly rounded product.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dequant.cuh"
#include "layout.h"

namespace ql {

struct EmbedParams {
    const uint8_t* body;
    const __half* chan_scales;           // nullptr when grouped
    const int32_t* ids;                  // [n] row numbers; rows outside [0, N) give zeros
    __half* y;                           // [n, K]
    int32_t n, N, K, n_kc, block_bytes;
};

template <int BITS, bool GROUPED>
__global__ void __launch_bounds__(128) embed_kernel(const EmbedParams p)
{
    const int t = blockIdx.x;
    const int row = p.ids[t];
    __half* yrow = p.y + (int64_t)t * p.K;
    constexpr int CHUNK_K = BITS == 4 ? 64 : 32;
    if (row < 0 || row >= p.N) {
        for (int k = threadIdx.x; k < p.K; k += blockDim.x) yrow[k] = __float2half_rn(0.f);
        return;
    }
    const int rsb = row / kRsbRows, rb = (row % kRsbRows) / kRbRows;
    const int r16 = row % kRbRows, g = r16 & 7, hi = r16 >> 3;          // lane group and row half inside the row-block
    const uint8_t* base = p.body + (int64_t)rsb * p.n_kc * p.block_bytes + rb * 512 + g * 64;
    float cs = 1.f;
    if (!GROUPED) cs = __half2float(p.chan_scales[row]);
    for (int piece = threadIdx.x; piece < p.n_kc * 4; piece += blockDim.x) {
        const int kc = piece >> 2, c = piece & 3;
        const uint8_t* blk = base + (int64_t)kc * p.block_bytes;
        const uint4 w = *reinterpret_cast<const uint4*>(blk + c * 16);
        float s0 = cs, s1 = cs;                                         // scales of the chunk's two groups
        if (GROUPED) {
            const uint2 sc = *reinterpret_cast<const uint2*>(blk - (rb * 512 + g * 64) + kWeightBlockBytes + rb * 64 + g * 8);
            const __half2 h = *reinterpret_cast<const __half2*>(hi ? &sc.y : &sc.x);
            s0 = __low2float(h);
            s1 = __high2float(h);
        }
        const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
        constexpr int NW = BITS == 4 ? 4 : 2;
#pragma unroll
        for (int i = 0; i < NW; ++i) {
            uint32_t a[4];
            if (BITS == 4) unpack_int4_word(ww[i], a);
            else unpack_int8_words(ww[2 * i], ww[2 * i + 1], a);
#pragma unroll
            for (int jj = 0; jj < 2; ++jj) {                            // registers hi and hi + 2 hold this row
                const __half2 q2 = *reinterpret_cast<const __half2*>(&a[hi + 2 * jj]);
                const int kin = BITS == 4 ? int4_k_in_chunk(c, i, 2 * jj) : 8 * c + 4 * i + 2 * jj;
                const int k = kc * CHUNK_K + kin;
                const float s = (BITS == 4 && kin >= 32) ? s1 : s0;
                if (k < p.K)
                    *reinterpret_cast<__half2*>(yrow + k) =
                        __halves2half2(__float2half_rn(s * __low2float(q2)), __float2half_rn(s * __high2float(q2)));
            }
        }
    }
}

}  // namespace ql
