// Decode kernel for int8 layers with MANY rows and a SHORT K (at most 8 chunks of 32): the score product over a KV
// cache held as weights (paper Section 3.8: the K cache is a layer with O = cache positions and I = d_h), for all KV
// heads of an attention layer at once.
//
// In gemv.cuh a warp's whole job would be one row-block of d_h / 32 chunks (2 KB for d_h = 128): the kernel is then
// bound by CTA turnover -- launch, ring fill, x, sums, store, exit per 16 KB -- and streams a long cache at a quarter
// of the memory bandwidth.  Here the grid is persistent: a CTA's 8 warps take the 8 row-blocks of one row super-block
// (one contiguous piece of the blob), the CTA walks over super-blocks with stride gridDim.x, and the bytes of its next
// super-block are in flight (second half of a two-stage cp.async buffer) while it works on the current one.  A warp
// holds a row-block's complete K, so there is no reduction across warps, no shared-memory hand-over and no barrier:
// every lane stores the (at most 4) outputs of its accumulator fragment.  Same chunk order and the same MMA sequence as
// gemv.cuh with an undivided K: bit-identical results.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dequant.cuh"
#include "gemv.cuh"
#include "layout.h"

namespace ql {

struct GemvRowsParams {
    const uint8_t* body[kGemvMaxBatch];          // first block of each packed body
    const __half* chan_scales[kGemvMaxBatch];
    __half* y[kGemvMaxBatch];                    // [M, N_i]
    const __half* xl[kGemvMaxBatch];             // [M, K], one input per layer
    int32_t N[kGemvMaxBatch];
    int32_t rsb_end[kGemvMaxBatch];              // row super-blocks of layers 0..i
    int32_t n_layers, M, K, n_rsb, block_bytes;
};

// NKC: chunks of 32 along K (K = 32 * NKC).
template <int NKC>
__global__ void __launch_bounds__(kGemvThreads, NKC <= 4 ? 4 : 3) gemv_rows_kernel(const GemvRowsParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, c = lane & 3;
    // two stages of NKC chunk slots per warp; a lane reads back exactly the 16 bytes it copied
    const uint32_t ring = (uint32_t)__cvta_generic_to_shared(smem_raw) + (uint32_t)(warp * 2 * NKC * 512 + lane * 16);

    auto place = [&](int sb, int& ly, int& sb_local) {                  // which layer a super-block belongs to
        ly = 0;
#pragma unroll
        for (int i = 1; i < kGemvMaxBatch; ++i)
            if (i < p.n_layers && sb >= p.rsb_end[i - 1]) ly = i;
        sb_local = sb - (ly ? p.rsb_end[ly - 1] : 0);
    };
    auto issue = [&](int sb, int stage) {                               // this warp's row-block of super-block sb -> stage
        if (sb < p.n_rsb) {
            int ly, sb_local;
            place(sb, ly, sb_local);
            const uint8_t* src = p.body[ly] + (int64_t)sb_local * NKC * p.block_bytes + warp * 512 + lane * 16;
#pragma unroll
            for (int kc = 0; kc < NKC; ++kc)
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ring + (uint32_t)((stage * NKC + kc) * 512)),
                             "l"(src + (int64_t)kc * p.block_bytes) : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");            // (an empty group keeps the count of groups in step)
    };

    int sb = blockIdx.x, stage = 0;
    issue(sb, 0);                                                       // weights do not depend on the previous kernel
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    for (; sb < p.n_rsb; sb += gridDim.x, stage ^= 1) {
        issue(sb + gridDim.x, stage ^ 1);
        int ly, sb_local;
        place(sb, ly, sb_local);
        const int row0 = sb_local * kRsbRows + warp * kRbRows + g, N = p.N[ly];
        float s0 = 0.f, s1 = 0.f;
        if (row0 < N) s0 = __half2float(p.chan_scales[ly][row0]);
        if (row0 + 8 < N) s1 = __half2float(p.chan_scales[ly][row0 + 8]);
        // lanes whose token column does not exist read the last real token; those columns are never stored
        const __half* x = p.xl[ly] + (int64_t)min(g, p.M - 1) * p.K + 8 * c;
        uint4 xv[NKC];
#pragma unroll
        for (int kc = 0; kc < NKC; ++kc)
            asm volatile("ld.global.ca.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(xv[kc].x), "=r"(xv[kc].y), "=r"(xv[kc].z), "=r"(xv[kc].w) : "l"(x + 32 * kc));
        asm volatile("cp.async.wait_group 1;" ::: "memory");
        float total[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int kc = 0; kc < NKC; ++kc) {
            uint4 w;
            asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(w.x), "=r"(w.y), "=r"(w.z), "=r"(w.w) : "r"(ring + (uint32_t)((stage * NKC + kc) * 512)));
            uint32_t a[4];
            unpack_int8_words(w.x, w.y, a);
            mma_16816_pure(total, a, xv[kc].x, xv[kc].y);
            unpack_int8_words(w.z, w.w, a);
            mma_16816_pure(total, a, xv[kc].z, xv[kc].w);
        }
        // accumulator fragment: total[0], total[1] = row g, tokens 2c, 2c + 1; total[2], total[3] = row g + 8
        __half* y = p.y[ly];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int row = row0 + 8 * (i >> 1), tok = 2 * c + (i & 1);
            if (row < N && tok < p.M) y[(int64_t)tok * N + row] = __float2half_rn((0.f + total[i]) * ((i >> 1) ? s1 : s0));
        }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

}  // namespace ql
