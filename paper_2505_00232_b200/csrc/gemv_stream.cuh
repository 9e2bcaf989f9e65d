// Decode kernel, streaming form: a persistent grid in which every CTA streams one contiguous byte
// range of the packed weights through a ring of shared-memory stages filled by bulk TMA copies
// (paper Section 3.7 / 4.2: decode is bound by the weight bytes read, so the kernel is built around
// keeping HBM busy).
//
//   * The (row super-block, k-chunk) blocks of the blob are numbered in storage order; CTA p of P takes
//     blocks [p*B/P, (p+1)*B/P): equal work for every CTA whatever the layer shape (no wave tail).
//   * One producer thread keeps the ring full: per stage one bulk copy of the block (4096 or 4608
//     bytes) and M small bulk copies of the matching 64-/32-wide slices of x.  Bytes in flight are set
//     by the ring depth, not by registers or occupancy.
//   * Eight consumer warps each own one row-block (16 channels) of every block: 16-byte shared loads,
//     register unpack, mma.m16n8k16 with the <= 8 tokens as the 8 columns, fp32 accumulation.
//   * A range that ends inside a row super-block leaves a partial sum.  Partials go to a scratch area
//     (one slot pair per CTA) and the warp that arrives last at a per-(super-block, row-block) counter
//     adds them in CTA order and writes y: fixed summation order, no spinning, no float atomics.
//
// The scratch area and the counters belong to the handle; calls on one handle must be stream-ordered.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dequant.cuh"
#include "gemv.cuh"
#include "layout.h"
#include "sm100_ptx.cuh"

namespace ql {

constexpr int kStreamConsumerWarps = 8;
constexpr int kStreamThreads = (kStreamConsumerWarps + 1) * 32;
constexpr int kStreamMaxStages = 24;
constexpr int kStreamPartialFloats = kStreamConsumerWarps * 128;        // one slot: 8 row-blocks x 16 rows x 8 tokens


struct StreamParams {
    const uint8_t* body;
    const __half* chan_scales;
    const __half* x;
    __half* y;
    float* scratch;                      // [P][2][kStreamPartialFloats]
    unsigned int* counters;              // [n_rsb][8], zero between launches
    int32_t M, N, K;
    int32_t n_rsb, n_kc, block_bytes;
    int32_t P;                           // CTAs in the grid (<= number of blocks)
    int32_t stages;
};

template <int BITS>
struct StreamStage {
    static constexpr int kChunkK = BITS == 4 ? 64 : 32;
    static constexpr int kXRowBytes = kChunkK * 2;                       // one token's slice
    static constexpr int kXStride = BITS == 4 ? 192 : 64;                // == 64 (mod 128): conflict-free 16-byte loads
    static constexpr int kXOffset = BITS == 4 ? (kWeightBlockBytes + kScaleBlockBytes) : kWeightBlockBytes;
    static constexpr int kBytes = kXOffset + 8 * kXStride;               // 6144 / 4608
};

__host__ __device__ inline int64_t stream_range_begin(int64_t p, int64_t B, int64_t P) { return p * B / P; }
__host__ __device__ inline int stream_owner(int64_t b, int64_t B, int64_t P) { return (int)(((b + 1) * P - 1) / B); }

// Accumulator flush of (row super-block rsb, row-block warp): either the final store (this CTA saw every
// chunk of the super-block) or a partial sum handed to the last-arriver reduction.  Out of line: it runs
// once per super-block, the unrolled main loop stays small.
template <bool GROUPED>
__device__ __noinline__ void stream_flush(const StreamParams& p, int rsb, int rsb_first, bool complete, int warp, int lane,
                                          float t0, float t1, float t2, float t3)
{
    const int g = lane >> 2, c = lane & 3;
    const int row_g = rsb * kRsbRows + warp * kRbRows + g;
    auto store_final = [&](const float v[4]) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int row = row_g + 8 * (j >> 1), tok = 2 * c + (j & 1);
            if (row < p.N && tok < p.M) {
                float o = v[j];
                if (!GROUPED) o *= __half2float(p.chan_scales[row]);
                p.y[(int64_t)tok * p.N + row] = __float2half_rn(o);
            }
        }
    };
    const float total[4] = {t0, t1, t2, t3};
    if (complete) {
        store_final(total);
        return;
    }
    const int64_t B = (int64_t)p.n_rsb * p.n_kc;
    const int slot = (rsb == rsb_first) ? 0 : 1;
    float* mine = p.scratch + ((int64_t)blockIdx.x * 2 + slot) * kStreamPartialFloats + warp * 128 + lane * 4;
    __stcg(reinterpret_cast<float4*>(mine), make_float4(t0, t1, t2, t3));
    __threadfence();
    __syncwarp();
    const int p_lo = stream_owner((int64_t)rsb * p.n_kc, B, p.P);
    const int p_hi = stream_owner((int64_t)(rsb + 1) * p.n_kc - 1, B, p.P);
    unsigned int old = 0;
    if (lane == 0) old = atomicAdd(&p.counters[rsb * 8 + warp], 1u);
    old = __shfl_sync(0xffffffffu, old, 0);
    if ((int)old != p_hi - p_lo) return;
    // last contributor: add all partials in CTA order
    __threadfence();
    float v[4] = {0.f, 0.f, 0.f, 0.f};
    // CTA p_lo is the only contributor that may have reached the super-block from an earlier one
    const int slot_lo = ((int)(stream_range_begin(p_lo, B, p.P) / p.n_kc) == rsb) ? 0 : 1;
    const float* base = p.scratch + warp * 128 + lane * 4;
    for (int q0 = p_lo; q0 <= p_hi; q0 += 8) {
        float4 t[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {                                    // independent loads first, then the ordered sum
            const int q = q0 + j;
            const int qslot = q == p_lo ? slot_lo : 0;
            t[j] = q <= p_hi ? __ldcg(reinterpret_cast<const float4*>(base + ((int64_t)q * 2 + qslot) * kStreamPartialFloats))
                             : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) { v[0] += t[j].x; v[1] += t[j].y; v[2] += t[j].z; v[3] += t[j].w; }
    }
    store_final(v);
    if (lane == 0) p.counters[rsb * 8 + warp] = 0;                       // ready for the next launch
}

// One block's worth of registers for a consumer lane.
struct StreamFrag {
    uint4 w;
    uint2 sc;
    uint4 x0, x1;
};

template <int BITS, bool GROUPED>
__device__ __forceinline__ void stream_load(StreamFrag& f, const unsigned char* st, int w_off, int s_off, int x_off)
{
    using ST = StreamStage<BITS>;
    f.w = *reinterpret_cast<const uint4*>(st + w_off);
    if (GROUPED) f.sc = *reinterpret_cast<const uint2*>(st + s_off);
    // Lanes whose token column does not exist (g >= M) read the last real token instead: MMA columns are
    // independent, and those columns are never stored.
    f.x0 = *reinterpret_cast<const uint4*>(st + x_off);
    if (BITS == 4) f.x1 = *reinterpret_cast<const uint4*>(st + x_off + 64);
    (void)sizeof(ST);
}

template <int BITS, bool GROUPED>
__device__ __forceinline__ void stream_math(const StreamFrag& f, float total[4])
{
    uint32_t a[4];
    if (BITS == 4) {
        const uint32_t ww[4] = {f.w.x, f.w.y, f.w.z, f.w.w};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint4 xv = h == 0 ? f.x0 : f.x1;
            if (GROUPED) {
                float acc[4] = {0.f, 0.f, 0.f, 0.f};
                unpack_int4_word(ww[2 * h], a);
                mma_16816_pure(acc, a, xv.x, xv.y);
                unpack_int4_word(ww[2 * h + 1], a);
                mma_16816_pure(acc, a, xv.z, xv.w);
                const __half2 s_lo = *reinterpret_cast<const __half2*>(&f.sc.x);            // row g:   G0, G1
                const __half2 s_hi = *reinterpret_cast<const __half2*>(&f.sc.y);            // row g+8: G0, G1
                const float sg = h == 0 ? __low2float(s_lo) : __high2float(s_lo);
                const float sg8 = h == 0 ? __low2float(s_hi) : __high2float(s_hi);
                total[0] = fmaf(sg, acc[0], total[0]);
                total[1] = fmaf(sg, acc[1], total[1]);
                total[2] = fmaf(sg8, acc[2], total[2]);
                total[3] = fmaf(sg8, acc[3], total[3]);
            } else {
                unpack_int4_word(ww[2 * h], a);
                mma_16816_pure(total, a, xv.x, xv.y);
                unpack_int4_word(ww[2 * h + 1], a);
                mma_16816_pure(total, a, xv.z, xv.w);
            }
        }
    } else {
        unpack_int8_words(f.w.x, f.w.y, a);
        mma_16816_pure(total, a, f.x0.x, f.x0.y);
        unpack_int8_words(f.w.z, f.w.w, a);
        mma_16816_pure(total, a, f.x0.z, f.x0.w);
    }
}

template <int BITS, bool GROUPED, int NS>
__global__ void __launch_bounds__(kStreamThreads, 3) gemv_stream_kernel(const StreamParams p)
{
    using ST = StreamStage<BITS>;
    static_assert(NS % 2 == 0 && NS <= kStreamMaxStages, "the ring is consumed in stage pairs");
    extern __shared__ __align__(128) unsigned char smem_dyn[];
    __shared__ __align__(8) unsigned long long bars[2 * NS];
    __shared__ uint32_t abort_word[3];           // [0] abort, [2] past griddepcontrol.wait (see wait_expired)

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t B = (int64_t)p.n_rsb * p.n_kc;
    const int64_t b0 = stream_range_begin(blockIdx.x, B, p.P), b1 = stream_range_begin(blockIdx.x + 1, B, p.P);
    const int nb = (int)(b1 - b0);
    volatile uint32_t* abort_flag = abort_word;

    const uint32_t stage0 = smem_u32(smem_dyn);
    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8 * s; };
    auto empty_bar = [&](int s) { return bar0 + 8 * (NS + s); };

    if (threadIdx.x == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), kStreamConsumerWarps);
        }
        abort_word[0] = 0;
        abort_word[1] = 0;
        abort_word[2] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp == kStreamConsumerWarps) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            const uint8_t* src = p.body + b0 * p.block_bytes;
            const int kc_first = (int)(b0 % p.n_kc);
            const uint32_t stage_tx = (uint32_t)p.block_bytes + (uint32_t)p.M * ST::kXRowBytes;
            auto issue_w = [&](int i, int s) {
                mbar_expect_tx(full_bar(s), stage_tx);
                bulk_copy_g2s(stage0 + s * ST::kBytes, src + (int64_t)i * p.block_bytes, (uint32_t)p.block_bytes, full_bar(s));
            };
            auto issue_x = [&](int s, int kc_) {
                for (int m = 0; m < p.M; ++m)
                    bulk_copy_g2s(stage0 + s * ST::kBytes + ST::kXOffset + m * ST::kXStride,
                                  p.x + (int64_t)m * p.K + (int64_t)kc_ * ST::kChunkK, ST::kXRowBytes, full_bar(s));
            };
            // Weights do not depend on the previous kernel in the stream: fill the ring with them first,
            // wait for the previous kernel, then add the x slices of those stages.
            const int pro = min(NS, nb);
            for (int i = 0; i < pro; ++i) issue_w(i, i);
            asm volatile("griddepcontrol.wait;" ::: "memory");
            abort_flag[2] = 1;
            int kcp = kc_first;
            for (int i = 0; i < pro; ++i) { issue_x(i, kcp); kcp = kcp + 1 == p.n_kc ? 0 : kcp + 1; }
            int s = 0;                                                   // pro == NS whenever this loop runs
            uint32_t par = 0;                                            // parity of the consumers' first release
            for (int i = pro; i < nb; ++i) {
                if (!mbar_wait<true>(empty_bar(s), par, abort_flag, 0x600 + s)) break;
                issue_w(i, s);
                issue_x(s, kcp);
                kcp = kcp + 1 == p.n_kc ? 0 : kcp + 1;
                if (++s == NS) { s = 0; par ^= 1; }
            }
        }
        return;
    }

    // ---------------------------------------------------------------------- consumers
    const int g = lane >> 2, c = lane & 3;
    const int w_off = warp * 512 + lane * 16;
    const int s_off = kWeightBlockBytes + warp * 64 + g * 8;
    const int x_off = ST::kXOffset + min(g, p.M - 1) * ST::kXStride + c * 16;
    float total[4] = {0.f, 0.f, 0.f, 0.f};
    int rsb = (int)(b0 / p.n_kc), kc = (int)(b0 % p.n_kc);
    const int rsb_first = rsb;
    bool covers_start = (kc == 0);                                       // current super-block entered at its first chunk
    const int n_kc = p.n_kc;

    // bookkeeping after one block: flush at the end of a super-block or of the range
    auto advance = [&](bool last) {
        const bool end_of_rsb = (kc + 1 == n_kc);
        if (end_of_rsb || last) {
            stream_flush<GROUPED>(p, rsb, rsb_first, covers_start && end_of_rsb, warp, lane, total[0], total[1], total[2], total[3]);
            total[0] = total[1] = total[2] = total[3] = 0.f;
            covers_start = true;                                         // the next super-block starts at chunk 0
        }
        if (end_of_rsb) { kc = 0; ++rsb; } else ++kc;
    };

    const int npairs = nb >> 1;
    int j = 0;
    uint32_t par = 0;
    while (j < npairs) {
#pragma unroll
        for (int s = 0; s < NS; s += 2) {
            if (j >= npairs) break;
            if (!mbar_wait<true>(full_bar(s), par, abort_flag, 0x700 + s)) return;
            if (!mbar_wait<true>(full_bar(s + 1), par, abort_flag, 0x700 + s + 1)) return;
            StreamFrag fa, fb;
            stream_load<BITS, GROUPED>(fa, smem_dyn + s * ST::kBytes, w_off, s_off, x_off);
            stream_load<BITS, GROUPED>(fb, smem_dyn + (s + 1) * ST::kBytes, w_off, s_off, x_off);
            __syncwarp();
            if (lane == 0) {                                             // data is in registers: free both stages
                mbar_arrive(empty_bar(s));
                mbar_arrive(empty_bar(s + 1));
            }
            stream_math<BITS, GROUPED>(fa, total);
            advance(false);
            stream_math<BITS, GROUPED>(fb, total);
            ++j;
            advance(2 * j == nb);
        }
        par ^= 1;
    }
    if (nb & 1) {                                                        // odd range: one more block
        const int s = (nb - 1) % NS;
        const uint32_t par_last = (uint32_t)((nb - 1) / NS) & 1u;
        if (!mbar_wait<true>(full_bar(s), par_last, abort_flag, 0x700 + s)) return;
        StreamFrag fa;
        stream_load<BITS, GROUPED>(fa, smem_dyn + s * ST::kBytes, w_off, s_off, x_off);
        stream_math<BITS, GROUPED>(fa, total);
        advance(true);
    }
}

}  // namespace ql
