// Decode kernel with int8 activations (paper Section 3.7: in the memory-bound decode stage the quantisation of
// the input activations is done INSIDE the fully-connected kernel, and the products with the pre-quantised
// weights use integer instructions, with the dequantisation applied to the output).
//
// Steps, in the order the section gives them:
//   1. quantise x per token:  amax = max |x[m,:]|,  r = 127 / amax,  xq = round-half-even(x * r) clamped to
//      [-127, 127],  scale_x = amax / 127  (IEEE fp32 operations, one rounding each; a zero row: scale 1, xq 0)
//   2. integer dot products of xq with the stored weight integers on the tensor cores
//      (mma.m16n8k32, u8 x s8 -> s32): exact
//   3. dequantise the output:  y = scale_x[m] * sum_g s[n,g] * acc[m,n,g]   (fp32), rounded once to fp16
//
// Work decomposition, ring and reductions are those of gemv.cuh: a warp owns one row-block and one K slice.  The
// weights are stored with an offset (q + 8, q + 128), so the products come out as sum (q + off) * xq; the term
// off * sum xq is known per token and 32-k group once x is quantised, and enters the MMA as its accumulator input.
// int4 unpack is two logic operations per 8 weights (the low and the high nibbles of a word are the 4-byte
// operand registers of rows g and g + 8), against nine for the fp16 path.
#pragma once
#include <cooperative_groups.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gemv.cuh"
#include "layout.h"

namespace ql {

struct GemvA8Params {
    const uint8_t* body;
    const __half* chan_scales;           // per-channel scales (nullptr when grouped)
    const __half* x;                     // [M, K] fp16
    __half* y;                           // [M, N]
    int32_t M, N, K;
    int32_t n_rb, n_kc, block_bytes;
    int32_t ks_cta, ks_cta_log2, cl, cps;
    int32_t xq_stride;                   // bytes between tokens in the shared xq slab (span + 32: rows land 8 banks apart)
    int32_t xq_bytes;                    // bytes of the slab
    int32_t sg_bytes;                    // bytes of the per-group sums that follow it
};

// D = A (16 x 32, u8: stored weight integers) . B (32 x 8, s8: quantised activations) + C, exact in s32.
__device__ __forceinline__ void imma_16832(int d[4], const uint32_t a[4], uint32_t b0, uint32_t b1, const int c[4])
{
    asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};"
        : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "r"(c[0]), "r"(c[1]), "r"(c[2]), "r"(c[3]));
}

// Step 1 for one value, bit for bit as stated above.  |x| <= amax gives |x * r| <= 127 (1 + 2^-22), which rounds
// into [-127, 127] by itself: the clamp of the definition never acts, and is left to the byte packing's saturation.
__device__ __forceinline__ int quantize_one(float x, float r) { return __float2int_rn(__fmul_rn(x, r)); }

// Four s32 values in [-128, 127] as the four bytes of a word (lowest byte first).
__device__ __forceinline__ uint32_t pack_s8x4(int b0, int b1, int b2, int b3)
{
    uint32_t hi, out;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, 0;" : "=r"(hi) : "r"(b3), "r"(b2));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(out) : "r"(b1), "r"(b0), "r"(hi));
    return out;
}
// Sum of the four signed bytes of a word.
__device__ __forceinline__ int sum_s8x4(uint32_t w) { return __dp4a((int)w, 0x01010101, 0); }

template <int BITS, bool GROUPED>
__global__ void __launch_bounds__(kGemvThreads, 4) gemv_a8_kernel(const GemvA8Params p)
{
    namespace cg = cooperative_groups;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ int red[kGemvWarps][128];                                 // per-warp results: s32, or fp32 bits when GROUPED
    __shared__ int part[128];
    __shared__ float amax_w[kGemvWarps][8];
    __shared__ float scale_x[8], recip_x[8];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, c = lane & 3;
    constexpr int CHUNK_K = BITS == 4 ? 64 : 32;
    constexpr int OFFSET = BITS == 4 ? 8 : 128;                          // storage offset of the weight integers

    uint32_t crank_u, rb_group_u;
    asm("mov.u32 %0, %%cluster_ctarank;" : "=r"(crank_u));
    asm("mov.u32 %0, %%clusterid.x;" : "=r"(rb_group_u));
    const int crank = (int)crank_u, rb_group = (int)rb_group_u;
    const int rb_per_cta = kGemvWarps >> p.ks_cta_log2;
    const int ks_local = warp & (p.ks_cta - 1);
    const int rb = rb_group * rb_per_cta + (warp >> p.ks_cta_log2);
    const bool rb_live = rb < p.n_rb;
    const int ks = crank * p.ks_cta + ks_local;
    const int kc0 = min(ks * p.cps, p.n_kc);
    const int kc1 = rb_live ? min(kc0 + p.cps, p.n_kc) : kc0;
    const int kc_cta0 = min(crank * p.ks_cta * p.cps, p.n_kc);           // first chunk of this CTA's K range
    const int kc_cta1 = min(kc_cta0 + p.ks_cta * p.cps, p.n_kc);
    const int k_cta0 = kc_cta0 * CHUNK_K, span = (kc_cta1 - kc_cta0) * CHUNK_K;

    signed char* xq = reinterpret_cast<signed char*>(smem_raw);          // [M][xq_stride], int4: each 4 k stored in order 0, 2, 1, 3
    int* sg = reinterpret_cast<int*>(smem_raw + p.xq_bytes);             // [32-k groups of the span][8 tokens]: -OFFSET * sum xq
    constexpr int WARP_SMEM = kGemvRing * 512 + (GROUPED ? 2 * 512 : 0);
    unsigned char* ring = smem_raw + p.xq_bytes + p.sg_bytes + warp * WARP_SMEM;
    unsigned char* sbuf = ring + kGemvRing * 512;
    const uint32_t ring_u32 = (uint32_t)__cvta_generic_to_shared(ring) + lane * 16;
    const uint32_t sbuf_u32 = (uint32_t)__cvta_generic_to_shared(sbuf) + lane * 16;
    const uint8_t* blk = p.body + ((int64_t)(rb >> 3) * p.n_kc + kc0) * p.block_bytes;
    const uint8_t* wsrc = blk + (rb & 7) * 512 + lane * 16;
    const int s_off = (lane >> 2) * p.block_bytes + kWeightBlockBytes - (rb & 7) * 448 + (lane & 3) * 16 - lane * 16;

    auto copy16 = [](uint32_t dst, const void* src, bool in_range) {     // out of range: reads nothing, writes zeros
        const uint32_t sz = in_range ? 16u : 0u;
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
    };
    auto commit = [] { asm volatile("cp.async.commit_group;" ::: "memory"); };

    // Weights do not depend on the previous kernel: fill the ring before waiting for it.
    if (GROUPED) copy16(sbuf_u32, wsrc + s_off, kc0 + (lane >> 2) < kc1);
#pragma unroll
    for (int d = 0; d < kGemvRing; ++d) {
        copy16(ring_u32 + d * 512, wsrc, kc0 + d < kc1);
        commit();
        wsrc += p.block_bytes;
    }
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // ---- step 1a: amax of every token over its WHOLE row (every CTA needs it, whatever its K range)
    {
        float am[8];
#pragma unroll
        for (int m = 0; m < 8; ++m) am[m] = 0.f;
        const int vec_per_row = p.K >> 3;
        // eight independent 16-byte loads per thread and turn, so that their latencies overlap
#pragma unroll
        for (int m = 0; m < 8; ++m) {
            if (m < p.M) {
                const uint4* row = reinterpret_cast<const uint4*>(p.x + (int64_t)m * p.K);
                for (int v0 = threadIdx.x; v0 < vec_per_row; v0 += 8 * kGemvThreads) {
                    uint4 u[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int v = v0 + j * kGemvThreads;
                        u[j] = v < vec_per_row ? row[v] : make_uint4(0, 0, 0, 0);
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const __half2* h = reinterpret_cast<const __half2*>(&u[j]);
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const float2 f = __half22float2(__habs2(h[i]));
                            am[m] = fmaxf(am[m], fmaxf(f.x, f.y));
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int m = 0; m < 8; ++m) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) am[m] = fmaxf(am[m], __shfl_xor_sync(0xffffffffu, am[m], o));
            if (lane == 0) amax_w[warp][m] = am[m];
        }
        __syncthreads();
        if (threadIdx.x < 8) {
            float a = 0.f;
            for (int w = 0; w < kGemvWarps; ++w) a = fmaxf(a, amax_w[w][threadIdx.x]);
            const bool live = a > 0.f;
            const float safe = live ? a : 1.f;
            recip_x[threadIdx.x] = __fdiv_rn(127.f, safe);
            scale_x[threadIdx.x] = live ? __fdiv_rn(safe, 127.f) : 1.f;
        }
        __syncthreads();
    }
    // ---- step 1b: quantise this CTA's K range, and -OFFSET * (sum of xq) per token and 32-k group
    {
        // 8 values per thread and turn, 4 threads per 32-k group; four turns' loads are issued together
        const int vec_per_tok = span >> 3, total = p.M * vec_per_tok;
        constexpr int B = 4;
        for (int i0 = warp * 32; i0 < total; i0 += B * kGemvThreads) {
            uint4 u[B];
            int mm[B], vv[B];
#pragma unroll
            for (int b = 0; b < B; ++b) {
                const int i = i0 + b * kGemvThreads + lane;
                mm[b] = 0; vv[b] = 0;
                u[b] = make_uint4(0, 0, 0, 0);
                if (i < total) {
                    mm[b] = i / vec_per_tok;
                    vv[b] = i - mm[b] * vec_per_tok;
                    const int k = k_cta0 + vv[b] * 8;
                    if (k < p.K) u[b] = *reinterpret_cast<const uint4*>(p.x + (int64_t)mm[b] * p.K + k);
                }
            }
#pragma unroll
            for (int b = 0; b < B; ++b) {
                if (i0 + b * kGemvThreads >= total) break;               // (warp-uniform)
                const int i = i0 + b * kGemvThreads + lane, m = mm[b], v = vv[b];
                const __half2* h = reinterpret_cast<const __half2*>(&u[b]);
                const float r = recip_x[m];
                int q8[8];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float2 f = __half22float2(h[j]);
                    q8[2 * j] = quantize_one(f.x, r);
                    q8[2 * j + 1] = quantize_one(f.y, r);
                }
                uint2 out;
                if (BITS == 4) { out.x = pack_s8x4(q8[0], q8[2], q8[1], q8[3]); out.y = pack_s8x4(q8[4], q8[6], q8[5], q8[7]); }
                else { out.x = pack_s8x4(q8[0], q8[1], q8[2], q8[3]); out.y = pack_s8x4(q8[4], q8[5], q8[6], q8[7]); }
                if (i < total) *reinterpret_cast<uint2*>(xq + m * p.xq_stride + v * 8) = out;
                int s8 = sum_s8x4(out.x) + sum_s8x4(out.y);
                s8 += __shfl_xor_sync(0xffffffffu, s8, 1);
                s8 += __shfl_xor_sync(0xffffffffu, s8, 2);
                if (i < total && (lane & 3) == 0) sg[(v >> 2) * 8 + m] = -OFFSET * s8;
            }
        }
        __syncthreads();
    }

    // ---- steps 2 and 3 over this warp's chunks
    float ftotal[4] = {0.f, 0.f, 0.f, 0.f};                              // GROUPED: sum_g s * acc, fp32
    int itotal[4] = {0, 0, 0, 0};                                        // per channel: the integer sum (offset term added below)
    const signed char* xrow = xq + min(g, p.M - 1) * p.xq_stride + 8 * c;   // columns g >= M copy the last token, never stored
    [[maybe_unused]] const uint32_t sc_u32 = sbuf_u32 - lane * 16 + g * 8;   // (read by the grouped form only)
    int sflip = 0;
    for (int kc = kc0; kc < kc1; kc += kGemvRing) {
#pragma unroll
        for (int d = 0; d < kGemvRing; ++d) {
            if (kc + d >= kc1) break;
            asm volatile("cp.async.wait_group %0;" ::"n"(kGemvRing - 1) : "memory");
            if (GROUPED && d == 0) {
                __syncwarp();                                            // scales of this pass visible; last pass's reads done
                copy16(sbuf_u32 + (sflip ^ 1) * 512, wsrc + s_off, kc + kGemvRing + (lane >> 2) < kc1);
            }
            const uint4 w = *reinterpret_cast<const uint4*>(ring + d * 512 + lane * 16);
            uint2 sc = make_uint2(0, 0);
            if (GROUPED) sc = *reinterpret_cast<const uint2*>(sbuf + sflip * 512 + d * 64 + g * 8);
            copy16(ring_u32 + d * 512, wsrc, kc + d + kGemvRing < kc1);
            commit();
            wsrc += p.block_bytes;
            const int kl = (kc + d - kc_cta0) * CHUNK_K;                 // first k of the chunk inside the CTA's range
            if (BITS == 4) {
                const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int h = 0; h < 2; ++h) {                            // the chunk's two 32-k groups
                    uint32_t a[4];
                    a[0] = ww[2 * h] & 0x0F0F0F0Fu;                      // row g:     k 8c + {0, 2, 1, 3}
                    a[1] = (ww[2 * h] >> 4) & 0x0F0F0F0Fu;               // row g + 8
                    a[2] = ww[2 * h + 1] & 0x0F0F0F0Fu;                  // row g:     k 8c + 4 + {0, 2, 1, 3}
                    a[3] = (ww[2 * h + 1] >> 4) & 0x0F0F0F0Fu;
                    const uint2 xb = *reinterpret_cast<const uint2*>(xrow + kl + 32 * h);
                    if (GROUPED) {
                        const int2 off = *reinterpret_cast<const int2*>(sg + ((kl >> 5) + h) * 8 + 2 * c);
                        const int cin[4] = {off.x, off.y, off.x, off.y};
                        int acc[4];
                        imma_16832(acc, a, xb.x, xb.y, cin);
                        const __half2 s_lo = *reinterpret_cast<const __half2*>(&sc.x);      // row g:   G0, G1
                        const __half2 s_hi = *reinterpret_cast<const __half2*>(&sc.y);      // row g+8: G0, G1
                        const float s0 = h == 0 ? __low2float(s_lo) : __high2float(s_lo);
                        const float s8 = h == 0 ? __low2float(s_hi) : __high2float(s_hi);
                        ftotal[0] = fmaf(s0, (float)acc[0], ftotal[0]);
                        ftotal[1] = fmaf(s0, (float)acc[1], ftotal[1]);
                        ftotal[2] = fmaf(s8, (float)acc[2], ftotal[2]);
                        ftotal[3] = fmaf(s8, (float)acc[3], ftotal[3]);
                    } else {
                        imma_16832(itotal, a, xb.x, xb.y, itotal);
                    }
                }
            } else {
                uint32_t a[4];
                a[0] = __byte_perm(w.x, w.y, 0x5410);                    // row g:     k 8c + 0..3
                a[1] = __byte_perm(w.x, w.y, 0x7632);                    // row g + 8
                a[2] = __byte_perm(w.z, w.w, 0x5410);                    // row g:     k 8c + 4..7
                a[3] = __byte_perm(w.z, w.w, 0x7632);
                const uint2 xb = *reinterpret_cast<const uint2*>(xrow + kl);
                imma_16832(itotal, a, xb.x, xb.y, itotal);
            }
        }
        sflip ^= 1;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    if (!GROUPED) {                                                      // the offset term of this warp's K slice, per token column
        int o0 = 0, o1 = 0;
        const int g0 = ((kc0 - kc_cta0) * CHUNK_K) >> 5, g1 = ((kc1 - kc_cta0) * CHUNK_K) >> 5;
        for (int gi = g0; gi < g1; ++gi) {
            const int2 off = *reinterpret_cast<const int2*>(sg + gi * 8 + 2 * c);
            o0 += off.x; o1 += off.y;
        }
        itotal[0] += o0; itotal[1] += o1; itotal[2] += o0; itotal[3] += o1;
    }

    // ---- K reduction across warps (shared memory), then across the cluster (distributed shared memory)
    if (GROUPED) *reinterpret_cast<float4*>(&red[warp][lane * 4]) = make_float4(ftotal[0], ftotal[1], ftotal[2], ftotal[3]);
    else *reinterpret_cast<int4*>(&red[warp][lane * 4]) = make_int4(itotal[0], itotal[1], itotal[2], itotal[3]);
    __syncthreads();

    // element e of a row-block's 128 results: lane e / 4, register e % 4
    auto store_out = [&](int rbl, int e, float fsum, int isum) {
        const int out_rb = rb_group * rb_per_cta + rbl;
        const int el = e >> 2, i = e & 3;
        const int row = out_rb * kRbRows + (el >> 2) + 8 * (i >> 1);
        const int tok = 2 * (el & 3) + (i & 1);
        if (row < p.N && tok < p.M) {
            const float v = GROUPED ? fsum : __half2float(p.chan_scales[row]) * (float)isum;
            p.y[(int64_t)tok * p.N + row] = __float2half_rn(scale_x[tok] * v);
        }
    };
    auto add = [](float& f, int& i, int bits) {
        if (GROUPED) f += __int_as_float(bits); else i += bits;
    };

    const int t = threadIdx.x;
    if (p.cl > 1) {                                                      // ks_cta == 8: one row-block per CTA
        cg::cluster_group cluster = cg::this_cluster();
        if (t < 128) {
            float f = 0.f; int i = 0;
            for (int s = 0; s < kGemvWarps; ++s) add(f, i, red[s][t]);
            part[t] = GROUPED ? __float_as_int(f) : i;
        }
        cluster.sync();
        if (crank == 0 && t < 128) {
            float f = 0.f; int i = 0;
            for (int r = 0; r < p.cl; ++r) add(f, i, *cluster.map_shared_rank(&part[t], r));
            store_out(0, t, f, i);
        }
        // peers keep `part` alive until it has been read: a rendezvous only (relaxed arrive, plain wait)
        asm volatile("barrier.cluster.arrive.relaxed.aligned;\n\tbarrier.cluster.wait.aligned;" ::: "memory");
    } else {
        for (int idx = t; idx < rb_per_cta * 128; idx += kGemvThreads) {
            const int rbl = idx >> 7, e = idx & 127;
            float f = 0.f; int i = 0;
            for (int s = 0; s < p.ks_cta; ++s) add(f, i, red[rbl * p.ks_cta + s][e]);
            store_out(rbl, e, f, i);
        }
    }
}

// The quantisation kernel of the prefill stage (Section 3.7): x fp16 [M, K] -> xq int8 [M, K] and one fp32
// scale per token, by the same steps as above; rowsum (may be null) receives the sum of each quantised row, which
// the integer matmul needs to remove the weights' storage offset.  One CTA per token.
__global__ void __launch_bounds__(256) quantize_activations_kernel(const __half* x, signed char* xq, float* scale, int32_t* rowsum, int M, int K)
{
    __shared__ float wmax[8];
    __shared__ int wsum[8];
    __shared__ float recip;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int m = blockIdx.x;
    const uint4* row = reinterpret_cast<const uint4*>(x + (int64_t)m * K);
    float am = 0.f;
    for (int v = threadIdx.x; v < (K >> 3); v += 256) {
        const uint4 u = row[v];
        const __half2* h = reinterpret_cast<const __half2*>(&u);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 f = __half22float2(h[j]);
            am = fmaxf(am, fmaxf(fabsf(f.x), fabsf(f.y)));
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, o));
    if ((threadIdx.x & 31) == 0) wmax[threadIdx.x >> 5] = am;
    __syncthreads();
    if (threadIdx.x == 0) {
        float a = 0.f;
        for (int w = 0; w < 8; ++w) a = fmaxf(a, wmax[w]);
        const bool live = a > 0.f;
        const float safe = live ? a : 1.f;
        recip = __fdiv_rn(127.f, safe);
        scale[m] = live ? __fdiv_rn(safe, 127.f) : 1.f;
    }
    __syncthreads();
    const float r = recip;
    int total = 0;
    for (int v = threadIdx.x; v < (K >> 3); v += 256) {
        const uint4 u = row[v];
        const __half2* h = reinterpret_cast<const __half2*>(&u);
        int q8[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 f = __half22float2(h[j]);
            q8[2 * j] = quantize_one(f.x, r);
            q8[2 * j + 1] = quantize_one(f.y, r);
        }
        uint2 out;
        out.x = pack_s8x4(q8[0], q8[1], q8[2], q8[3]);
        out.y = pack_s8x4(q8[4], q8[5], q8[6], q8[7]);
        *reinterpret_cast<uint2*>(xq + (int64_t)m * K + v * 8) = out;
        total += sum_s8x4(out.x) + sum_s8x4(out.y);
    }
    if (rowsum) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
        if ((threadIdx.x & 31) == 0) wsum[threadIdx.x >> 5] = total;
        __syncthreads();
        if (threadIdx.x == 0) {
            int t = 0;
            for (int w = 0; w < 8; ++w) t += wsum[w];
            rowsum[m] = t;
        }
    }
}

}  // namespace ql
