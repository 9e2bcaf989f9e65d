// Decode kernel: y = x . W^T for M <= 8 tokens (paper Section 3.7: the memory-bound decode stage is
// served by a fully-connected kernel; Section 4.2: decode speed follows the weight bytes streamed).
//
// Work decomposition: a warp owns one row-block (16 output channels) and one K slice.  Per chunk it
// issues one 16-byte load per lane (512 contiguous bytes per warp), unpacks in registers and feeds
// mma.m16n8k16 with the weights as the 16-row operand and the <= 8 tokens as the 8 columns, so the
// fp32 accumulation and the cross-lane part of the K reduction happen inside the tensor core.  The
// K slices of a row-block are reduced across the warps of a CTA through shared memory and, when the
// split is wider than one CTA, across the CTAs of a thread-block cluster through distributed shared
// memory, always in a fixed order (deterministic, no atomics, no global scratch).
//
// Weight loads do not depend on the previous kernel in the stream, so the first batch is issued
// before griddepcontrol.wait; with programmatic dependent launch the load ramp of this kernel then
// overlaps the tail of the previous one.
#pragma once
#include <cooperative_groups.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dequant.cuh"
#include "layout.h"

namespace ql {
namespace cg = cooperative_groups;

constexpr int kGemvWarps = 8;
constexpr int kGemvThreads = kGemvWarps * 32;
constexpr int kGemvRing = 8;             // chunks prefetched per warp (cp.async ring slots)

constexpr int kGemvMaxGroup = 4;         // layers that may share one launch (same K and scheme)
constexpr int kGemvMaxBatch = 8;         // ... in the form that serves the KV heads of an attention layer (NG = 8)

// NG: capacity of the per-layer arrays.  The linear layers of a block come in groups of at most 4; the wider form is
// a separate instantiation because the longer parameter block and layer searches cost the 4-layer launches about 1 %.
template <int NG>
struct GemvParamsT {
    // One launch serves up to kGemvMaxGroup layers that read the same x (q/k/v, gate/up): their row-blocks
    // are numbered one after the other; rb_end[i] is the number of row-blocks of layers 0..i.
    const uint8_t* body[NG];  // first block of each packed body
    const __half* chan_scales[NG];   // per-channel scales (nullptr when grouped)
    __half* y[NG];            // [M, N_i]
    int32_t N[NG];
    int32_t rb_end[NG];
    int32_t n_layers;
    const __half* x;                     // [M, K]
    // Batched form (layers with DIFFERENT inputs in one launch, e.g. the score products of several KV heads): the input
    // of layer i; the plain and grouped forms set every entry to x.  Only the direct form (XDIRECT) reads it per layer.
    const __half* xl[NG];
    // XSCALE form (the V-cache product of paper Section 3.8): layer i's input is multiplied element-wise by the fp16 vector
    // xscale[i][0 .. K) on its way to the tensor core (x'[m, k] = fp16(x[m, k] * xscale[k])): the per-token scales of a
    // value cache folded into the attention probabilities without a pass of their own.
    const __half* xscale[NG];
    int32_t M, K;
    int32_t n_rb;                        // row-blocks holding at least one real row, all layers
    int32_t n_kc;                        // chunks along K
    int32_t block_bytes;
    int32_t ks_cta;                      // K slices handled inside one CTA: 1, 2, 4 or 8
    int32_t ks_cta_log2;
    int32_t cl;                          // CTAs per cluster along K (1 = no cluster)
    int32_t cps;                         // chunks per slice
    int32_t x_stride;                    // halves between tokens in the shared x slab
    int32_t x_bytes;                     // bytes of the x slab (the warp rings follow it)
    int32_t act;                         // gated form only: activation of the gate branch (QL_ACT_*)
};
using GemvParams = GemvParamsT<kGemvMaxGroup>;

// GATED: the launch serves exactly two layers of equal shape, gate (0) and up (1), whose row-blocks are dealt out
// alternately, so that a CTA (which then holds an even number of row-blocks, no cluster) has both branches of
// every output channel it owns; the epilogue writes y[0] = act(gate) * up (paper Section 3.6: element-wise
// operators of two branches fused with a fully connected operator).
template <int BITS, bool GROUPED, bool XDIRECT, bool GATED = false, bool XSCALE = false, int NG = kGemvMaxGroup>
__global__ void __launch_bounds__(kGemvThreads, 4) gemv_kernel(const GemvParamsT<NG> p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __half* xs = reinterpret_cast<__half*>(smem_raw);                   // [M][x_stride]
    __shared__ float red[kGemvWarps][128];
    __shared__ float part[128];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, c = lane & 3;
    constexpr int CHUNK_K = BITS == 4 ? 64 : 32;

    // No integer division on the way in: ks_cta is a power of two, and the position inside the cluster
    // comes from the special registers (without a cluster launch they read rank 0, cluster id = block id).
    uint32_t crank_u, rb_group_u;
    asm("mov.u32 %0, %%cluster_ctarank;" : "=r"(crank_u));
    asm("mov.u32 %0, %%clusterid.x;" : "=r"(rb_group_u));
    const int crank = (int)crank_u, rb_group = (int)rb_group_u;
    const int rb_per_cta = kGemvWarps >> p.ks_cta_log2;
    const int ks_local = warp & (p.ks_cta - 1);
    const int rb_all = rb_group * rb_per_cta + (warp >> p.ks_cta_log2);  // numbered through all layers of the launch
    const bool rb_live = rb_all < p.n_rb;
    int layer = 0;
    if (GATED) layer = rb_all & 1;
    else {
#pragma unroll
        for (int i = 1; i < NG; ++i)
            if (i < p.n_layers && rb_all >= p.rb_end[i - 1]) layer = i;
    }
    const int rb = GATED ? rb_all >> 1 : rb_all - (layer ? p.rb_end[layer - 1] : 0);   // row-block inside its layer
    const int ks = crank * p.ks_cta + ks_local;
    const int kc0 = min(ks * p.cps, p.n_kc);
    const int kc1 = rb_live ? min(kc0 + p.cps, p.n_kc) : kc0;
    const int kc_cta0 = crank * p.ks_cta * p.cps;                        // first chunk of this CTA's K range
    const int k_cta0 = kc_cta0 * CHUNK_K;
    const int k_cta1 = min((kc_cta0 + p.ks_cta * p.cps) * CHUNK_K, p.n_kc * CHUNK_K);

    // Warp-private ring of kGemvRing chunk slots filled by cp.async: the prefetch depth does not cost
    // registers and a lane reads back exactly the 16 bytes it copied.  The group scales of a whole
    // ring pass (8 chunks x 64 bytes) are fetched by one extra 16-byte copy per lane into one of two
    // per-warp pass buffers.  The steady state has no divergent branch.
    static_assert(kGemvRing == 8, "one scale copy per lane covers exactly 8 chunks");
    constexpr int WARP_SMEM = kGemvRing * 512 + (GROUPED ? 2 * 512 : 0);
    unsigned char* ring = smem_raw + p.x_bytes + warp * WARP_SMEM;
    unsigned char* sbuf = ring + kGemvRing * 512;
    const uint32_t ring_u32 = (uint32_t)__cvta_generic_to_shared(ring) + lane * 16;
    const uint32_t sbuf_u32 = (uint32_t)__cvta_generic_to_shared(sbuf) + lane * 16;
    const uint8_t* blk = p.body[layer] + ((int64_t)(rb >> 3) * p.n_kc + kc0) * p.block_bytes;
    const uint8_t* wsrc = blk + (rb & 7) * 512 + lane * 16;
    // lane L copies part (L & 3) of the scales of chunk (pass start + L / 4); the address is kept relative
    // to the weight address of the pass's first chunk (wsrc at the top of a pass)
    const int s_off = (lane >> 2) * p.block_bytes + kWeightBlockBytes - (rb & 7) * 448 + (lane & 3) * 16 - lane * 16;

    auto copy16 = [](uint32_t dst, const void* src, bool in_range) {     // out of range: reads nothing, writes zeros
        const uint32_t sz = in_range ? 16u : 0u;
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
    };
    auto commit = [] { asm volatile("cp.async.commit_group;" ::: "memory"); };

    // Weights do not depend on the previous kernel: fill the ring before waiting for it.
    if (GROUPED) copy16(sbuf_u32, wsrc + s_off, kc0 + (lane >> 2) < kc1);
#pragma unroll
    for (int d = 0; d < kGemvRing; ++d) {                                // one commit group per pair of chunks
        copy16(ring_u32 + d * 512, wsrc, kc0 + d < kc1);
        if (d & 1) commit();
        wsrc += p.block_bytes;
    }
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // Per-channel scales are weights too: the (at most 4) this thread will apply when it stores outputs are requested
    // now, so that their latency does not sit at the very end of the kernel.
    const int t = threadIdx.x;
    float pre_scale[4] = {1.f, 1.f, 1.f, 1.f};
    auto out_place = [&](int rbl, int e, int& ly, int& row, int& tok) {  // where element e of the CTA's rbl-th row-block goes
        int out_rb = rb_group * rb_per_cta + rbl;
        ly = 0;
#pragma unroll
        for (int i = 1; i < NG; ++i)
            if (i < p.n_layers && out_rb >= p.rb_end[i - 1]) ly = i;
        out_rb -= ly ? p.rb_end[ly - 1] : 0;
        const int el = e >> 2, i = e & 3;                                // lane that produced it, register index
        row = out_rb * kRbRows + (el >> 2) + 8 * (i >> 1);
        tok = 2 * (el & 3) + (i & 1);
    };
    if (!GROUPED && !GATED) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int idx = t + k * kGemvThreads;
            if (idx < (p.cl > 1 ? 128 : rb_per_cta * 128)) {
                int ly, row, tok;
                out_place(idx >> 7, idx & 127, ly, row, tok);
                if (row < p.N[ly]) pre_scale[k] = __half2float(p.chan_scales[ly][row]);
            }
        }
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // Stage this CTA's K range of x (zero beyond K) in shared memory -- or, in the direct form, read the
    // x fragments straight from global memory (they stay in L1: every row-block reuses the same slice).
    if (!XDIRECT) {
        const int span = k_cta1 - k_cta0;                                // multiple of 32
        const int vec_per_tok = span >> 3;
        for (int i = threadIdx.x; i < p.M * vec_per_tok; i += kGemvThreads) {
            const int m = i / vec_per_tok, v = i - m * vec_per_tok;
            const int k = k_cta0 + v * 8;
            uint4 val = make_uint4(0, 0, 0, 0);
            if (k < p.K) val = *reinterpret_cast<const uint4*>(p.x + (int64_t)m * p.K + k);
            *reinterpret_cast<uint4*>(xs + m * p.x_stride + v * 8) = val;
        }
        __syncthreads();
    }

    float total[4] = {0.f, 0.f, 0.f, 0.f};
    // Lanes whose token column does not exist (g >= M) read the last real token: MMA columns are
    // independent and those columns are never stored.
    const __half* xpass = XDIRECT ? p.xl[layer] + (int64_t)min(g, p.M - 1) * p.K + 8 * c + kc0 * CHUNK_K
                                  : xs + min(g, p.M - 1) * p.x_stride + 8 * c + (kc0 * CHUNK_K - k_cta0);
    static_assert(!XSCALE || (XDIRECT && BITS == 8 && !GATED), "the scaled-input form exists for int8 layers read straight from global memory");
    const __half* spass = XSCALE ? p.xscale[layer] + 8 * c + kc0 * CHUNK_K : nullptr;
    auto scale_x = [](uint4 v, const __half* sptr) {                     // fp16 products, one rounding each
        const uint4 sv = *reinterpret_cast<const uint4*>(sptr);
        const __half2* a = reinterpret_cast<const __half2*>(&v);
        const __half2* b = reinterpret_cast<const __half2*>(&sv);
        uint4 r;
        __half2* o = reinterpret_cast<__half2*>(&r);
#pragma unroll
        for (int i = 0; i < 4; ++i) o[i] = __hmul2(a[i], b[i]);
        return r;
    };
    // Direct form: the host chooses it only when K is a whole number of chunks, so every chunk in
    // [kc0, kc1) lies inside the token's row and the loads need no bounds check.
    auto load_x = [&](const __half* ptr) {
        uint4 v;
        if (!XDIRECT) v = *reinterpret_cast<const uint4*>(ptr);
        else asm volatile("ld.global.ca.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(ptr));
        return v;
    };
    // reads of the ring and of the scale buffers go through 32-bit shared-window addresses
    auto lds128 = [](uint32_t addr) {
        uint4 v;
        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
        return v;
    };
    auto lds64 = [](uint32_t addr) {
        uint2 v;
        asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
        return v;
    };
    const uint32_t sc_u32 = sbuf_u32 - lane * 16 + g * 8;                // this lane's scales inside a pass buffer
    int sflip = 0;                                                       // scale buffer of the current pass

    // one chunk: unpack in registers, feed the tensor core, apply the group scales in fp32
    auto chunk_math = [&](const uint4& w, const uint2& sc, const uint4& xa, const uint4& xb) {
        uint32_t a[4];
        if (BITS == 4) {
            const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const uint4 xv = h == 0 ? xa : xb;
                if (GROUPED) {
                    float acc[4];
                    unpack_int4_word(ww[2 * h], a);
                    mma_16816_zero(acc, a, xv.x, xv.y);
                    unpack_int4_word(ww[2 * h + 1], a);
                    mma_16816_pure(acc, a, xv.z, xv.w);
                    const __half2 s_lo = *reinterpret_cast<const __half2*>(&sc.x);          // row g:   G0, G1
                    const __half2 s_hi = *reinterpret_cast<const __half2*>(&sc.y);          // row g+8: G0, G1
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
            const uint4 xv = xa;
            unpack_int8_words(w.x, w.y, a);
            mma_16816_pure(total, a, xv.x, xv.y);
            unpack_int8_words(w.z, w.w, a);
            mma_16816_pure(total, a, xv.z, xv.w);
        }
    };

    // One pass = one trip round the ring.  Two chunks per iteration: both are read into registers and
    // their slots refilled before the math, so the two independent unpack/MMA chains interleave.
    // `checked` is a literal at both call sites: a pass called with false lies, with all its refills,
    // inside the warp's K slice and carries no range test at all.
    auto pass = [&](const bool checked, const int kc) {
#pragma unroll
        for (int d = 0; d < kGemvRing; d += 2) {
            if (checked && kc + d >= kc1) break;
            const bool two = !checked || kc + d + 1 < kc1;
            // x fragments first: their latency (L1 / shared) runs under the wait for the weights
            const __half* xk = xpass + d * CHUNK_K;
            const __half* xk1 = two ? xk + CHUNK_K : xk;                 // odd tail: stay inside the row
            uint4 x00 = load_x(xk), x10 = load_x(xk1);
            if (XSCALE) {
                x00 = scale_x(x00, spass + d * CHUNK_K);
                x10 = scale_x(x10, spass + (two ? d + 1 : d) * CHUNK_K);
            }
            uint4 x01 = x00, x11 = x10;
            if (BITS == 4) { x01 = load_x(xk + 32); x11 = load_x(xk1 + 32); }
            asm volatile("cp.async.wait_group %0;" ::"n"(kGemvRing / 2 - 1) : "memory");
            if (GROUPED && d == 0) {
                __syncwarp();                                            // scales of this pass visible; last pass's reads done
                copy16(sbuf_u32 + (sflip ^ 1) * 512, wsrc + s_off, !checked || kc + kGemvRing + (lane >> 2) < kc1);
            }
            const uint4 w0 = lds128(ring_u32 + d * 512);
            const uint4 w1 = lds128(ring_u32 + (d + 1) * 512);
            uint2 sc0 = make_uint2(0, 0), sc1 = make_uint2(0, 0);
            if (GROUPED) {
                sc0 = lds64(sc_u32 + sflip * 512 + d * 64);
                sc1 = lds64(sc_u32 + sflip * 512 + (d + 1) * 64);
            }
            copy16(ring_u32 + d * 512, wsrc, !checked || kc + d + kGemvRing < kc1);      // refill the slots just read
            copy16(ring_u32 + (d + 1) * 512, wsrc + p.block_bytes, !checked || kc + d + 1 + kGemvRing < kc1);
            commit();                                                    // (one group per pair)
            wsrc += 2 * (int64_t)p.block_bytes;
            if (two) {
                chunk_math(w0, sc0, x00, x01);
                chunk_math(w1, sc1, x10, x11);
            } else {
                chunk_math(w0, sc0, x00, x01);
            }
        }
    };
    for (int kc = kc0; kc < kc1; kc += kGemvRing) {
        // Measured: the test-free pass pays for int8 (+12 %), while the int4 form runs slower without the
        // branches that keep its four pairs apart (LM head -20 %), so int4 always takes the checked pass.
        if (BITS == 8 && kc + 2 * kGemvRing <= kc1) pass(false, kc);
        else pass(true, kc);
        xpass += kGemvRing * CHUNK_K;
        if (XSCALE) spass += kGemvRing * CHUNK_K;
        sflip ^= 1;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");

    // ---- K reduction across warps (shared memory), then across the cluster (distributed shared memory)
    *reinterpret_cast<float4*>(&red[warp][lane * 4]) = make_float4(total[0], total[1], total[2], total[3]);
    __syncthreads();

    auto store_out = [&](int rbl, int e, float v, float scale) {
        int ly, row, tok;
        out_place(rbl, e, ly, row, tok);
        if (row < p.N[ly] && tok < p.M) {
            if (!GROUPED) v *= scale;
            p.y[ly][(int64_t)tok * p.N[ly] + row] = __float2half_rn(v);
        }
    };

    if (p.cl > 1) {                                                      // ks_cta == 8: one row-block per CTA
        cg::cluster_group cluster = cg::this_cluster();
        if (t < 128) {
            float v = 0.f;
            for (int s = 0; s < kGemvWarps; ++s) v += red[s][t];
            part[t] = v;
        }
        // partial sums published to the cluster: every CTA releases, only the reading CTA has to acquire
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        if (crank == 0) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
        else asm volatile("barrier.cluster.wait.aligned;" ::: "memory");
        if (crank == 0 && t < 128) {
            float v = 0.f;
            for (int r = 0; r < p.cl; ++r) v += *cluster.map_shared_rank(&part[t], r);
            store_out(0, t, v, pre_scale[0]);
        }
        // peers keep `part` alive until it has been read: a rendezvous only, nothing is handed over, so the arrive
        // needs no release and the wait no acquire
        asm volatile("barrier.cluster.arrive.relaxed.aligned;\n\tbarrier.cluster.wait.aligned;" ::: "memory");
    } else if (GATED) {
        for (int idx = t; idx < (rb_per_cta >> 1) * 128; idx += kGemvThreads) {
            const int pr = idx >> 7, e = idx & 127;                      // pair of row-blocks (gate, up), element
            float gv = 0.f, uv = 0.f;
            for (int s = 0; s < p.ks_cta; ++s) { gv += red[(2 * pr) * p.ks_cta + s][e]; uv += red[(2 * pr + 1) * p.ks_cta + s][e]; }
            const int out_rb = ((rb_group * rb_per_cta) >> 1) + pr;
            const int el = e >> 2, i = e & 3;
            const int row = out_rb * kRbRows + (el >> 2) + 8 * (i >> 1), tok = 2 * (el & 3) + (i & 1);
            if (row < p.N[0] && tok < p.M) {
                if (!GROUPED) { gv *= __half2float(p.chan_scales[0][row]); uv *= __half2float(p.chan_scales[1][row]); }
                p.y[0][(int64_t)tok * p.N[0] + row] = __float2half_rn(gate_activation(gv, p.act) * uv);
            }
        }
    } else {
        if (GROUPED) {
            for (int idx = t; idx < rb_per_cta * 128; idx += kGemvThreads) {
                const int rbl = idx >> 7, e = idx & 127;
                float v = 0.f;
                for (int s = 0; s < p.ks_cta; ++s) v += red[rbl * p.ks_cta + s][e];
                store_out(rbl, e, v, 1.f);
            }
        } else {
#pragma unroll
            for (int k = 0; k < 4; ++k) {                                // rb_per_cta <= 8: at most 4 elements per thread
                const int idx = t + k * kGemvThreads;
                if (idx >= rb_per_cta * 128) break;
                const int rbl = idx >> 7, e = idx & 127;
                float v = 0.f;
                for (int s = 0; s < p.ks_cta; ++s) v += red[rbl * p.ks_cta + s][e];
                store_out(rbl, e, v, pre_scale[k]);
            }
        }
    }
}

}  // namespace ql
