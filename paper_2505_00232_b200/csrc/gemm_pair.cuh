// Prefill kernel, CTA-pair form (tcgen05 cta_group::2): two CTAs of a cluster compute one 256 x 256 output
// tile -- 256 output channels (two row super-blocks, one per CTA) x 256 tokens -- with one MMA issued by
// the leader CTA.  Each CTA stages only its own 128 channels of weights and its own 128 tokens of x, so
// the x traffic from L2 and the shared-memory operand reads per flop are half of the single-CTA kernel's
// (paper Section 3.7: the prefill stage is compute-bound; the point here is to keep it that way).
//
// Roles per CTA are those of gemm.cuh.  Cross-CTA protocol (every CTA issues its own loads; nothing is loaded for a peer):
//   * dequantise warps arrive on their own CTA's afull barrier (a warp dequantises only after its CTA's
//     TMA data landed, so "A tile written" implies "x half landed"); in the peer CTA one spare warp per A
//     slot relays each completed afull phase to the leader with ONE remote arrive, on the leader's
//     afull barrier (17 arrivals there: its own 16 warps and the relay);
//   * the leader's tcgen05.commit signals the empty / tfull barriers of BOTH CTAs (cluster mask 3 on the commit);
//   * the epilogue warps of both CTAs arrive on the leader's tempty barrier (8 arrivals);
//   * cluster barriers bracket the kernel so that no CTA exits while its peer can still touch it.
#pragma once
#include "gemm.cuh"

namespace ql {

// Shared memory: a deep ring of TMA stages (this CTA's x half + packed weights) that covers the load
// latency, and a short ring of dequantised A tiles (produced on chip, consumed a few hundred cycles later).
// Warp roles: 0 producer, 1 MMA issuer, 2..22 except ids with (id % 4 == 1): 16 dequantise warps, 5/9/13/17/21: relays, 24..27 epilogue.
constexpr int kPairFirstEpilogueWarp = 24;
constexpr int kPairThreads = 28 * 32;

// TB = token blocks (of 256) per tile.  With TB = 2 every dequantised A slot feeds two MMA groups (two
// accumulators of 256 columns fill the tensor memory, so the epilogue is no longer hidden under the next
// tile): half the dequantise work and half the A-slot hand-offs per flop.
// I8: the integer form (int8 activations, kind::i8): a k-step is 128 k, i.e. again 128 bytes per tile row.
template <int BITS, int TB, bool I8 = false>
struct GemmPairSmem {
    static constexpr int kKStep = I8 ? 128 : kGemmKStep;
    static constexpr int kXBlockBytes = 128 * 128;                       // this CTA's 128 tokens x one k-step of one token block
    static constexpr int kXBytes = TB * kXBlockBytes;
    static constexpr int kWpkStride = I8 ? (BITS == 4 ? 8192 : 16384) : (BITS == 4 ? 5120 : 8192);   // packed block(s) of one k-step
    static constexpr int kStageBytes = kXBytes + kWpkStride;
    static constexpr int kStages = I8 ? (BITS == 4 ? 6 : 4) : TB == 2 ? 4 : (BITS == 4 ? 6 : 5);
    static constexpr int kASlots = (I8 || TB == 2) ? 4 : 5;              // one relay warp per slot (spare warps 5, 9, 13, 17, 21)
    static constexpr int kAOffset = kStages * kStageBytes;
    static constexpr int kBarOffset = kAOffset + kASlots * kGemmATileBytes;
    static constexpr int kTotal = kBarOffset + 512 + 1024;               // barriers + alignment slack
};

// Work unit t of the grid: a whole tile (t < n_whole) or one K part of a split tile.  Whole tiles fill the
// full rounds of the persistent grid; the tiles of the last, partial round are split so that it is short.
struct PairUnit {
    int tile, part, parts, step0, nsteps, slab;
};
__device__ __forceinline__ PairUnit pair_unit(int t, const GemmParams& p)
{
    PairUnit u;
    if (t < p.n_whole) {
        u.tile = t; u.part = 0; u.parts = 1; u.step0 = 0; u.nsteps = p.n_ksteps; u.slab = 0;
    } else {
        const int v = t - p.n_whole;
        u.slab = v / p.split;                                            // index among the split tiles (scratch slot)
        u.tile = p.n_whole + u.slab;
        u.part = v - u.slab * p.split;
        u.parts = p.split;
        u.nsteps = p.n_ksteps / p.split;
        u.step0 = u.part * u.nsteps;
    }
    return u;
}

// Row super-block numbered through all layers of the launch -> (layer, row super-block inside it).
__device__ __forceinline__ int pair_layer(const GemmParams& p, int& rsb)
{
    int ly = 0;
#pragma unroll
    for (int i = 1; i < kGemmMaxGroup; ++i)
        if (i < p.n_layers && rsb >= p.rsb_end[i - 1]) ly = i;
    rsb -= ly ? p.rsb_end[ly - 1] : 0;
    return ly;
}

// GATED (TB == 1 only): the launch serves two layers of equal shape, gate (0) and up (1).  A cluster runs the gate
// tile and the up tile of the same (row super-block pair, token block) back to back into its two accumulators.
// While the up tile's main loop runs, the epilogue warps turn the finished gate accumulator into act(gate) in
// place (tensor memory load, activation, tensor memory store); when the up tile is complete they write
// fp16(act(gate) * up), the only tensor that ever goes to memory (paper Section 3.6), and free both accumulators.
// Work unit t then counts (row super-block pair, token block) positions of ONE layer; every unit is two tiles.
// I8 (TB == 1, per-channel schemes, not gated): x_map describes int8 activations; the weight integers go to the A
// tile unconverted (RepackLane), the MMAs are kind::i8 with an s32 accumulator, and the epilogue removes the storage
// offset (off * sum of the token's quantised row) and applies both scales (paper Section 3.7, prefill stage).
template <int BITS, bool GROUPED, int TB, bool GATED = false, bool I8 = false>
__global__ void __launch_bounds__(kPairThreads, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap x_map, const GemmParams p)
{
    static_assert(!GATED || TB == 1, "the gated form uses both accumulators for one output tile");
    static_assert(!I8 || (TB == 1 && !GATED && !GROUPED), "the integer form: per-channel scales, 256-token tiles");
    using S = GemmPairSmem<BITS, TB, I8>;
    constexpr int NS = S::kStages;
    constexpr int NA = S::kASlots;
    constexpr int BN = 256;                                              // tokens per MMA (128 per CTA)
    constexpr int TILE_N = BN * TB;                                      // tokens per tile
    extern __shared__ unsigned char smem_dyn[];
    const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
    auto xs_addr = [&](int s) { return base + s * S::kStageBytes; };
    auto wpk_addr = [&](int s) { return base + s * S::kStageBytes + S::kXBytes; };
    auto wpk_ptr = [&](int s) { return base_ptr + s * S::kStageBytes + S::kXBytes; };
    auto a_addr = [&](int a) { return base + S::kAOffset + a * kGemmATileBytes; };
    auto a_ptr = [&](int a) { return base_ptr + S::kAOffset + a * kGemmATileBytes; };
    const uint32_t bar0 = base + S::kBarOffset;
    auto full_bar = [&](int s) { return bar0 + 8 * s; };                 // local: this CTA's TMA data landed
    auto empty_bar = [&](int s) { return bar0 + 8 * (NS + s); };         // local, signalled by the leader's commit
    auto afull_bar = [&](int a) { return bar0 + 8 * (2 * NS + a); };     // local: this CTA's A tile written
    auto tfull_bar = [&](int b) { return bar0 + 8 * (2 * NS + 3 * NA + b); };        // local, signalled by the leader's commit
    auto tempty_bar = [&](int b) { return bar0 + 8 * (2 * NS + 3 * NA + 2 + b); };   // leader: both epilogues drained buffer b
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + S::kBarOffset + 8 * (2 * NS + 3 * NA + 4));
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();                             // 0 = leader
    const int KS = p.split;
    // Tile t = (row-super-block pair t / n_mblk, token block t % n_mblk): clusters that run side by side share
    // weight blocks and read different x tiles, which spreads the L2 traffic over more lines.
    const int n_mblk = (p.M + TILE_N - 1) / TILE_N;
    const int first_tile = blockIdx.x >> 1, tile_stride = gridDim.x >> 1;   // tile = (rsb pair, token block)
    // The j-th tile this cluster runs: work unit t and, in the gated form, which of the two layers.
    auto tile_of = [&](int j, int& t, int& gl) {
        t = first_tile + (GATED ? j >> 1 : j) * tile_stride;
        gl = GATED ? (j & 1) : 0;
        return t < p.n_tiles;
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < NA; ++a) {
            mbar_init(afull_bar(a), kGemmDequantWarps + (rank == 0 ? 1 : 0));   // leader: + the peer's relay lane
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(tfull_bar(b), 1);
            mbar_init(tempty_bar(b), 2 * kGemmEpilogueWarps);
        }
        abort_flag[0] = 0;                                               // [0] abort, [1] abort of the exit drain,
        abort_flag[1] = 0;                                               // [2], [3] "past griddepcontrol.wait" (see wait_expired)
        abort_flag[2] = 0;
        abort_flag[3] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc_pair(smem_u32((const void*)tmem_slot), 2 * BN);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                                  // both CTAs' barriers exist before any remote arrive
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ producer (each CTA feeds itself)
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&x_map) : "memory");
            constexpr int CHUNKS = S::kKStep / (BITS == 4 ? 64 : 32);      // packed blocks per k-step
            int s = 0, issued = 0;
            uint32_t par = 1;
            bool waited_dep = false, ok = true;
            int t, gl;
            for (int j = 0; tile_of(j, t, gl) && ok; ++j) {
                const PairUnit u = pair_unit(t, p);
                const int tile = u.tile, step0 = u.step0, n_steps = u.nsteps;
                int rsb = 2 * (tile / n_mblk) + (int)rank;
                const int ly = GATED ? gl : pair_layer(p, rsb);
                const int m0 = (tile % n_mblk) * TILE_N + 128 * (int)rank;   // this CTA's 128 tokens of each token block
                const uint8_t* wsrc = p.lbody[ly] + (int64_t)rsb * p.n_kc * p.block_bytes;
                for (int it = 0; it < n_steps; ++it) {
                    if (!mbar_wait_hot(empty_bar(s), par, abort_flag, 0x100 + s)) { ok = false; break; }
                    const int kc = (step0 + it) * CHUNKS;
                    const int nblk = min(CHUNKS, p.n_kc - kc);
                    const uint32_t wbytes = (uint32_t)nblk * p.block_bytes;
                    mbar_expect_tx(full_bar(s), wbytes + S::kXBytes);
                    bulk_copy_g2s(wpk_addr(s), wsrc + (int64_t)kc * p.block_bytes, wbytes, full_bar(s));
                    if (!waited_dep) {
                        asm volatile("griddepcontrol.wait;" ::: "memory");
                        waited_dep = true;
                        abort_flag[2] = 1;                               // from here on, waiting counts against the time limit
                        abort_flag[3] = 1;
                    }
#pragma unroll
                    for (int tb = 0; tb < TB; ++tb)
                        tma_load_2d(xs_addr(s) + tb * S::kXBlockBytes, &x_map, (step0 + it) * S::kKStep, m0 + tb * BN, full_bar(s));
                    ++issued;
                    if (++s == NS) { s = 0; par ^= 1; }
                }
            }
            if (*abort_flag) {
                for (int j = max(0, issued - NS); j < issued; ++j)
                    mbar_wait(full_bar(j % NS), (j / NS) & 1, abort_flag + 1, 0);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        // The whole warp runs the loop (warp-uniform control flow: counters and descriptors stay in uniform
        // registers); one elected lane issues.
        if (rank == 0) {
            // f16 x f16 -> f32, or (integer form) u8 weights x s8 activations -> s32; both operands K-major, M = 256 per pair
            constexpr uint32_t idesc = (I8 ? (2u << 4) | (1u << 10) : (1u << 4)) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
            const uint32_t a_lo0 = umma_desc_lo(a_addr(0)), b_lo0 = umma_desc_lo(xs_addr(0));
            int s = 0, a = 0;
            uint32_t apar = 0;
            bool ok = true;
            int t, gl;
            for (int j = 0; tile_of(j, t, gl) && ok; ++j) {
                // TB = 1: two accumulators alternate; TB = 2: both are used by every tile
                const int buf = TB == 1 ? (j & 1) : 0;
                const uint32_t use = TB == 1 ? (uint32_t)(j >> 1) : (uint32_t)j;
                const int n_steps = pair_unit(t, p).nsteps;
                if (!mbar_wait(tempty_bar(buf), (use & 1) ^ 1, abort_flag, 0x800 + buf)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + (uint32_t)(buf * BN);
                for (int it = 0; it < n_steps; ++it) {
                    // 16 local dequantise warps + the peer's relay lane: both A tiles written, both x halves landed
                    if (!mbar_wait_hot(afull_bar(a), apar, abort_flag, 0x300 + a)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_lo = a_lo0 + (uint32_t)a * (kGemmATileBytes >> 4);
                    const uint32_t b_lo = b_lo0 + (uint32_t)s * (S::kStageBytes >> 4);
                    if (elect_one()) {
#pragma unroll
                        for (int tb = 0; tb < TB; ++tb) {
                            const uint32_t d = tmem_d + (uint32_t)(tb * BN), bl = b_lo + (uint32_t)tb * (S::kXBlockBytes >> 4);
                            if (I8) umma_i8_pair_lo(d, a_lo, bl, idesc, it > 0 ? 1u : 0u);
                            else umma_f16_pair_lo(d, a_lo, bl, idesc, it > 0 ? 1u : 0u);
#pragma unroll
                            for (int k4 = 1; k4 < 4; ++k4) {             // +32 bytes along K inside the swizzle row
                                if (I8) umma_i8_pair_lo(d, a_lo + 2 * k4, bl + 2 * k4, idesc, 1u);
                                else umma_f16_pair_lo(d, a_lo + 2 * k4, bl + 2 * k4, idesc, 1u);
                            }
                        }
                        umma_commit_pair(empty_bar(s));                  // frees the TMA stage and the A slot in both CTAs
                    }
                    __syncwarp();
                    if (++s == NS) s = 0;
                    if (++a == NA) { a = 0; apar ^= 1; }
                }
                if (ok && elect_one()) umma_commit_pair(tfull_bar(buf));
                __syncwarp();
            }
        }
    } else if (warp < kPairFirstEpilogueWarp) {
        // ------------------------------------------------------------------ dequantise
        // The MMA-issuing warp (warp 1) lives on scheduler 1 (warp id % 4); dequantise work is kept off
        // that scheduler so that the issuing thread is never queued behind ALU-heavy warps.
        if ((warp & 3) == 1 || warp == 23) {
            // Spare warps 5, 9, 13, 17, 21, 23 of the PEER CTA relay "A slot ready" to the leader: one warp per A
            // slot (a waiting warp is suspended as a whole, so relay lanes of one warp would serialise),
            // one remote arrive per slot phase on the leader's afull barrier.
            const int a = warp == 23 ? 5 : (warp - 5) >> 2;
            if (rank != 0 && lane == 0 && a < NA) {
                uint32_t apar = 0;
                int total_steps = 0;
                int t, gl;
                for (int j = 0; tile_of(j, t, gl); ++j) total_steps += pair_unit(t, p).nsteps;
                for (int g = a; g < total_steps; g += NA) {
                    if (!mbar_wait(afull_bar(a), apar, abort_flag, 0xA00 + a)) break;
                    mbar_arrive_remote(afull_bar(a), 0);
                    apar ^= 1;
                }
            }
        } else {                                                         // 16 dequantise warps
        const DequantLane dq(warp - 2 - ((warp - 1) >> 2), lane);
        const RepackLane rp(warp - 2 - ((warp - 1) >> 2), lane);
        int s = 0, a = 0;
        uint32_t par = 0;
        // A slot a was last read by the MMAs of step (gstep - NA); their retirement is the phase of the
        // empty barrier of that step's TMA stage.
        int s_old = 0;
        uint32_t par_old = 0;
        bool ok = true;
        int gstep = 0;
        int t, gl;
        for (int j = 0; tile_of(j, t, gl) && ok; ++j) {
            const int n_steps = pair_unit(t, p).nsteps;
            for (int it = 0; it < n_steps; ++it, ++gstep) {
                if (!mbar_wait(full_bar(s), par, abort_flag, 0x400 + s)) { ok = false; break; }
                if (gstep >= NA) {
                    if (!mbar_wait(empty_bar(s_old), par_old, abort_flag, 0xB00 + s_old)) { ok = false; break; }
                    if (++s_old == NS) { s_old = 0; par_old ^= 1; }
                }
                if (I8) rp.template step<BITS>(wpk_ptr(s), a_ptr(a));
                else dq.template step<BITS, GROUPED>(wpk_ptr(s), a_ptr(a));
                fence_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(afull_bar(a));
                if (++s == NS) { s = 0; par ^= 1; }
                if (++a == NA) a = 0;
            }
        }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (each CTA stores its 128 channels)
        const int quarter = warp & 3;
        bool ok = true;
        int t, gl;
        for (int j = 0; tile_of(j, t, gl) && ok; ++j) {
            const int buf = TB == 1 ? (j & 1) : 0;
            const uint32_t use = TB == 1 ? (uint32_t)(j >> 1) : (uint32_t)j;
            const PairUnit u = pair_unit(t, p);
            const int tile = u.tile, part = u.part;
            int rsb = 2 * (tile / n_mblk) + (int)rank;
            const int ly = GATED ? 0 : pair_layer(p, rsb);
            const int m0 = (tile % n_mblk) * TILE_N, N = p.lN[ly];
            if (!mbar_wait<true>(tfull_bar(buf), use & 1, abort_flag, 0x500 + buf)) { ok = false; break; }
            tc_fence_after();
            const int n = rsb * kRsbRows + quarter * 32 + lane;
            if (GATED) {
                // accumulator 0 holds the gate projection of this tile, accumulator 1 the up projection
                float sg = 1.f, su = 1.f;
                if (!GROUPED && n < N) { sg = __half2float(p.lscales[0][n]); su = __half2float(p.lscales[1][n]); }
                const uint32_t tg = tmem_base + ((uint32_t)(quarter * 32) << 16);
                const int m_left = min(TILE_N, p.M - m0);
                if (gl == 0) {
                    // The gate accumulator is complete while the up tile's main loop runs: apply scale and activation
                    // in place now, so that only a product is left to do once the up tile is complete.
#pragma unroll 1
                    for (int cc = 0; cc < m_left; cc += 16) {
                        uint32_t rg[16];
                        tmem_ld16(tg + (uint32_t)cc, rg);
#pragma unroll
                        for (int q = 0; q < 16; ++q) rg[q] = __float_as_uint(gate_activation(__uint_as_float(rg[q]) * sg, p.act));
                        tmem_st16(tg + (uint32_t)cc, rg);
                    }
                    tc_fence_before();
                    continue;
                }
                __half* yrow = p.ly[0] + (int64_t)m0 * N + n;
#pragma unroll 1
                for (int cc = 0; cc < m_left; cc += 16) {
                    uint32_t rg[16], ru[16];
                    tmem_ld16(tg + (uint32_t)cc, rg);
                    tmem_ld16(tg + (uint32_t)(BN + cc), ru);
                    if (n < N) {
#pragma unroll
                        for (int q = 0; q < 16; ++q)
                            if (cc + q < m_left)
                                yrow[(int64_t)(cc + q) * N] = __float2half_rn(__uint_as_float(rg[q]) * (__uint_as_float(ru[q]) * su));
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) { mbar_arrive_remote(tempty_bar(0), 0); mbar_arrive_remote(tempty_bar(1), 0); }
                continue;
            }
            if (I8) {
                // acc = sum (q + off) * xq: remove off * (sum of the token's quantised row), then both scales
                constexpr int OFF = BITS == 4 ? 8 : 128;
                const float sn = n < N ? __half2float(p.lscales[ly][n]) : 0.f;
                const uint32_t ta = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * BN);
                __half* yr = p.ly[ly] + (int64_t)m0 * N + n;
                const int ml = min(TILE_N, p.M - m0);
#pragma unroll 1
                for (int cc = 0; cc < ml; cc += 16) {
                    uint32_t r[16];
                    // the 16 tokens' scales and row sums first (whole 64-byte lines; the arrays are padded to whole tiles)
                    float sx[16];
                    int rs[16];
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        const float4 f = __ldg(reinterpret_cast<const float4*>(p.a8_scale + m0 + cc) + v);
                        const int4 i = __ldg(reinterpret_cast<const int4*>(p.a8_rowsum + m0 + cc) + v);
                        sx[4 * v] = f.x; sx[4 * v + 1] = f.y; sx[4 * v + 2] = f.z; sx[4 * v + 3] = f.w;
                        rs[4 * v] = i.x; rs[4 * v + 1] = i.y; rs[4 * v + 2] = i.z; rs[4 * v + 3] = i.w;
                    }
                    tmem_ld16(ta + (uint32_t)cc, r);
                    if (n < N) {
#pragma unroll
                        for (int q = 0; q < 16; ++q)
                            if (cc + q < ml) {
                                const float v = (float)((int)r[q] - OFF * rs[q]);
                                yr[(int64_t)(cc + q) * N] = __float2half_rn(sx[q] * (sn * v));
                            }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_remote(tempty_bar(buf), 0);
                continue;
            }
            float scale = 1.f;
            if (!GROUPED && n < N) scale = __half2float(p.lscales[ly][n]);
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * BN);
            __half* yrow = p.ly[ly] + (int64_t)m0 * N + n;
            const int m_left = min(TILE_N, p.M - m0);                    // accumulator column = token m0 + column
            if (u.parts == 1) {
#pragma unroll 1
                for (int cc = 0; cc < m_left; cc += 16) {
                    uint32_t r[16];
                    tmem_ld16(taddr + (uint32_t)cc, r);
                    if (n < N) {
#pragma unroll
                        for (int q = 0; q < 16; ++q)
                            if (cc + q < m_left) yrow[(int64_t)(cc + q) * N] = __float2half_rn(__uint_as_float(r[q]) * scale);
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_remote(tempty_bar(buf), 0);
            } else {
                // K-split tile: park this part's fp32 accumulator in scratch ([token][channel], so a warp
                // writes 128 contiguous bytes per token), free the accumulator, then count arrivals; the
                // last part to arrive adds all parts in part order (fixed order, no float atomics) and stores y.
                float* slab = p.scratch + (((int64_t)u.slab * KS + part) * 2 + rank) * (BN * 128) + quarter * 32 + lane;
#pragma unroll 1
                for (int cc = 0; cc < m_left; cc += 16) {
                    uint32_t r[16];
                    tmem_ld16(taddr + (uint32_t)cc, r);
#pragma unroll
                    for (int q = 0; q < 16; ++q) __stcg(slab + (cc + q) * 128, __uint_as_float(r[q]));
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_remote(tempty_bar(buf), 0);
                __threadfence();
                __syncwarp();
                unsigned int old = 0;
                unsigned int* cnt = p.counters + (u.slab * 2 + rank) * 4 + quarter;
                if (lane == 0) old = atomicAdd(cnt, 1u);
                old = __shfl_sync(0xffffffffu, old, 0);
                if ((int)old == KS - 1) {
                    __threadfence();
                    const float* first = p.scratch + (((int64_t)u.slab * KS) * 2 + rank) * (BN * 128) + quarter * 32 + lane;
                    // all loads of a 16-token batch (every part) are issued before the ordered sum, so that
                    // the L2 round trips overlap
#pragma unroll 1
                    for (int cc = 0; cc < m_left; cc += 16) {
                        float acc[16];
#pragma unroll
                        for (int q = 0; q < 16; ++q) acc[q] = __ldcg(first + (cc + q) * 128);
                        if (KS == 2) {
                            float v[16];
#pragma unroll
                            for (int q = 0; q < 16; ++q) v[q] = __ldcg(first + (int64_t)2 * (BN * 128) + (cc + q) * 128);
#pragma unroll
                            for (int q = 0; q < 16; ++q) acc[q] += v[q];
                        } else {
                            float v1[16], v2[16], v3[16];
#pragma unroll
                            for (int q = 0; q < 16; ++q) {
                                v1[q] = __ldcg(first + (int64_t)2 * (BN * 128) + (cc + q) * 128);
                                v2[q] = __ldcg(first + (int64_t)4 * (BN * 128) + (cc + q) * 128);
                                v3[q] = __ldcg(first + (int64_t)6 * (BN * 128) + (cc + q) * 128);
                            }
#pragma unroll
                            for (int q = 0; q < 16; ++q) acc[q] = ((acc[q] + v1[q]) + v2[q]) + v3[q];
                        }
                        if (n < N) {
#pragma unroll
                            for (int q = 0; q < 16; ++q)
                                if (cc + q < m_left) yrow[(int64_t)(cc + q) * N] = __float2half_rn(acc[q] * scale);
                        }
                    }
                    if (lane == 0) *cnt = 0;                             // ready for the next launch
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                                  // the peer no longer reads this CTA's memory
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, 2 * BN);
    }
}

// K split of every tile: used when there are fewer tiles than half the clusters, so that the whole GPU works
// on skinny layers.  Units never exceed the cluster count, which bounds the scratch (see gemm_pair_scratch_bytes).
inline int gemm_pair_split(int tiles /* of the last, partial round */, int n_ksteps, int num_sms, bool have_scratch)
{
    if (!have_scratch) return 1;
    const int clusters = num_sms / 2;
    int split = 1;
    if (tiles == 0) return 1;
    if (gemm_config().force_split > 0) split = gemm_config().force_split;
    else if (tiles * 4 <= clusters) split = 4;
    else if (tiles * 2 <= clusters) split = 2;
    while (split > 1 && (n_ksteps % split || n_ksteps / split < 8 || tiles * split > clusters)) split >>= 1;
    return split == 3 ? 2 : split;                                       // the kernel adds 2 or 4 parts
}
// (at least 40 MB: the same buffer holds the int8 activations of the integer form, up to M x K = 2048 x 14336, and
// the two projections of the unfused gating route)
inline size_t gemm_pair_scratch_bytes(int num_sms) { return std::max<size_t>((size_t)(num_sms / 2) * 2 * 256 * 128 * sizeof(float), (size_t)40 << 20); }
// (the tensor-memory form counts arrivals per (tile, CTA, 16 epilogue warps) for up to num_sms / 4 split tiles)
inline size_t gemm_pair_counter_count(int num_sms) { return (size_t)(num_sms / 2) * 32; }

// The layers of one launch: all read the same x and agree in K and scheme; each has an even number of row
// super-blocks.  L is the layout of the first one (K, chunking and scheme are taken from it).
struct GemmPairLayers {
    int n;
    const Layout* L[kGemmMaxGroup];
    const uint8_t* blob[kGemmMaxGroup];
    void* y[kGemmMaxGroup];
    const CUtensorMap* wmap[kGemmMaxGroup];      // packed body as 64-byte rows (tensor-memory form), or nullptr
    int n_rsb() const { int t = 0; for (int i = 0; i < n; ++i) t += L[i]->n_rsb; return t; }
};

// act < 0: the plain form.  act >= 0 (TB == 1): the gated form, set = {gate, up} of equal shape, y[0] the output.
// a8_scale != nullptr: the integer form; x is then the int8 activations, a8_scale / a8_rowsum their per-token arrays.
template <int BITS, bool GROUPED, int TB, bool GATED = false, bool I8 = false>
ql_status gemm_pair_launch(const GemmPairLayers& set, const void* x, int M, cudaStream_t st, int device,
                           bool pdl, int num_sms, float* scratch, unsigned int* counters, int act = -1,
                           const float* a8_scale = nullptr, const int32_t* a8_rowsum = nullptr)
{
    using S = GemmPairSmem<BITS, TB, I8>;
    const Layout& L = *set.L[0];
    CUtensorMap map;
    if (!x_tensor_map(x, L.K, M, 128, &map, I8 ? 1 : 2)) return QL_ERR_CUDA;
    auto kern = gemm_pair_kernel<BITS, GROUPED, TB, GATED, I8>;
    static std::atomic<bool> attr_set[64];
    if (device >= 0 && device < 64 && !attr_set[device]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, S::kTotal) != cudaSuccess) {
            cudaGetLastError();
            return QL_ERR_CUDA;
        }
        attr_set[device] = true;
    }
    GemmParams prm{};
    int n_rsb = 0;
    for (int i = 0; i < set.n; ++i) {
        const Layout& Li = *set.L[i];
        prm.lbody[i] = set.blob[i] + Li.body_offset;
        prm.lscales[i] = Li.grouped ? nullptr : reinterpret_cast<const __half*>(set.blob[i] + Li.chan_scale_offset);
        prm.ly[i] = static_cast<__half*>(set.y[i]);
        prm.lN[i] = Li.N;
        n_rsb += Li.n_rsb;
        prm.rsb_end[i] = n_rsb;
    }
    prm.n_layers = set.n;
    prm.act = act;
    if (GATED) n_rsb = L.n_rsb;                                          // work units count positions of one layer
    prm.M = M; prm.N = L.N; prm.K = L.K;
    prm.n_kc = L.n_kc; prm.block_bytes = L.block_bytes;
    prm.n_ksteps = (L.K + S::kKStep - 1) / S::kKStep;
    prm.a8_scale = a8_scale; prm.a8_rowsum = a8_rowsum;
    prm.n_rsb = n_rsb;
    const int tiles = (n_rsb / 2) * ((M + 256 * TB - 1) / (256 * TB));
    // whole tiles fill the full rounds of the persistent grid; the tiles of the last partial round are split
    const int clusters = num_sms / 2;
    // (splitting the tail of a multi-round schedule was measured and does not pay: the exposed scratch
    // reduction costs what the shorter last round saves; only single-round layers are split)
    const int tail = tiles < clusters ? tiles : 0;
    prm.split = (TB == 1 && !GATED && !I8) ? gemm_pair_split(tail, prm.n_ksteps, num_sms, scratch != nullptr) : 1;
    prm.n_whole = prm.split > 1 ? tiles - tail : tiles;
    prm.scratch = scratch;
    prm.counters = counters;
    prm.n_tiles = prm.n_whole + (tiles - prm.n_whole) * prm.split;       // work units
    const int n_clusters = prm.n_tiles < num_sms / 2 ? prm.n_tiles : num_sms / 2;

    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(2 * n_clusters);
    cfg.blockDim = dim3(kPairThreads);
    cfg.dynamicSmemBytes = S::kTotal;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 2 : 1;
    if (cudaLaunchKernelEx(&cfg, kern, map, prm) != cudaSuccess) {
        cudaGetLastError();
        return QL_ERR_CUDA;
    }
    return QL_OK;
}

// The pair kernel needs an even number of row super-blocks and enough tokens to fill a 256-wide tile.
inline bool gemm_pair_applicable(const Layout& L, int M)
{
    return gemm_config().pair && (L.n_rsb % 2) == 0 && M > 128;
}

inline ql_status gemm_pair_forward(const GemmPairLayers& set, const void* x, int M, cudaStream_t st,
                                   int device, bool pdl, int num_sms, float* scratch, unsigned int* counters)
{
    // Token blocks per tile: a step of a 512-token tile costs two steps of a 256-token tile (the kernel is
    // bound by the tensor pipe and its operand traffic, not by dequantisation), so the wider tile only pays
    // where it saves rounds of the persistent grid.
    const Layout& L = *set.L[0];
    int tb = gemm_config().force_tb;
    if (tb == 0) {
        const int clusters = num_sms / 2, pairs = set.n_rsb() / 2;
        const int tiles1 = pairs * ((M + 255) / 256), tiles2 = pairs * ((M + 511) / 512);
        const int rounds1 = (tiles1 + clusters - 1) / clusters, rounds2 = (tiles2 + clusters - 1) / clusters;
        tb = (tiles1 >= clusters && 2 * rounds2 <= rounds1) ? 2 : 1;
    }
    if (tb == 2 && M > 256) {
        if (L.bits == 8) return gemm_pair_launch<8, false, 2>(set, x, M, st, device, pdl, num_sms, scratch, counters);
        if (L.grouped) return gemm_pair_launch<4, true, 2>(set, x, M, st, device, pdl, num_sms, scratch, counters);
        return gemm_pair_launch<4, false, 2>(set, x, M, st, device, pdl, num_sms, scratch, counters);
    }
    if (L.bits == 8) return gemm_pair_launch<8, false, 1>(set, x, M, st, device, pdl, num_sms, scratch, counters);
    if (L.grouped) return gemm_pair_launch<4, true, 1>(set, x, M, st, device, pdl, num_sms, scratch, counters);
    return gemm_pair_launch<4, false, 1>(set, x, M, st, device, pdl, num_sms, scratch, counters);
}

// Integer form (per-channel schemes, K a multiple of 128): xq int8 [M, K] with per-token scale and row sum.
inline ql_status gemm_pair_forward_i8(const GemmPairLayers& set, const void* xq, const float* scale, const int32_t* rowsum, int M,
                                      cudaStream_t st, int device, bool pdl, int num_sms)
{
    const Layout& L = *set.L[0];
    if (L.bits == 8) return gemm_pair_launch<8, false, 1, false, true>(set, xq, M, st, device, pdl, num_sms, nullptr, nullptr, -1, scale, rowsum);
    return gemm_pair_launch<4, false, 1, false, true>(set, xq, M, st, device, pdl, num_sms, nullptr, nullptr, -1, scale, rowsum);
}

// Gated form: set = {gate, up}, both pair-applicable and of equal shape; y[0] receives act(gate) * up.
inline ql_status gemm_pair_forward_gated(const GemmPairLayers& set, const void* x, int M, int act, cudaStream_t st,
                                         int device, bool pdl, int num_sms)
{
    const Layout& L = *set.L[0];
    if (L.bits == 8) return gemm_pair_launch<8, false, 1, true>(set, x, M, st, device, pdl, num_sms, nullptr, nullptr, act);
    if (L.grouped) return gemm_pair_launch<4, true, 1, true>(set, x, M, st, device, pdl, num_sms, nullptr, nullptr, act);
    return gemm_pair_launch<4, false, 1, true>(set, x, M, st, device, pdl, num_sms, nullptr, nullptr, act);
}

}  // namespace ql
