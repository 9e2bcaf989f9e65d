// Prefill kernel, CTA-pair form with the dequantised weights in TENSOR MEMORY (paper Section 3.7: the compute-bound
// prefill stage; Section 3.1: weights stored in the order the kernel reads them).
//
// The CTA-pair kernel of gemm_pair.cuh writes every dequantised 128 x 64 fp16 weight tile to shared memory and the
// tensor core reads it back from there: 32 KB of shared-memory traffic per k-step and CTA on top of the x tile,
// in a kernel that is bound by exactly that traffic.  Here the dequantise warps store the fp16 values straight
// into tensor memory (tcgen05.st) and the MMA takes its A operand from there (tcgen05.mma with a tensor-memory A
// address); shared memory only carries the TMA stages (packed weights + x) and the B operand reads.
//
// Layout consequences:
//   * tensor memory (512 columns): one 256-column fp32 accumulator + 8 A slots of 32 columns (64 k of fp16); there
//     is no room for a second accumulator, so the epilogue is not hidden under the next tile.  It is kept short
//     instead: 16 warps take the accumulator out together (64 columns each) as soon as they see the tile complete,
//     free it, and leave fp16 values in a shared output tile that bulk copies drain under the next main loop;
//     meanwhile up to 6 A slots of the next tile are already filled, so the MMA restarts at once;
//   * a thread of a dequantise warp owns ONE tile row (its TMEM lane): it needs 32 consecutive k of that row, which
//     the packed block keeps in four 16-byte pieces (lane columns c = 0..3 of its row-block line), 64 bytes apart
//     from the neighbouring row's: the packed block is therefore fetched with a tiled TMA copy (rows of 64 bytes,
//     64-byte swizzle) instead of a plain bulk copy, which makes those reads free of bank conflicts;
//   * a warp converts the 32 rows of its lane quarter x one 32-k half of every third k-step (24 warps: 4 quarters x
//     2 halves x 3 turns); rows g and g + 8 of a row-block read the same bytes and take the low or the high nibbles
//     (int4) / the low or the high byte pair (int8);
//   * two TMA rings (the weights of a k-step are needed early, its x tile only at MMA time) and one barrier per A slot
//     on which the slot's 8 warps, the step's x tile and the peer CTA arrive, so that the issuing thread waits once
//     per k-step.
//
// What bounded it (measured): not the tensor pipe (halving the MMA width changed nothing) but the instruction stream
// of the dequantise warps and of the polling threads around them, which is why every warp loops over its own steps
// only and no thread polls in the main loop.  As it stands the tensor pipe is active 86-91 % of the cycles in which an
// SM has work (tiles of 64 k-steps; 71 % with 36), at the clock the power limit leaves: what is missing is a constant
// 3-4 us per tile boundary -- last MMAs retire, epilogue warps finish their step, meet, take the accumulator out, tell
// the leader across the SM pair -- which is why both cross-SM signals on that path (the relay's and the epilogue's)
// are relaxed arrives.
//
// Forms of the kernel (template flags): the plain product, whole tiles dealt out round-robin or, for launches with
// few tiles, 2 or 4 K parts per tile that meet in the device scratch; GATED (y = act(gate) * up, Section 3.6); I8
// (int8 activations, kind::i8 on the stored weight bytes, Section 3.7).
//
// Protocol between the two CTAs: own loads only; the leader issues; commits are multicast to both CTAs; the peer relays
// "slot ready" (see the relay below).
#pragma once
#include "gemm_pair.cuh"

namespace ql {

constexpr int kTaFirstDequantWarp = 4;       // warps 4..27: dequantise, six per TMEM lane quarter; 4..19 also run the epilogue
constexpr int kTaDequantWarps = 24;
constexpr int kTaStepWarps = 8;              // warps that share one k-step: 4 lane quarters x 2 halves of 32 k
constexpr int kTaEpilogueWarps = 16;
constexpr int kTaSlotCols = 32;              // 64 k of fp16
constexpr int kTaAccCols = 256;

// I8: the integer form (int8 activations, kind::i8): a k-step is 128 k, i.e. again 128 bytes per x row and 32 columns per A slot.
template <int BITS, bool I8 = false>
struct GemmTaSmem {
    // Two rings, because the two operands are needed at different times: the packed weights of a k-step are needed
    // early (they still have to be dequantised), its x tile only when the MMA is issued.  A deep ring of small
    // weight stages lets the dequantise warps run ahead; the x ring only has to cover the TMA latency.
    static constexpr int kXBytes = 128 * 128;                            // this CTA's 128 tokens x 64 k
    static constexpr int kKStep = I8 ? 128 : kGemmKStep;
    static constexpr int kXStages = (I8 && BITS == 8) ? 6 : 7;           // <= kASlots: the x producer reads "stage free" off the A-slot barrier
    static constexpr int kWBlocks = (I8 ? 2 : 1) * (BITS == 4 ? 1 : 2);  // packed blocks per k-step
    static constexpr int kWBytes = I8 ? kWBlocks * kWeightBlockBytes : (BITS == 4 ? 5120 : 8192);
    // A ring length that is a multiple of the 3 dequantise turns keeps every stage with one turn, whose warps then see all
    // of the stage's phases in order; the 16 KB stages of the int8 integer form leave room for 4 only, and its warps first
    // wait for the stage's release (see the main loop of the dequantise warps).
    static constexpr int kWStages = I8 ? (BITS == 4 ? 6 : 4) : (BITS == 4 ? 9 : 6);
    static constexpr int kASlots = 8;                                    // tensor memory: 8 x 32 columns beside the accumulator
    static constexpr int kEarlySteps = kASlots - 2;                      // steps of the next tile dequantised before the epilogue is forced
    static constexpr int kWOffset = kXStages * kXBytes;
    static constexpr int kOutOffset = kWOffset + kWStages * kWBytes;     // fp16 output tile [256 tokens][128 channels]
    static constexpr int kOutBytes = 256 * 256;
    static constexpr int kBarOffset = kOutOffset + kOutBytes;
    static constexpr int kTotal = kBarOffset + 512 + 1024;               // barriers + alignment slack
    static_assert(kXStages <= kASlots, "x stage g % kXStages is free when A slot g % kASlots is");
    static_assert(kTotal <= 227 * 1024, "shared memory");
};

struct TaMaps {
    CUtensorMap x;                       // [M, K] fp16, box 64 k x 128 tokens, 128-byte swizzle
    CUtensorMap w[kGemmMaxGroup];        // packed body of each layer as rows of 64 bytes, 64-byte swizzle
};

// The packed body of a layer as a 2-D tensor of 64-byte rows; box = the block(s) of one 64-k step.
// i8: the integer form's box (128 k: two int4 blocks or four int8 blocks; per-channel schemes only).
inline bool w_tensor_map(const Layout& L, const uint8_t* blob, CUtensorMap* out, bool i8 = false)
{
    EncodeTiledFn enc = get_encode_tiled();
    if (!enc) return false;
    if (i8 && L.grouped) return false;
    const int64_t rows = (int64_t)L.n_rsb * L.n_kc * (L.block_bytes / 64);
    const int box_rows = (i8 ? 2 : 1) * (L.bits == 4 ? L.block_bytes / 64 : 2 * (kWeightBlockBytes / 64));
    if (rows < box_rows || rows > 0x7FFFFFFFll) return false;
    const cuuint64_t gdim[2] = {64, (cuuint64_t)rows};
    const cuuint64_t gstr[1] = {64};
    const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(blob + L.body_offset), gdim, gstr, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Per-thread constants of a dequantise warp: the thread's tile row is TMEM lane 32 * quarter + lane, i.e. row-block
// 2 * quarter + lane / 16, lane-row g = lane % 8, upper half (rows g + 8) for lanes 8..15 and 24..31.
// Shared-memory loads through 32-bit shared-window addresses (a generic pointer costs 64-bit address arithmetic per load).
__device__ __forceinline__ uint2 lds_u64(uint32_t addr)
{
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint4 lds_u128(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds_u16(uint32_t addr)
{
    uint16_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr));
    return v;
}

struct DequantRowTa {
    int off[4];                  // byte offset, inside the packed block, of piece c of the row's 64-byte line (64-byte swizzle:
                                 // piece c sits at position c ^ ((line / 2) & 3))
    int s_off;                   // grouped int4: byte offset of the row's scale of group 0 (group 1: + 2)
    uint32_t mask, mul, add;     // int4: nibble mask and the exact fp16 fix-up of the chosen nibbles
    uint32_t sel;                // int8: byte pair of the chosen row
    __device__ DequantRowTa(int quarter, int lane)
    {
        const int rb = 2 * quarter + (lane >> 4), g = lane & 7, hi = (lane >> 3) & 1;
        for (int c = 0; c < 4; ++c) off[c] = (rb * 8 + g) * 64 + ((c ^ ((g >> 1) & 3)) << 4);
        // scales: 64-byte line 64 + rb of the block (swizzle term (rb >> 1) & 3 = quarter), piece g / 2
        s_off = kWeightBlockBytes + rb * 64 + (((g >> 1) ^ quarter) << 4) + (g & 1) * 8 + hi * 4;
        mask = hi ? 0x00F000F0u : 0x000F000Fu;
        mul = hi ? 0x2C002C00u : 0x3C003C00u;                            // {1/16, 1/16} or {1, 1}
        add = hi ? 0xD480D480u : 0xE408E408u;                            // {-72, -72} or {-1032, -1032}
        sel = hi ? 0x4342u : 0x4140u;
    }
    // 32 consecutive k of the row (half h of the 64-k step) -> 16 registers = 16 columns of the row's TMEM lane.
    // Same arithmetic as unpack_int4_word / unpack_int8_words (exact integers, then one multiplication by the scale).
    template <int BITS, bool GROUPED, bool I8 = false>
    __device__ __forceinline__ void convert(uint32_t wp, int h, uint32_t r[16]) const   // wp: shared-window address of the stage
    {
        if (I8) {
            // integer form: 64 consecutive k of the row (half h of the 128-k step) as the stored unsigned bytes
            // (q + 8 or q + 128), 4 per column: no arithmetic, only the choice of nibbles / bytes and their order
            if (BITS == 4) {
                const uint32_t rp = wp + h * kWeightBlockBytes;                              // packed block h of the step
                const uint32_t sh = mask == 0x000F000Fu ? 0u : 4u;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint4 w = lds_u128(rp + off[c]);
                    // a word's nibbles of this row are slots 0, 2, 1, 3 (layout.h): k 8c .. 8c + 3 of a 32-k half per word pair
                    r[2 * c + 0] = __byte_perm((w.x >> sh) & 0x0F0F0F0Fu, 0, 0x3120);
                    r[2 * c + 1] = __byte_perm((w.y >> sh) & 0x0F0F0F0Fu, 0, 0x3120);
                    r[8 + 2 * c + 0] = __byte_perm((w.z >> sh) & 0x0F0F0F0Fu, 0, 0x3120);
                    r[8 + 2 * c + 1] = __byte_perm((w.w >> sh) & 0x0F0F0F0Fu, 0, 0x3120);
                }
            } else {
                const uint32_t bsel = sel == 0x4140u ? 0x5410u : 0x7632u;                    // this row's byte pair of two words
#pragma unroll
                for (int b = 0; b < 2; ++b) {                                                // blocks 2h, 2h + 1: 32 k each
                    const uint32_t rp = wp + (2 * h + b) * kWeightBlockBytes;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const uint4 w = lds_u128(rp + off[c]);
                        r[8 * b + 2 * c + 0] = __byte_perm(w.x, w.y, bsel);
                        r[8 * b + 2 * c + 1] = __byte_perm(w.z, w.w, bsel);
                    }
                }
            }
            return;
        }
        if (BITS == 4) {
            const uint32_t rp = wp + 8 * h;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint2 w = lds_u64(rp + off[c]);
                r[4 * c + 0] = h2_fma(lop3_and_or(w.x, mask, 0x64006400u), mul, add);        // k 8c + 0, 1
                r[4 * c + 1] = h2_fma(lop3_and_or(w.x >> 8, mask, 0x64006400u), mul, add);   // k 8c + 2, 3
                r[4 * c + 2] = h2_fma(lop3_and_or(w.y, mask, 0x64006400u), mul, add);        // k 8c + 4, 5
                r[4 * c + 3] = h2_fma(lop3_and_or(w.y >> 8, mask, 0x64006400u), mul, add);   // k 8c + 6, 7
            }
            if (GROUPED) {
                const uint32_t s = lds_u16(wp + s_off + 2 * h);
                const uint32_t s2 = s | (s << 16);
#pragma unroll
                for (int i = 0; i < 16; ++i) r[i] = h2_mul(r[i], s2);
            }
        } else {
            const uint32_t rp = wp + h * kWeightBlockBytes;                                  // chunk h of the step
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint4 w = lds_u128(rp + off[c]);
                r[4 * c + 0] = h2_sub(__byte_perm(w.x, 0x64646464u, sel), 0x64806480u);
                r[4 * c + 1] = h2_sub(__byte_perm(w.y, 0x64646464u, sel), 0x64806480u);
                r[4 * c + 2] = h2_sub(__byte_perm(w.z, 0x64646464u, sel), 0x64806480u);
                r[4 * c + 3] = h2_sub(__byte_perm(w.w, 0x64646464u, sel), 0x64806480u);
            }
        }
    }
};

// Warp roles: 0 weight producer, 1 MMA issuer (leader) / relay (peer), 2 x producer, 3 spare, 4..27 dequantise (4..19 also epilogue).
// GATED: the launch serves two layers of equal shape, gate (0) and up (1).  A cluster runs the gate tile and then the up
// tile of the same (row super-block pair, token block) position.  The gate tile's epilogue leaves fp16(act(gate)) in
// the shared output tile (nothing is sent to memory); the up tile's epilogue multiplies what it finds there by the up
// projection, every thread reading back the values it wrote itself, and only that product goes to y (paper Section
// 3.6).  n_tiles then counts positions of ONE layer.
// I8 (per-channel schemes, not gated): maps.x describes int8 activations; the stored weight integers go to the A slots
// unconverted, the MMAs are kind::i8 with an s32 accumulator, and the epilogue removes the storage offset (offset x the
// sum of the token's quantised row) and applies both scales (paper Section 3.7, prefill stage).
template <int BITS, bool GROUPED, bool GATED = false, bool I8 = false>
__global__ void __launch_bounds__(kPairThreads, 1)
gemm_pair_ta_kernel(const __grid_constant__ TaMaps maps, const GemmParams p)
{
    static_assert(!I8 || (!GATED && !GROUPED), "the integer form: per-channel scales, plain output");
    using S = GemmTaSmem<BITS, I8>;
    constexpr int NX = S::kXStages, NW = S::kWStages, NA = S::kASlots;
    constexpr int BN = 256;
    constexpr int W_BOX_BYTES = I8 ? S::kWBytes : BITS == 4 ? (GROUPED ? kWeightBlockBytes + kScaleBlockBytes : kWeightBlockBytes) : 2 * kWeightBlockBytes;
    extern __shared__ unsigned char smem_dyn[];
    const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
    auto xs_addr = [&](int s) { return base + s * S::kXBytes; };
    auto wpk_addr = [&](int s) { return base + S::kWOffset + s * S::kWBytes; };
    const uint32_t bar0 = base + S::kBarOffset;
    // (barrier slots 0 .. NX-1 are unused: the x tile of a step completes on the step's afull barrier)
    auto wfull_bar = [&](int s) { return bar0 + 8 * (NX + s); };         // local: this CTA's packed block landed
    auto wempty_bar = [&](int s) { return bar0 + 8 * (NX + NW + s); };   // local: the 8 warps of the step have read the block
    auto afull_bar = [&](int a) { return bar0 + 8 * (NX + 2 * NW + a); };        // local: this CTA's A slot written
    auto aempty_bar = [&](int a) { return bar0 + 8 * (NX + 2 * NW + NA + a); };  // local, signalled by the leader's commit:
                                                                                 // the step's MMAs retired (A slot and x stage free)
    const uint32_t tfull_bar = bar0 + 8 * (NX + 2 * NW + 2 * NA);        // local, signalled by the leader's commit
    const uint32_t tempty_bar = tfull_bar + 8;                           // leader: both CTAs drained the accumulator
    // local: the four warps that share 64 tokens of the output tile meet here (b = 0: rows free again, b = 1: rows written)
    auto grp_bar = [&](int wi, int b) { return tempty_bar + 8 + 8 * (2 * wi + b); };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + S::kBarOffset + 8 * (NX + 2 * NW + 2 * NA + 10));
    volatile uint32_t* abort_flag = tmem_slot + 1;
    static_assert(8 * (NX + 2 * NW + 2 * NA + 10) + 32 <= 512, "barrier area");

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();                             // 0 = leader
    const int n_mblk = (p.M + BN - 1) / BN;
    const int first_tile = blockIdx.x >> 1, tile_stride = gridDim.x >> 1;   // tile = (rsb pair, token block)
    // K split (p.split = 2 or 4 parts per tile; launches with so few tiles that every cluster then has ONE unit of work):
    // work unit v = tile * split + part, this cluster's part covers k-steps [it_base, it_base + n_steps) of its tile
    const int P = GATED ? 1 : p.split;
    const int part = P > 1 ? first_tile % P : 0;
    const int it_base = part * p.n_ksteps / P;
    const int n_steps = (part + 1) * p.n_ksteps / P - it_base;          // k-steps per unit of work of this cluster
    // the j-th unit of work of this cluster: a tile and, in the gated form, which of the two layers
    auto unit = [&](int j, int& tile, int& gl) {
        const int v = first_tile + (GATED ? j >> 1 : j) * tile_stride;
        tile = P > 1 ? v / P : v;
        gl = GATED ? (j & 1) : 0;
        return v < p.n_tiles * P;
    };
    int n_units = 0;
    for (int v = first_tile; v < p.n_tiles * P; v += tile_stride) n_units += GATED ? 2 : 1;
    const int total_steps = n_units * n_steps;
    const int w_rows = p.block_bytes >> 6;                               // 64-byte rows per packed block

    if (threadIdx.x == 0) {
        for (int s = 0; s < NW; ++s) {
            mbar_init(wfull_bar(s), 1);
            mbar_init(wempty_bar(s), kTaStepWarps);
        }
        for (int a = 0; a < NA; ++a) {
            // this CTA's 8 warps of the step + its x tile (one arrival with the byte count) + (leader) the peer's relay
            mbar_init(afull_bar(a), kTaStepWarps + 1 + (rank == 0 ? 1 : 0));
            mbar_init(aempty_bar(a), 1);
        }
        mbar_init(tfull_bar, 1);
        mbar_init(tempty_bar, 2 * kTaEpilogueWarps);
        for (int i = 0; i < 8; ++i) mbar_init(grp_bar(i >> 1, i & 1), 4);
        abort_flag[0] = 0;                                               // [0] abort, [1] abort of the exit drain,
        abort_flag[1] = 0;                                               // [2], [3] "past griddepcontrol.wait" (see wait_expired)
        abort_flag[2] = 0;
        abort_flag[3] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc_pair(smem_u32((const void*)tmem_slot), 512);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                                  // both CTAs' barriers exist before any remote arrive
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // The next kernel in the stream may move onto SMs this grid has left (the last, partial round of tiles) and set up
    // there; whatever it reads of this grid's output comes after its own griddepcontrol.wait.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // Relay (peer CTA): "A slot written, x tile landed" -> one arrive on the leader's afull barrier; two threads (warps 1 and
    // 3 of the peer) take alternate steps.  The arrive is RELAXED: with release semantics at cluster scope it took about a
    // microsecond here, several k-steps.  Nothing it would publish crosses the two SMs: the A slot (tensor memory) and the
    // x tile (shared memory) were written inside the peer SM, their writes had completed (tcgen05.wait::st, TMA
    // complete_tx) before the peer's own barrier completed, and they are read by the peer's own tensor core, which the
    // leader's MMA instruction starts only after it has seen this arrive.  Only the signal travels.
    auto relay = [&](int r) {
        int a = r;
        uint32_t apar = 0;
        for (int g = r; g < total_steps; g += 2) {
            if (!mbar_wait(afull_bar(a), apar, abort_flag, 0xA00 + a)) break;
            tc_fence_before();
            mbar_arrive_remote_relaxed(afull_bar(a), 0);
            a += 2; if (a >= NA) { a -= NA; apar ^= 1; }
        }
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ weight producer (each CTA feeds itself)
        if (lane == 0) {
            constexpr int CHUNKS = S::kWBlocks;                          // packed blocks per k-step
            int s = 0, issued = 0;
            uint32_t par = 1;
            bool ok = true;
            int tile, gl;
            for (int j = 0; ok && unit(j, tile, gl); ++j) {
                int rsb = 2 * (tile / n_mblk) + (int)rank;
                const int ly = GATED ? gl : pair_layer(p, rsb);
                const int row0 = rsb * p.n_kc * w_rows;
                const CUtensorMap* wm = &maps.w[ly];
                for (int it = 0; it < n_steps; ++it) {
                    if (!mbar_wait(wempty_bar(s), par, abort_flag, 0x100 + s)) { ok = false; break; }
                    mbar_expect_tx(wfull_bar(s), W_BOX_BYTES);
                    tma_load_2d(wpk_addr(s), wm, 0, row0 + (it_base + it) * CHUNKS * w_rows, wfull_bar(s));
                    ++issued;
                    if (++s == NW) { s = 0; par ^= 1; }
                }
            }
            if (*abort_flag) {
                for (int j = max(0, issued - NW); j < issued; ++j)
                    mbar_wait(wfull_bar(j % NW), (j / NW) & 1, abort_flag + 1, 0);
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------------ x producer (each CTA loads its 128 tokens)
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&maps.x) : "memory");
            asm volatile("griddepcontrol.wait;" ::: "memory");           // x may come from the previous kernel
            abort_flag[2] = 1;                                           // from here on, waiting counts against the time limit
            abort_flag[3] = 1;
            int s = 0, g = 0;
            bool ok = true;
            int tile, gl;
            for (int j = 0; ok && unit(j, tile, gl); ++j) {
                const int m0 = (tile % n_mblk) * BN + 128 * (int)rank;   // this CTA's 128 tokens
                for (int it = 0; it < n_steps; ++it, ++g) {
                    // stage s was last used by step g - NX, whose MMAs signal A-slot barrier (g - NX) % NA; by then the
                    // afull barrier of step g's slot has completed its previous phase (step g - NA was issued earlier)
                    if (g >= NX) {
                        const int ao = (g - NX) % NA;
                        if (!mbar_wait(aempty_bar(ao), (uint32_t)((g - NX) / NA) & 1, abort_flag, 0x180 + ao)) { ok = false; break; }
                    }
                    mbar_expect_tx(afull_bar(g % NA), S::kXBytes);
                    tma_load_2d(xs_addr(s), &maps.x, (it_base + it) * S::kKStep, m0, afull_bar(g % NA));
                    if (++s == NX) s = 0;
                }
            }
            if (*abort_flag) {                                           // let the copies in flight land before the CTA leaves
                const long long t0 = clock64();
                while (clock64() - t0 < (1ll << 18)) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        // The whole warp runs the loop (warp-uniform control flow, so counters and descriptors can stay in uniform
        // registers); one elected lane issues.
        if (rank == 0) {
            // f16 x f16 -> f32, both operands K-major (A from tensor memory), M = 256 per pair, N = 256
            // (integer form: u8 weights x s8 activations -> s32)
            const uint32_t idesc = (I8 ? (2u << 4) | (1u << 10) : (1u << 4)) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
            const uint32_t b_lo0 = umma_desc_lo(xs_addr(0));
            int s = 0, a = 0;
            uint32_t apar = 0;
            bool ok = true;
            int tile, gl;
            for (int j = 0; ok && unit(j, tile, gl); ++j) {
                if (!mbar_wait_hot(tempty_bar, (uint32_t)(j & 1) ^ 1, abort_flag, 0x800)) { ok = false; break; }
                tc_fence_after();
                for (int it = 0; it < n_steps; ++it) {
                    // both CTAs' A slots written and both x tiles landed (8 local warps, the local x tile, the peer's relay)
                    // (the dequantise warps run ahead, so the phase is normally complete already: test, else suspend)
                    if (!mbar_wait(afull_bar(a), apar, abort_flag, 0x300 + a)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t ta = tmem_base + (uint32_t)(kTaAccCols + a * kTaSlotCols);
                    const uint32_t b_lo = b_lo0 + (uint32_t)s * (S::kXBytes >> 4);
                    if (elect_one()) {
#pragma unroll
                        for (int k4 = 0; k4 < 4; ++k4) {                 // 16 k (32 k of bytes): 8 columns of A, 32 bytes of the B swizzle row
                            if (I8) umma_i8_pair_ta(tmem_base, ta + 8 * k4, b_lo + 2 * k4, idesc, (it > 0 || k4 > 0) ? 1u : 0u);
                            else umma_f16_pair_ta(tmem_base, ta + 8 * k4, b_lo + 2 * k4, idesc, (it > 0 || k4 > 0) ? 1u : 0u);
                        }
                        umma_commit_pair(aempty_bar(a));                 // frees the A slot and the x stage in both CTAs
                    }
                    __syncwarp();
                    if (++s == NX) s = 0;
                    if (++a == NA) { a = 0; apar ^= 1; }
                }
                if (ok && elect_one()) umma_commit_pair(tfull_bar);
                __syncwarp();
            }
        } else if (lane == 0) relay(0);
    } else if (warp == 3) {
        if (rank != 0 && lane == 0) relay(1);
    } else if (warp >= kTaFirstDequantWarp) {
        // ------------------------------------------------------------------ dequantise + epilogue
        const int quarter = warp & 3, wi = (warp - kTaFirstDequantWarp) >> 2;
        const int half = wi & 1, my_turn = wi >> 1;                      // 32-k half of the step; this warp takes every third step
        const bool epi_warp = wi < 4;                                    // the first 16 warps also run the epilogue (64 tokens each)
        const DequantRowTa dq(quarter, lane);
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        bool ok = true;

        // The epilogue of the j-th tile of this cluster: this warp takes columns (tokens) 64 wi .. + 63 of its lane
        // quarter (32 channels) out of the accumulator, frees the accumulator, and leaves fp16 values in the
        // shared output tile [token][channel]; the four warps that share the 64 tokens then meet at a barrier
        // and send each token's 256 bytes to y with one bulk copy, which drains under the next tile's main loop.
        const uint32_t out_addr = base + S::kOutOffset;
        unsigned char* out_ptr = base_ptr + S::kOutOffset;
        const int grp_thread = quarter * 32 + lane;                      // 0..127 inside the group of four warps
        // K-split tile: every part parks its fp32 accumulator in the device's scratch ([token][channel], a warp writes
        // 128 contiguous bytes per token), frees the accumulator and counts itself in; the part that arrives last adds all
        // parts in part order (fixed order, no float atomics, nobody waits) and stores y.
        auto split_epilogue = [&](int j, int tile) {
            int rsb = 2 * (tile / n_mblk) + (int)rank;
            const int ly = pair_layer(p, rsb);
            const int N = p.lN[ly];
            const int m0 = (tile % n_mblk) * BN + 64 * wi;
            float* slab0 = p.scratch + ((int64_t)((tile * P) * 2 + (int)rank) * BN + 64 * wi) * 128 + grp_thread;   // part 0
            const int64_t part_stride = (int64_t)2 * BN * 128;
            unsigned int* cnt = p.counters + ((tile * 2 + (int)rank) * 4 + wi) * 4 + quarter;
            if (!mbar_wait(tfull_bar, (uint32_t)(j & 1), abort_flag, 0x500)) { ok = false; return; }
            tc_fence_after();
            const uint32_t taddr = tmem_base + lane_base + (uint32_t)(64 * wi);
            float* mine = slab0 + part * part_stride;
#pragma unroll 1
            for (int cc = 0; cc < 64; cc += 16) {
                uint32_t r[16];
                tmem_ld16(taddr + (uint32_t)cc, r);
#pragma unroll
                for (int q = 0; q < 16; ++q) __stcg(mine + (cc + q) * 128, __uint_as_float(r[q]));
            }
            tc_fence_before();
            __threadfence();
            __syncwarp();
            unsigned int old = 0;
            if (lane == 0) { mbar_arrive_remote_relaxed(tempty_bar, 0); old = atomicAdd(cnt, 1u); }
            old = __shfl_sync(0xffffffffu, old, 0);
            if ((int)old != P - 1) return;
            __threadfence();
            const int n = rsb * kRsbRows + quarter * 32 + lane;
            float scale = 1.f;
            if (!GROUPED && n < N) scale = __half2float(p.lscales[ly][n]);
            __half* yrow = p.ly[ly] + (int64_t)m0 * N + n;
            const int m_left = min(64, p.M - m0);
#pragma unroll 1
            for (int cc = 0; cc < m_left; cc += 8) {
                float acc[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) acc[q] = __ldcg(slab0 + (cc + q) * 128);
                for (int pp = 1; pp < P; ++pp) {
                    float v[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) v[q] = __ldcg(slab0 + pp * part_stride + (cc + q) * 128);
#pragma unroll
                    for (int q = 0; q < 8; ++q) acc[q] += v[q];
                }
                if (n < N) {
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        if (cc + q < m_left) yrow[(int64_t)(cc + q) * N] = __float2half_rn(acc[q] * scale);
                }
            }
            if (lane == 0) *cnt = 0;                                     // ready for the next launch
        };
        auto epilogue = [&](int j) {
            int tile, gl;
            unit(j, tile, gl);
            if (P > 1) { split_epilogue(j, tile); return; }
            int rsb = 2 * (tile / n_mblk) + (int)rank;
            const int ly = GATED ? 0 : pair_layer(p, rsb);
            const int N = p.lN[ly];
            const int m0 = (tile % n_mblk) * BN + 64 * wi;
            const uint32_t gpar = (uint32_t)(GATED ? j >> 1 : j) & 1;   // phase of the group barriers: once per output tile
            bool live = true;
            if (!GATED || gl == 0) {
                // the bulk copies of the previous output tile have read their rows of the shared tile
                if (grp_thread < 64) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(grp_bar(wi, 0));
                live = mbar_wait(grp_bar(wi, 0), gpar, abort_flag, 0xC00 + wi);
            }
            live = live && mbar_wait(tfull_bar, (uint32_t)(j & 1), abort_flag, 0x500);
            if (live) {
                tc_fence_after();
                const int n = rsb * kRsbRows + quarter * 32 + lane;
                float scale = 1.f;
                if (!GROUPED && n < N) scale = __half2float(p.lscales[GATED ? gl : ly][n]);
                const uint32_t taddr = tmem_base + lane_base + (uint32_t)(64 * wi);
                __half* orow = reinterpret_cast<__half*>(out_ptr + (64 * wi) * 256) + grp_thread;
#pragma unroll
                for (int cc = 0; cc < 64; cc += 32) {
                    uint32_t r[32];
                    tmem_ld32(taddr + (uint32_t)cc, r);
                    if (cc == 32) {                                      // accumulator read: the next tile's MMAs may start
                        // RELAXED arrive, like the relay's: what must precede the leader's next MMA is the completion of
                        // this warp's tensor-memory loads, which tcgen05.wait::ld (inside tmem_ld32) has already waited
                        // for; nothing in shared or global memory is handed over.  With release semantics at cluster
                        // scope the arrive sat on the critical path of every tile boundary (Llama gate: 179 -> 176 us).
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_remote_relaxed(tempty_bar, 0);
                    }
                    if (I8) {
                        // acc = sum (q + off) * xq: remove off * (sum of the token's quantised row), then both scales; the 32
                        // tokens' scales and row sums come as whole lines (the arrays are padded to whole tiles)
                        constexpr int OFF = BITS == 4 ? 8 : 128;
#pragma unroll
                        for (int v4 = 0; v4 < 8; ++v4) {
                            const float4 f = __ldg(reinterpret_cast<const float4*>(p.a8_scale + m0 + cc) + v4);
                            const int4 i = __ldg(reinterpret_cast<const int4*>(p.a8_rowsum + m0 + cc) + v4);
                            orow[(cc + 4 * v4 + 0) * 128] = __float2half_rn(f.x * (scale * (float)((int)r[4 * v4 + 0] - OFF * i.x)));
                            orow[(cc + 4 * v4 + 1) * 128] = __float2half_rn(f.y * (scale * (float)((int)r[4 * v4 + 1] - OFF * i.y)));
                            orow[(cc + 4 * v4 + 2) * 128] = __float2half_rn(f.z * (scale * (float)((int)r[4 * v4 + 2] - OFF * i.z)));
                            orow[(cc + 4 * v4 + 3) * 128] = __float2half_rn(f.w * (scale * (float)((int)r[4 * v4 + 3] - OFF * i.w)));
                        }
                    } else {
                        // (the kind of activation is chosen outside the element loop: inside it, the compiler evaluates
                        // every kind and selects)
                        auto store32 = [&](auto f) {
#pragma unroll
                            for (int q = 0; q < 32; ++q) orow[(cc + q) * 128] = __float2half_rn(f(__uint_as_float(r[q]) * scale, q));
                        };
                        if (!GATED) store32([](float v, int) { return v; });
                        else if (gl == 1) store32([&](float v, int q) { return v * __half2float(orow[(cc + q) * 128]); });   // this thread's own act(gate)
                        else if (p.act == QL_ACT_SILU) store32([](float v, int) { return gate_activation(v, QL_ACT_SILU); });
                        else if (p.act == QL_ACT_GELU_TANH) store32([](float v, int) { return gate_activation(v, QL_ACT_GELU_TANH); });
                        else store32([](float v, int) { return v; });
                    }
                }
                fence_async_smem();
            }
            if (GATED && gl == 0) {                                      // the product is sent when the up tile is done
                if (!live) ok = false;
                return;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(grp_bar(wi, 1));
            live = mbar_wait(grp_bar(wi, 1), gpar, abort_flag, 0xC10 + wi) && live;
            if (live && grp_thread < 64 && m0 + grp_thread < p.M) {
                const int n0 = rsb * kRsbRows;
                const uint32_t bytes = (uint32_t)min(kRsbRows, N - n0) * 2;
                bulk_copy_s2g(p.ly[ly] + (int64_t)(m0 + grp_thread) * N + n0, out_addr + (uint32_t)(64 * wi + grp_thread) * 256, bytes);
            }
            if (grp_thread < 64) asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            if (!live) ok = false;
        };
        auto tile_complete = [&](int j) {                                // non-blocking: has the j-th tile's last MMA retired?
            uint32_t done;
            asm volatile("{\n\t.reg .pred p;\n\t"
                         "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                         "selp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(done) : "r"(tfull_bar), "r"((uint32_t)(j & 1)) : "memory");
            return done != 0;
        };

        // The k-steps of all tiles of this cluster are numbered through (g); this warp takes g = my_turn, my_turn + 3, ...
        const int forced = min(S::kEarlySteps, n_steps - 1);
        int s = my_turn, a = my_turn;                                    // W stage and A slot of step g (my_turn < NW, NA)
        uint32_t wpar = 0, apar = 1;                                     // A slots start out free
        int tile_j = 0, tile_g0 = 0;                                     // tile of step g and its first step
        int next_epi = 0;                                                // tiles leave through the epilogue in order
        for (int g = my_turn; g < total_steps && ok; g += 3) {
            while (g >= tile_g0 + n_steps) { ++tile_j; tile_g0 += n_steps; }
            // an earlier tile still holds the accumulator: run its epilogue once it is complete, or, at the latest,
            // after `forced` steps of this tile have been dequantised
            if (epi_warp && next_epi < tile_j && (g - tile_g0 >= forced || tile_complete(next_epi))) {
                epilogue(next_epi);
                ++next_epi;
                if (!ok) break;
            }
            uint32_t r[16];
            // A weight stage whose ring length is not a multiple of the 3 turns is served by a different turn every time
            // round, so this warp has not seen the stage's previous phase: the load of step g - NW may still be in flight
            // (bulk copies complete in any order), and a parity test alone would then take that phase for this one.  The
            // producer issues the load of step g only after step g - NW's warps have released the stage: wait for that first.
            if (NW % 3 != 0 && !mbar_wait(wempty_bar(s), wpar ^ 1, abort_flag, 0x480 + s)) { ok = false; break; }
            if (!mbar_wait(wfull_bar(s), wpar, abort_flag, 0x400 + s)) { ok = false; break; }
            dq.template convert<BITS, GROUPED, I8>(wpk_addr(s), half, r);
            // the MMAs that read slot a (step g - NA) have retired
            if (!mbar_wait(aempty_bar(a), apar, abort_flag, 0xB00 + a)) { ok = false; break; }
            tc_fence_after();
            tmem_st16(tmem_base + lane_base + (uint32_t)(kTaAccCols + a * kTaSlotCols + 16 * half), r);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) { mbar_arrive(wempty_bar(s)); mbar_arrive(afull_bar(a)); }
            s += 3; if (s >= NW) { s -= NW; wpar ^= 1; }
            a += 3; if (a >= NA) { a -= NA; apar ^= 1; }
        }
        while (epi_warp && ok && next_epi < n_units) { epilogue(next_epi); ++next_epi; }
        asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");        // y written before the kernel ends
    }

    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                                  // the peer no longer reads this CTA's memory
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, 512);
    }
}

// The tensor-memory form: 256-token tiles, whole tiles dealt out round-robin, or (fewer tiles than half the CTA pairs)
// 2 or 4 K parts per tile that meet in the device's scratch.
// K parts per tile for a launch of `tiles` tiles: 1 unless the tiles would leave half of the CTA pairs (or more) idle.
inline int gemm_pair_ta_split(int tiles, int n_ksteps, int num_sms, bool have_scratch)
{
    const int clusters = num_sms / 2;
    int split = 1;
    if (!have_scratch || tiles >= clusters) return 1;
    if (gemm_config().force_split > 0) split = gemm_config().force_split >= 4 ? 4 : gemm_config().force_split >= 2 ? 2 : 1;
    else if (tiles * 4 <= clusters) split = 4;
    else if (tiles * 2 <= clusters) split = 2;
    while (split > 1 && (n_ksteps / split < 8 || tiles * split > clusters)) split >>= 1;
    return split;
}

// act < 0: the plain form.  act >= 0: the gated form, set = {gate, up} of equal shape, y[0] the output.
// scratch / counters: the device's shared fp32 scratch and arrival counters for the K-split case (null: no split).
// a8_scale != nullptr: the integer form; x is then the int8 activations, a8_scale / a8_rowsum their per-token arrays, and
// set.wmap the integer form's weight maps (boxes of 128 k).
template <int BITS, bool GROUPED, bool GATED = false, bool I8 = false>
ql_status gemm_pair_ta_launch(const GemmPairLayers& set, const void* x, int M, cudaStream_t st, int device, bool pdl, int num_sms, int act = -1,
                              float* scratch = nullptr, unsigned int* counters = nullptr,
                              const float* a8_scale = nullptr, const int32_t* a8_rowsum = nullptr)
{
    using S = GemmTaSmem<BITS, I8>;
    const Layout& L = *set.L[0];
    TaMaps maps;
    if (!x_tensor_map(x, L.K, M, 128, &maps.x, I8 ? 1 : 2)) return QL_ERR_CUDA;
    for (int i = 0; i < kGemmMaxGroup; ++i) maps.w[i] = *set.wmap[i < set.n ? i : 0];
    auto kern = gemm_pair_ta_kernel<BITS, GROUPED, GATED, I8>;
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
    prm.n_tiles = (n_rsb / 2) * ((M + 255) / 256);
    prm.split = (GATED || I8) ? 1 : gemm_pair_ta_split(prm.n_tiles, prm.n_ksteps, num_sms, scratch && counters);
    prm.scratch = scratch;
    prm.counters = counters;
    prm.n_whole = prm.n_tiles;
    const int units = prm.n_tiles * prm.split;
    const int n_clusters = units < num_sms / 2 ? units : num_sms / 2;

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
    if (cudaLaunchKernelEx(&cfg, kern, maps, prm) != cudaSuccess) {
        cudaGetLastError();
        return QL_ERR_CUDA;
    }
    return QL_OK;
}

// Any M the prefill path sees (tokens beyond M are zero-filled by TMA and never stored): below 129 tokens the tile is
// mostly padding, but the launch is bound by streaming and dequantising the weights, which this kernel spreads over
// the whole GPU (K split), not by the MMAs.
inline bool gemm_pair_ta_applicable(const GemmPairLayers& set, int M, int num_sms, bool gated = false)
{
    if (!gemm_config().ta || !gemm_config().pair) return false;
    for (int i = 0; i < set.n; ++i)
        if (!set.wmap[i] || (set.L[i]->n_rsb % 2)) return false;
    // the gated form needs a whole number of positions per round of the grid's clusters to be worth it; the plain form
    // takes every launch (few tiles: fewer clusters, or a K split through the device scratch)
    return !gated || (M > 128 && (set.L[0]->n_rsb / 2) * ((M + 255) / 256) >= num_sms / 2);
}

inline ql_status gemm_pair_ta_forward(const GemmPairLayers& set, const void* x, int M, cudaStream_t st, int device, bool pdl, int num_sms,
                                      float* scratch, unsigned int* counters)
{
    const Layout& L = *set.L[0];
    // a caller that keeps its outputs in the scratch itself (the unfused gating route) gets no K split
    const unsigned char* s0 = reinterpret_cast<const unsigned char*>(scratch);
    for (int i = 0; i < set.n && scratch; ++i) {
        const unsigned char* y = static_cast<const unsigned char*>(set.y[i]);
        if (y >= s0 && y < s0 + gemm_pair_scratch_bytes(num_sms)) scratch = nullptr;
    }
    if (L.bits == 8) return gemm_pair_ta_launch<8, false>(set, x, M, st, device, pdl, num_sms, -1, scratch, counters);
    if (L.grouped) return gemm_pair_ta_launch<4, true>(set, x, M, st, device, pdl, num_sms, -1, scratch, counters);
    return gemm_pair_ta_launch<4, false>(set, x, M, st, device, pdl, num_sms, -1, scratch, counters);
}

// Gated form: set = {gate, up}, both pair-applicable and of equal shape; y[0] receives act(gate) * up.
inline ql_status gemm_pair_ta_forward_gated(const GemmPairLayers& set, const void* x, int M, int act, cudaStream_t st, int device, bool pdl, int num_sms)
{
    const Layout& L = *set.L[0];
    if (L.bits == 8) return gemm_pair_ta_launch<8, false, true>(set, x, M, st, device, pdl, num_sms, act);
    if (L.grouped) return gemm_pair_ta_launch<4, true, true>(set, x, M, st, device, pdl, num_sms, act);
    return gemm_pair_ta_launch<4, false, true>(set, x, M, st, device, pdl, num_sms, act);
}

// Integer form (per-channel schemes, K a multiple of 128): xq int8 [M, K] with per-token scale and row sum; set.wmap
// holds the integer form's weight maps.  No K split: launches with fewer tiles than half the CTA pairs stay on the
// shared-memory kernel.
inline bool gemm_pair_ta_i8_applicable(const GemmPairLayers& set, int M, int num_sms)
{
    if (!gemm_config().ta || M <= 128 || !set.wmap[0]) return false;
    return set.L[0]->n_rsb / 2 * ((M + 255) / 256) * 2 > num_sms / 2;
}
inline ql_status gemm_pair_ta_forward_i8(const GemmPairLayers& set, const void* xq, const float* scale, const int32_t* rowsum, int M,
                                         cudaStream_t st, int device, bool pdl, int num_sms)
{
    const Layout& L = *set.L[0];
    if (L.bits == 8) return gemm_pair_ta_launch<8, false, false, true>(set, xq, M, st, device, pdl, num_sms, -1, nullptr, nullptr, scale, rowsum);
    return gemm_pair_ta_launch<4, false, false, true>(set, xq, M, st, device, pdl, num_sms, -1, nullptr, nullptr, scale, rowsum);
}

// The CTA-pair prefill call: the tensor-memory form where it applies, else the shared-memory form.
inline ql_status gemm_pair_forward_auto(const GemmPairLayers& set, const void* x, int M, cudaStream_t st,
                                        int device, bool pdl, int num_sms, float* scratch, unsigned int* counters)
{
    if (gemm_pair_ta_applicable(set, M, num_sms)) return gemm_pair_ta_forward(set, x, M, st, device, pdl, num_sms, scratch, counters);
    for (int i = 0; i < set.n; ++i)
        if (!gemm_pair_applicable(*set.L[i], M)) return QL_ERR_UNSUPPORTED;
    return gemm_pair_forward(set, x, M, st, device, pdl, num_sms, scratch, counters);
}

}  // namespace ql
