// Prefill kernel: y = x . W^T for M > 8 tokens on the 5th-generation tensor cores
// (paper Section 3.7: the compute-bound prefill stage gets its own matrix-multiply kernel reading
// the same resident weights; Section 4.2: prefill speed does not depend on the quantisation scheme).
//
// The product is computed transposed, D[n, m] = sum_k W[n,k] * x[m,k]: the 128 output channels of a
// row super-block are the MMA's M dimension, the tokens its N dimension, so that each dequantised
// weight is reused by up to 256 tokens.  The grid is persistent (one CTA per SM, tiles assigned
// round-robin) and the accumulator is double-buffered in tensor memory, so the epilogue of one tile
// runs under the main loop of the next.  Per CTA:
//
//   warp 0        producer: one bulk copy of the packed weight block(s) of the k-step (contiguous in
//                 the blob) and one TMA tile load of x [BN tokens x 64 k] (128-byte swizzle; every CTA loads for itself)
//   warps 2..17   dequantise: packed block (shared) -> registers -> exact fp16 integers (x group scale
//                 for grouped int4) -> the K-major 128-byte-swizzled A tile in shared memory
//   warp 1        issues tcgen05.mma (A, B from shared memory, fp32 accumulator in tensor memory),
//                 frees pipeline stages and publishes finished accumulators with tcgen05.commit
//   warps 18..21  epilogue: tcgen05.ld the accumulator, apply the per-channel scale, round to fp16, store
//
// Every mbarrier wait is bounded: on expiry the kernel records a code in g_device_flag, every role
// leaves its loop, tensor memory is released and the kernel returns.
#pragma once
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <mutex>

#include "../../include/qlinear.h"
#include "dequant.cuh"
#include "layout.h"
#include "sm100_ptx.cuh"

namespace ql {

constexpr int kGemmDequantWarps = 16;
constexpr int kGemmEpilogueWarps = 4;
constexpr int kGemmThreads = (2 + kGemmDequantWarps + kGemmEpilogueWarps) * 32;   // 22 warps
constexpr int kGemmKStep = 64;               // k per pipeline stage = one 128-byte swizzle row of fp16
constexpr int kGemmATileBytes = 128 * 128;   // 128 rows x 64 fp16

struct GemmParams {
    const uint8_t* body;
    const __half* chan_scales;
    __half* y;
    int32_t M, N, K;
    int32_t n_kc, block_bytes;
    int32_t n_ksteps;
    int32_t n_rsb, n_tiles;                  // work units of the grid (pair kernel: tiles x split)
    int32_t split;                           // pair kernel: K parts of the tiles that are split (1 = none are)
    int32_t n_whole;                         // pair kernel: units [0, n_whole) are whole tiles, the rest are parts
    float* scratch;                          // pair kernel, split > 1: fp32 partial tiles [tile][part][rank][256][128]
    unsigned int* counters;                  // pair kernel, split > 1: arrivals per (tile, rank, quarter), zero between launches
    // pair kernel: up to kGemmMaxGroup layers that read the same x in one launch; their row super-blocks are
    // numbered one after the other, rsb_end[i] = row super-blocks of layers 0..i (each layer an even number)
    const uint8_t* lbody[4];
    const __half* lscales[4];
    __half* ly[4];
    int32_t lN[4];
    int32_t rsb_end[4];
    int32_t n_layers;
    int32_t act;                             // pair kernel, gated form: activation of the gate branch (QL_ACT_*)
    // pair kernel, integer form (x_map then describes the int8 activations): per-token scale and sum of the
    // quantised row (device arrays, padded to whole token tiles)
    const float* a8_scale;
    const int32_t* a8_rowsum;
};
constexpr int kGemmMaxGroup = 4;

// Per-lane constants and the per-step work of a dequantise warp (shared by the 1-CTA and 2-CTA kernels).
// Warp dw handles row-block (dw & 7); of each lane's 16 packed bytes (two 32-wide k halves) a lane
// converts one half per step: half (dw >> 3) for even g, the other one for odd g; the partner warp
// (dw ^ 8) takes the rest.  Swizzled, the 8 lanes of a quarter-warp then store to 8 different 16-byte
// columns: no bank conflicts.
struct DequantLane {
    int half;
    uint32_t off_lo, off_hi, s_sel;
    int w_off4, w_off8, s_off;
    __device__ DequantLane(int dw, int lane)
    {
        const int g = lane >> 2, c = lane & 3;
        const int row0 = (dw & 7) * kRbRows + g;                         // rows row0 and row0 + 8 ((row & 7) == g)
        half = (dw >> 3) ^ (g & 1);                                      // which 32-k half of the 64-k step
        const uint32_t unit = ((uint32_t)(4 * half + c) ^ (uint32_t)g) * 16;
        off_lo = row0 * 128 + unit;
        off_hi = (row0 + 8) * 128 + unit;
        w_off4 = (dw & 7) * 512 + lane * 16 + 8 * half;
        w_off8 = half * kWeightBlockBytes + (dw & 7) * 512 + lane * 16;
        s_off = kWeightBlockBytes + (dw & 7) * 64 + g * 8;
        s_sel = half ? 0x3232u : 0x1010u;                                // broadcast the scale of this half's group
    }
    template <int BITS, bool GROUPED>
    __device__ __forceinline__ void step(const unsigned char* wp, unsigned char* at) const
    {
        uint32_t a0[4], a1[4];
        if (BITS == 4) {
            const uint2 w = *reinterpret_cast<const uint2*>(wp + w_off4);
            unpack_int4_word(w.x, a0);                                   // k 32*half + 8c     .. + 3
            unpack_int4_word(w.y, a1);                                   // k 32*half + 8c + 4 .. + 7
        } else {
            const uint4 w = *reinterpret_cast<const uint4*>(wp + w_off8);
            unpack_int8_words(w.x, w.y, a0);
            unpack_int8_words(w.z, w.w, a1);
        }
        uint4 lo = make_uint4(a0[0], a0[2], a1[0], a1[2]);               // row0
        uint4 hi = make_uint4(a0[1], a0[3], a1[1], a1[3]);               // row0 + 8
        if (GROUPED) {
            const uint2 sc = *reinterpret_cast<const uint2*>(wp + s_off);
            const uint32_t s_lo = __byte_perm(sc.x, 0, s_sel), s_hi = __byte_perm(sc.y, 0, s_sel);
            lo.x = h2_mul(lo.x, s_lo); lo.y = h2_mul(lo.y, s_lo); lo.z = h2_mul(lo.z, s_lo); lo.w = h2_mul(lo.w, s_lo);
            hi.x = h2_mul(hi.x, s_hi); hi.y = h2_mul(hi.y, s_hi); hi.z = h2_mul(hi.z, s_hi); hi.w = h2_mul(hi.w, s_hi);
        }
        *reinterpret_cast<uint4*>(at + off_lo) = lo;
        *reinterpret_cast<uint4*>(at + off_hi) = hi;
    }
};

// The integer form's counterpart (paper Section 3.7: pre-quantised weights meet int8 activations in integer
// instructions): the stored weight integers, as they are (q + 8 or q + 128, unsigned), become the K-major
// 128-byte-swizzled u8 tile of a 128-k step.  Warp dw handles row-block (dw & 7) and half of the step's chunks.
struct RepackLane {
    int rbk, half, g, c, lane;
    __device__ RepackLane(int dw, int lane_) : rbk(dw & 7), half(dw >> 3), g(lane_ >> 2), c(lane_ & 3), lane(lane_) {}
    // 8 bytes (k0 .. k0 + 7, k0 a multiple of 8) of tile row r
    __device__ __forceinline__ static void store8(unsigned char* at, int r, int k0, uint32_t lo, uint32_t hi)
    {
        *reinterpret_cast<uint2*>(at + r * 128 + ((((k0 >> 4) ^ (r & 7)) << 4) | (k0 & 8))) = make_uint2(lo, hi);
    }
    template <int BITS>
    __device__ __forceinline__ void step(const unsigned char* wp, unsigned char* at) const
    {
        const int r0 = rbk * kRbRows + g;                                // rows r0 and r0 + 8
        if (BITS == 8) {                                                 // 4 chunks of 32 k per step, two per warp
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int ch = 2 * half + j;
                const uint4 w = *reinterpret_cast<const uint4*>(wp + ch * kWeightBlockBytes + rbk * 512 + lane * 16);
                const int k0 = 32 * ch + 8 * c;
                store8(at, r0, k0, __byte_perm(w.x, w.y, 0x5410), __byte_perm(w.z, w.w, 0x5410));
                store8(at, r0 + 8, k0, __byte_perm(w.x, w.y, 0x7632), __byte_perm(w.z, w.w, 0x7632));
            }
        } else {                                                         // 2 chunks of 64 k per step, one per warp
            const uint4 w = *reinterpret_cast<const uint4*>(wp + half * kWeightBlockBytes + rbk * 512 + lane * 16);
            const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int h = 0; h < 2; ++h) {                                // the chunk's two 32-k halves
                // low nibbles of a word: row g at slots 0, 2, 1, 3; high nibbles: row g + 8 (layout.h)
                const uint32_t a = ww[2 * h], b = ww[2 * h + 1];
                const int k0 = 64 * half + 32 * h + 8 * c;
                store8(at, r0, k0, __byte_perm(a & 0x0F0F0F0Fu, 0, 0x3120), __byte_perm(b & 0x0F0F0F0Fu, 0, 0x3120));
                store8(at, r0 + 8, k0, __byte_perm((a >> 4) & 0x0F0F0F0Fu, 0, 0x3120), __byte_perm((b >> 4) & 0x0F0F0F0Fu, 0, 0x3120));
            }
        }
    }
};

// ----------------------------------------------------------------------------- shared-memory plan
template <int BITS, int BN>
struct GemmSmem {
    static constexpr int kWpkStride = 8192;                              // keeps every tile 1024-byte aligned
    static constexpr int kXBytes = BN * 128;
    static constexpr int kStageBytes = kXBytes + kGemmATileBytes + kWpkStride;
    static constexpr int kStages = (200 * 1024) / kStageBytes > 6 ? 6 : (200 * 1024) / kStageBytes;
    static constexpr int kBarOffset = kStages * kStageBytes;
    static constexpr int kTotal = kBarOffset + 256 + 1024;              // barriers + alignment slack
};

template <int BITS, bool GROUPED, int BN>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap x_map, const GemmParams p)
{
    using S = GemmSmem<BITS, BN>;
    constexpr int NS = S::kStages;
    extern __shared__ unsigned char smem_dyn[];
    const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
    auto xs_addr = [&](int s) { return base + s * S::kStageBytes; };
    auto a_addr = [&](int s) { return base + s * S::kStageBytes + S::kXBytes; };
    auto wpk_addr = [&](int s) { return base + s * S::kStageBytes + S::kXBytes + kGemmATileBytes; };
    auto wpk_ptr = [&](int s) { return base_ptr + s * S::kStageBytes + S::kXBytes + kGemmATileBytes; };
    auto a_ptr = [&](int s) { return base_ptr + s * S::kStageBytes + S::kXBytes; };
    const uint32_t bar0 = base + S::kBarOffset;
    auto full_bar = [&](int s) { return bar0 + 8 * s; };                 // TMA data of stage s landed
    auto afull_bar = [&](int s) { return bar0 + 8 * (NS + s); };         // A tile of stage s dequantised
    auto empty_bar = [&](int s) { return bar0 + 8 * (2 * NS + s); };     // MMAs of stage s retired
    auto tfull_bar = [&](int b) { return bar0 + 8 * (3 * NS + b); };     // accumulator b complete
    auto tempty_bar = [&](int b) { return bar0 + 8 * (3 * NS + 2 + b); };// accumulator b drained by the epilogue
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + S::kBarOffset + 8 * (3 * NS + 4));
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_steps = p.n_ksteps;
    const int first_tile = blockIdx.x, tile_stride = gridDim.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(afull_bar(s), kGemmDequantWarps);
            mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(tfull_bar(b), 1);
            mbar_init(tempty_bar(b), kGemmEpilogueWarps);
        }
        abort_flag[0] = 0;                                               // [0] abort, [1] abort of the exit drain,
        abort_flag[1] = 0;                                               // [2], [3] "past griddepcontrol.wait" (see wait_expired)
        abort_flag[2] = 0;
        abort_flag[3] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32((const void*)tmem_slot), 2 * BN);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&x_map) : "memory");
            constexpr int CHUNKS = BITS == 4 ? 1 : 2;                    // packed blocks per 64-k step
            int s = 0, issued = 0;
            uint32_t par = 1;                                            // first pass: stages start out free
            bool waited_dep = false, ok = true;
            for (int t = first_tile; t < p.n_tiles && ok; t += tile_stride) {
                const int rsb = t % p.n_rsb, m0 = (t / p.n_rsb) * BN;
                const uint8_t* wsrc = p.body + (int64_t)rsb * p.n_kc * p.block_bytes;
                for (int it = 0; it < n_steps; ++it) {
                    if (!mbar_wait(empty_bar(s), par, abort_flag, 0x100 + s)) { ok = false; break; }
                    const int kc = it * CHUNKS;
                    const int nblk = min(CHUNKS, p.n_kc - kc);
                    const uint32_t wbytes = (uint32_t)nblk * p.block_bytes;
                    mbar_expect_tx(full_bar(s), wbytes + S::kXBytes);
                    bulk_copy_g2s(wpk_addr(s), wsrc + (int64_t)kc * p.block_bytes, wbytes, full_bar(s));
                    if (!waited_dep) {                                   // x may come from the previous kernel
                        asm volatile("griddepcontrol.wait;" ::: "memory");
                        waited_dep = true;
                        abort_flag[2] = 1;                               // from here on, waiting counts against the time limit
                        abort_flag[3] = 1;
                    }
                    tma_load_2d(xs_addr(s), &x_map, it * kGemmKStep, m0, full_bar(s));
                    ++issued;
                    if (++s == NS) { s = 0; par ^= 1; }
                }
            }
            if (*abort_flag) {                                           // let copies in flight land before exit
                for (int j = max(0, issued - NS); j < issued; ++j)
                    mbar_wait(full_bar(j % NS), (j / NS) & 1, abort_flag + 1, 0);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_f16(BN);
            const uint32_t a_lo0 = umma_desc_lo(a_addr(0)), b_lo0 = umma_desc_lo(xs_addr(0));
            int s = 0;
            uint32_t par = 0;
            bool ok = true;
            int j = 0;                                                   // local tile counter
            for (int t = first_tile; t < p.n_tiles && ok; t += tile_stride, ++j) {
                const int buf = j & 1;
                const uint32_t use = (uint32_t)(j >> 1);
                // accumulator buf must have been drained by the epilogue of its previous use
                if (!mbar_wait(tempty_bar(buf), (use & 1) ^ 1, abort_flag, 0x800 + buf)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + (uint32_t)(buf * BN);
                for (int it = 0; it < n_steps; ++it) {
                    // A tile written; the dequantise warps waited for the stage's TMA data, so x landed too
                    ok = mbar_wait(afull_bar(s), par, abort_flag, 0x300 + s);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_lo = a_lo0 + (uint32_t)s * (S::kStageBytes >> 4);
                    const uint32_t b_lo = b_lo0 + (uint32_t)s * (S::kStageBytes >> 4);
                    umma_f16_lo(tmem_d, a_lo, b_lo, idesc, it > 0 ? 1u : 0u);
#pragma unroll
                    for (int k4 = 1; k4 < kGemmKStep / 16; ++k4)         // +32 bytes along K inside the swizzle row
                        umma_f16_lo(tmem_d, a_lo + 2 * k4, b_lo + 2 * k4, idesc, 1u);
                    umma_commit(empty_bar(s));
                    if (++s == NS) { s = 0; par ^= 1; }
                }
                umma_commit(tfull_bar(buf));
            }
        }
    } else if (warp < 2 + kGemmDequantWarps) {
        // ------------------------------------------------------------------ dequantise
        // Warp dw handles row-block (dw & 7); of each lane's 16 packed bytes (two 32-wide k halves) a
        // lane converts one half per step: half (dw >> 3) for even g, the other one for odd g, the
        // partner warp (dw ^ 8) takes the rest.  Swizzled, the 8 lanes of a quarter-warp then store to
        // 8 different 16-byte columns: no bank conflicts.
        const DequantLane dq(warp - 2, lane);
        int s = 0;
        uint32_t par = 0;
        bool ok = true;
        int gstep = 0;
        for (int t = first_tile; t < p.n_tiles && ok; t += tile_stride) {
            for (int it = 0; it < n_steps; ++it, ++gstep) {
                if (!mbar_wait(full_bar(s), par, abort_flag, 0x400 + s)) { ok = false; break; }
                dq.template step<BITS, GROUPED>(wpk_ptr(s), a_ptr(s));
                fence_async_smem();                                      // generic-proxy writes -> visible to the MMA
                __syncwarp();
                if (lane == 0) mbar_arrive(afull_bar(s));
                if (++s == NS) { s = 0; par ^= 1; }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        const int quarter = warp & 3;                                    // TMEM lanes 32*quarter .. +31
        bool ok = true;
        int j = 0;
        for (int t = first_tile; t < p.n_tiles && ok; t += tile_stride, ++j) {
            const int buf = j & 1;
            const uint32_t use = (uint32_t)(j >> 1);
            const int rsb = t % p.n_rsb, m0 = (t / p.n_rsb) * BN;
            if (!mbar_wait(tfull_bar(buf), use & 1, abort_flag, 0x500 + buf)) { ok = false; break; }
            tc_fence_after();
            const int n = rsb * kRsbRows + quarter * 32 + lane;
            float scale = 1.f;
            if (!GROUPED && n < p.N) scale = __half2float(p.chan_scales[n]);
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * BN);
            __half* yrow = p.y + (int64_t)m0 * p.N + n;
            const int m_left = p.M - m0;
#pragma unroll 1
            for (int cc = 0; cc < BN; cc += 16) {
                if (cc >= m_left) break;
                uint32_t r[16];
                tmem_ld16(taddr + (uint32_t)cc, r);
                if (n < p.N) {
#pragma unroll
                    for (int q = 0; q < 16; ++q)
                        if (cc + q < m_left) yrow[(int64_t)(cc + q) * p.N] = __float2half_rn(__uint_as_float(r[q]) * scale);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(buf));
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 2 * BN);
    }
}

// ----------------------------------------------------------------------------- host side
// Tuning switches of the prefill kernels, read from the environment once per process (see library_config()).
struct GemmConfig {
    int force_bn = 0;        // QLINEAR_GEMM_BN: token-tile width of the single-CTA kernel (0 = choose per shape)
    int force_split = 0;     // QLINEAR_GEMM_SPLIT: K parts of single-round layers in the CTA-pair kernel (0 = choose)
    int force_tb = 0;        // QLINEAR_GEMM_TB: token blocks per tile of the CTA-pair kernel (0 = choose)
    bool pair = true;        // QLINEAR_GEMM_PAIR=0 switches the CTA-pair kernel off
    bool ta = true;          // QLINEAR_GEMM_TA=0 switches off the CTA-pair kernel that keeps the dequantised weights in tensor memory
};
GemmConfig& gemm_config();

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn get_encode_tiled()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
        else
            cudaGetLastError();
    }
    return fn;
}

// The tensor map of x depends only on (pointer, K, M, box rows); callers reuse a few activation buffers, so the
// last encodings are kept (per process, a handful of entries) instead of calling the driver on every forward.
// elem_bytes: 2 = fp16 activations (box 64 k wide), 1 = int8 activations (box 128 k wide); either way 128 bytes.
inline bool x_tensor_map(const void* x, int K, int M, int box_rows, CUtensorMap* out, int elem_bytes = 2)
{
    struct Entry { const void* x; int K, M, rows, eb; CUtensorMap map; };
    constexpr int kEntries = 16;
    static Entry cache[kEntries] = {};
    static int next = 0;
    static std::mutex mu;
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < kEntries; ++i)
        if (cache[i].x == x && cache[i].K == K && cache[i].M == M && cache[i].rows == box_rows && cache[i].eb == elem_bytes) { *out = cache[i].map; return true; }
    EncodeTiledFn enc = get_encode_tiled();
    if (!enc) return false;
    const cuuint64_t gdim[2] = {(cuuint64_t)K, (cuuint64_t)M};
    const cuuint64_t gstr[1] = {(cuuint64_t)K * elem_bytes};
    const cuuint32_t box[2] = {(cuuint32_t)(128 / elem_bytes), (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    Entry e{x, K, M, box_rows, elem_bytes, {}};
    if (enc(&e.map, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(x), gdim, gstr, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    cache[next] = e;
    next = (next + 1) % kEntries;
    *out = e.map;
    return true;
}

inline int gemm_pick_bn(const Layout& L, int M, int num_sms)
{
    if (gemm_config().force_bn) return gemm_config().force_bn;
    if (M <= 32) return 32;
    if (M <= 64) return 64;
    if (M <= 128) return 128;
    // prefer the widest tile unless it leaves most SMs idle
    const int tiles256 = L.n_rsb * ((M + 255) / 256);
    if (tiles256 * 2 <= num_sms) return 128;
    return 256;
}

template <int BITS, bool GROUPED, int BN>
ql_status gemm_launch(const Layout& L, const uint8_t* blob, const void* x, void* y, int M, cudaStream_t st, int device, bool pdl, int num_sms)
{
    using S = GemmSmem<BITS, BN>;
    static_assert(S::kStages >= 2, "pipeline needs at least two stages");
    CUtensorMap map;
    if (!x_tensor_map(x, L.K, M, BN, &map)) return QL_ERR_CUDA;

    auto kern = gemm_kernel<BITS, GROUPED, BN>;
    static std::atomic<bool> attr_set[64];
    if (device >= 0 && device < 64 && !attr_set[device]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, S::kTotal) != cudaSuccess) {
            cudaGetLastError();
            return QL_ERR_CUDA;
        }
        attr_set[device] = true;
    }
    GemmParams prm{};
    prm.body = blob + L.body_offset;
    prm.chan_scales = L.grouped ? nullptr : reinterpret_cast<const __half*>(blob + L.chan_scale_offset);
    prm.y = static_cast<__half*>(y);
    prm.M = M; prm.N = L.N; prm.K = L.K;
    prm.n_kc = L.n_kc; prm.block_bytes = L.block_bytes;
    prm.n_ksteps = (L.K + kGemmKStep - 1) / kGemmKStep;
    prm.n_rsb = L.n_rsb;
    prm.n_tiles = L.n_rsb * ((M + BN - 1) / BN);

    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(prm.n_tiles < num_sms ? prm.n_tiles : num_sms);
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = S::kTotal;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    if (cudaLaunchKernelEx(&cfg, kern, map, prm) != cudaSuccess) {
        cudaGetLastError();
        return QL_ERR_CUDA;
    }
    return QL_OK;
}

template <int BITS, bool GROUPED>
ql_status gemm_dispatch_bn(int bn, const Layout& L, const uint8_t* blob, const void* x, void* y, int M, cudaStream_t st,
                           int device, bool pdl, int num_sms)
{
    switch (bn) {
        case 32: return gemm_launch<BITS, GROUPED, 32>(L, blob, x, y, M, st, device, pdl, num_sms);
        case 64: return gemm_launch<BITS, GROUPED, 64>(L, blob, x, y, M, st, device, pdl, num_sms);
        case 128: return gemm_launch<BITS, GROUPED, 128>(L, blob, x, y, M, st, device, pdl, num_sms);
        case 256: return gemm_launch<BITS, GROUPED, 256>(L, blob, x, y, M, st, device, pdl, num_sms);
    }
    return QL_ERR_INVALID_ARG;
}

inline ql_status gemm_forward(const Layout& L, const uint8_t* blob, const void* x, void* y, int M,
                              cudaStream_t st, int device, bool pdl, int num_sms)
{
    const int bn = gemm_pick_bn(L, M, num_sms);
    if (L.bits == 8) return gemm_dispatch_bn<8, false>(bn, L, blob, x, y, M, st, device, pdl, num_sms);
    if (L.grouped) return gemm_dispatch_bn<4, true>(bn, L, blob, x, y, M, st, device, pdl, num_sms);
    return gemm_dispatch_bn<4, false>(bn, L, blob, x, y, M, st, device, pdl, num_sms);
}

}  // namespace ql
