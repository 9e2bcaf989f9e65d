// Prefill kernel: y = x . W^T for M > 8 tokens on the 5th-generation tensor cores
// (paper Section 3.7: the compute-bound prefill stage gets its own matrix-multiply kernel reading
// the same resident weights; Section 4.2: prefill speed does not depend on the quantisation scheme).
//
// The product is computed transposed, D[n, m] = sum_k W[n,k] * x[m,k]: the 128 output channels of a
// row super-block are the MMA's M dimension, the tokens its N dimension, so that each dequantised
// weight is reused by up to 256 tokens.  Per CTA:
//
//   warp 0       producer: one bulk copy of the packed weight block(s) of the k-step (contiguous in
//                the blob) and one TMA tile load of x [BN tokens x 64 k] (128-byte swizzle)
//   warps 2..9   dequantise: packed block (shared) -> registers -> exact fp16 integers (x group scale
//                for grouped int4) -> the K-major 128-byte-swizzled A tile in shared memory
//   warp 1       issues tcgen05.mma (A, B from shared memory, fp32 accumulator in tensor memory) and
//                frees pipeline stages with tcgen05.commit
//   warps 2..9   epilogue: tcgen05.ld the accumulator, apply the per-channel scale, round to fp16, store
//
// Every mbarrier wait is bounded: on expiry the kernel records a code in g_device_flag, every role
// leaves its loop, tensor memory is released and the kernel returns.
#pragma once
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/qlinear.h"
#include "dequant.cuh"
#include "layout.h"
#include "sm100_ptx.cuh"

namespace ql {

constexpr int kGemmThreads = 320;            // 10 warps
constexpr int kGemmDequantWarps = 8;
constexpr int kGemmKStep = 64;               // k per pipeline stage = one 128-byte swizzle row of fp16
constexpr int kGemmATileBytes = 128 * 128;   // 128 rows x 64 fp16

struct GemmParams {
    const uint8_t* body;
    const __half* chan_scales;
    __half* y;
    int32_t M, N, K;
    int32_t n_kc, block_bytes;
    int32_t n_ksteps;
};

struct GemmPlan {
    int32_t dummy;
};

// ----------------------------------------------------------------------------- shared-memory plan
template <int BITS, int BN>
struct GemmSmem {
    static constexpr int kWpkBytes = BITS == 4 ? (kWeightBlockBytes + kScaleBlockBytes) : 2 * kWeightBlockBytes;
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
    auto full_bar = [&](int s) { return bar0 + 8 * s; };
    auto afull_bar = [&](int s) { return bar0 + 8 * (NS + s); };
    auto empty_bar = [&](int s) { return bar0 + 8 * (2 * NS + s); };
    const uint32_t accum_bar = bar0 + 8 * (3 * NS);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + S::kBarOffset + 8 * (3 * NS + 1));
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rsb = blockIdx.x, m0 = blockIdx.y * BN;
    const int n_steps = p.n_ksteps;

    if (threadIdx.x == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(afull_bar(s), kGemmDequantWarps);
            mbar_init(empty_bar(s), 1);
        }
        mbar_init(accum_bar, 1);
        abort_flag[0] = 0;
        abort_flag[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32((const void*)tmem_slot), BN);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&x_map) : "memory");
            constexpr int CHUNKS = BITS == 4 ? 1 : 2;                    // packed blocks per 64-k step
            const uint8_t* wsrc = p.body + (int64_t)rsb * p.n_kc * p.block_bytes;
            int issued = 0;
            bool waited_dep = false;
            for (int it = 0; it < n_steps; ++it) {
                const int s = it % NS, r = it / NS;
                if (!mbar_wait(empty_bar(s), (r & 1) ^ 1, abort_flag, 0x100 + s)) break;
                const int kc = it * CHUNKS;
                const int nblk = min(CHUNKS, p.n_kc - kc);
                const uint32_t wbytes = (uint32_t)nblk * p.block_bytes;
                mbar_expect_tx(full_bar(s), wbytes + S::kXBytes);
                bulk_copy_g2s(wpk_addr(s), wsrc + (int64_t)kc * p.block_bytes, wbytes, full_bar(s));
                if (!waited_dep) {                                       // x may come from the previous kernel
                    asm volatile("griddepcontrol.wait;" ::: "memory");
                    waited_dep = true;
                }
                tma_load_2d(xs_addr(s), &x_map, it * kGemmKStep, m0, full_bar(s));
                ++issued;
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
            bool ok = true;
            for (int it = 0; it < n_steps && ok; ++it) {
                const int s = it % NS, r = it / NS;
                ok = mbar_wait(full_bar(s), r & 1, abort_flag, 0x200 + s) &&
                     mbar_wait(afull_bar(s), r & 1, abort_flag, 0x300 + s);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int k4 = 0; k4 < kGemmKStep / 16; ++k4) {
                    const uint64_t ad = umma_desc_sw128(a_addr(s) + k4 * 32);
                    const uint64_t bd = umma_desc_sw128(xs_addr(s) + k4 * 32);
                    umma_f16(tmem_base, ad, bd, idesc, (it > 0 || k4 > 0) ? 1u : 0u);
                }
                umma_commit(empty_bar(s));
            }
            umma_commit(accum_bar);
        }
    } else {
        // ------------------------------------------------------------------ dequantise, then epilogue
        const int dw = warp - 2;                                         // 0..7 = row-block of the tile
        const int g = lane >> 2, c = lane & 3;
        const int row0 = dw * kRbRows + g;                               // rows row0 and row0 + 8
        const uint32_t sw = (uint32_t)g;                                 // (row & 7) of both rows
        bool ok = true;
        for (int it = 0; it < n_steps && ok; ++it) {
            const int s = it % NS, r = it / NS;
            ok = mbar_wait(full_bar(s), r & 1, abort_flag, 0x400 + s);
            if (!ok) break;
            const unsigned char* wp = wpk_ptr(s);
            unsigned char* at = a_ptr(s);
            if (BITS == 4) {
                const uint4 w = *reinterpret_cast<const uint4*>(wp + dw * 512 + lane * 16);
                uint32_t lo[4], hi[4];                                   // words 0,1 -> k 8c..8c+7; words 2,3 -> 32+8c..
                uint32_t a0[4], a1[4];
                unpack_int4_word(w.x, a0);
                unpack_int4_word(w.y, a1);
                lo[0] = a0[0]; lo[1] = a0[2]; lo[2] = a1[0]; lo[3] = a1[2];        // row0,   unit c
                hi[0] = a0[1]; hi[1] = a0[3]; hi[2] = a1[1]; hi[3] = a1[3];        // row0+8, unit c
                uint32_t lo2[4], hi2[4];
                unpack_int4_word(w.z, a0);
                unpack_int4_word(w.w, a1);
                lo2[0] = a0[0]; lo2[1] = a0[2]; lo2[2] = a1[0]; lo2[3] = a1[2];    // row0,   unit 4+c
                hi2[0] = a0[1]; hi2[1] = a0[3]; hi2[2] = a1[1]; hi2[3] = a1[3];    // row0+8, unit 4+c
                if (GROUPED) {
                    const uint2 sc = *reinterpret_cast<const uint2*>(wp + kWeightBlockBytes + dw * 64 + g * 8);
                    const uint32_t s_g0 = __byte_perm(sc.x, 0, 0x1010), s_g1 = __byte_perm(sc.x, 0, 0x3232);
                    const uint32_t s_h0 = __byte_perm(sc.y, 0, 0x1010), s_h1 = __byte_perm(sc.y, 0, 0x3232);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        lo[i] = h2_mul(lo[i], s_g0);  lo2[i] = h2_mul(lo2[i], s_g1);
                        hi[i] = h2_mul(hi[i], s_h0);  hi2[i] = h2_mul(hi2[i], s_h1);
                    }
                }
                const uint32_t u0 = ((uint32_t)c ^ sw) * 16, u1 = ((uint32_t)(4 + c) ^ sw) * 16;
                *reinterpret_cast<uint4*>(at + row0 * 128 + u0) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                *reinterpret_cast<uint4*>(at + row0 * 128 + u1) = make_uint4(lo2[0], lo2[1], lo2[2], lo2[3]);
                *reinterpret_cast<uint4*>(at + (row0 + 8) * 128 + u0) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                *reinterpret_cast<uint4*>(at + (row0 + 8) * 128 + u1) = make_uint4(hi2[0], hi2[1], hi2[2], hi2[3]);
            } else {
#pragma unroll
                for (int j = 0; j < 2; ++j) {                            // two 32-k chunks per step
                    const uint4 w = *reinterpret_cast<const uint4*>(wp + j * kWeightBlockBytes + dw * 512 + lane * 16);
                    uint32_t a0[4], a1[4];
                    unpack_int8_words(w.x, w.y, a0);
                    unpack_int8_words(w.z, w.w, a1);
                    const uint32_t u = ((uint32_t)(4 * j + c) ^ sw) * 16;
                    *reinterpret_cast<uint4*>(at + row0 * 128 + u) = make_uint4(a0[0], a0[2], a1[0], a1[2]);
                    *reinterpret_cast<uint4*>(at + (row0 + 8) * 128 + u) = make_uint4(a0[1], a0[3], a1[1], a1[3]);
                }
            }
            fence_async_smem();                                          // generic-proxy writes -> visible to the MMA
            __syncwarp();
            if (lane == 0) mbar_arrive(afull_bar(s));
        }

        // epilogue: warp (dw & 3) + 2 owns the TMEM lane quarter (warp % 4); two warps split the columns
        if (ok) ok = mbar_wait(accum_bar, 0, abort_flag, 0x500);
        if (ok) {
            tc_fence_after();
            const int quarter = warp & 3;
            const int half = dw >> 2;
            const int n = rsb * kRsbRows + quarter * 32 + lane;
            float scale = 1.f;
            if (!GROUPED && n < p.N) scale = __half2float(p.chan_scales[n]);
            constexpr int CW = BN / 2;
#pragma unroll 1
            for (int cc = 0; cc < CW; cc += 16) {
                const int col0 = half * CW + cc;
                if (m0 + col0 >= p.M) break;
                uint32_t r[16];
                tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)col0, r);
                if (n < p.N) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int m = m0 + col0 + j;
                        if (m < p.M) p.y[(int64_t)m * p.N + n] = __float2half_rn(__uint_as_float(r[j]) * scale);
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, BN);
    }
}

// ----------------------------------------------------------------------------- host side
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

inline ql_status gemm_plan(const Layout&, int, GemmPlan* p)
{
    p->dummy = 0;
    return QL_OK;
}

inline int gemm_pick_bn(const Layout& L, int M, int num_sms)
{
    const char* f = std::getenv("QLINEAR_GEMM_BN");
    if (f && *f) return std::atoi(f);
    if (M <= 32) return 32;
    if (M <= 64) return 64;
    if (M <= 128) return 128;
    // prefer the widest tile unless it leaves most SMs idle
    const int tiles256 = L.n_rsb * ((M + 255) / 256);
    if (tiles256 * 2 <= num_sms) return 128;
    return 256;
}

template <int BITS, bool GROUPED, int BN>
ql_status gemm_launch(const Layout& L, const uint8_t* blob, const void* x, void* y, int M, cudaStream_t st, int device, bool pdl)
{
    using S = GemmSmem<BITS, BN>;
    static_assert(S::kStages >= 2, "pipeline needs at least two stages");
    EncodeTiledFn enc = get_encode_tiled();
    if (!enc) return QL_ERR_CUDA;
    CUtensorMap map;
    const cuuint64_t gdim[2] = {(cuuint64_t)L.K, (cuuint64_t)M};
    const cuuint64_t gstr[1] = {(cuuint64_t)L.K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kGemmKStep, (cuuint32_t)BN};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(x), gdim, gstr, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return QL_ERR_CUDA;

    auto kern = gemm_kernel<BITS, GROUPED, BN>;
    static bool attr_set[64] = {};
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

    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(L.n_rsb, (M + BN - 1) / BN);
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
                           int device, bool pdl)
{
    switch (bn) {
        case 32: return gemm_launch<BITS, GROUPED, 32>(L, blob, x, y, M, st, device, pdl);
        case 64: return gemm_launch<BITS, GROUPED, 64>(L, blob, x, y, M, st, device, pdl);
        case 128: return gemm_launch<BITS, GROUPED, 128>(L, blob, x, y, M, st, device, pdl);
        case 256: return gemm_launch<BITS, GROUPED, 256>(L, blob, x, y, M, st, device, pdl);
    }
    return QL_ERR_INVALID_ARG;
}

inline ql_status gemm_forward(const Layout& L, const GemmPlan&, const uint8_t* blob, const void* x, void* y, int M,
                              cudaStream_t st, int device, bool pdl, int num_sms)
{
    const int bn = gemm_pick_bn(L, M, num_sms);
    if (L.bits == 8) return gemm_dispatch_bn<8, false>(bn, L, blob, x, y, M, st, device, pdl);
    if (L.grouped) return gemm_dispatch_bn<4, true>(bn, L, blob, x, y, M, st, device, pdl);
    return gemm_dispatch_bn<4, false>(bn, L, blob, x, y, M, st, device, pdl);
}

}  // namespace ql
