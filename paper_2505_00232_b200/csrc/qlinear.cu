// C-ABI of the qlinear library: handle life cycle, stage-aware dispatch (paper Section 3.7) and the
// launchers of the decode and prefill kernels.  Single translation unit for all device code.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>

#include "../../include/qlinear.h"
#include "layout.h"

namespace ql {
// Set by a kernel that gave up a bounded wait: [0] = non-zero code identifying the wait, [1] = count.
__device__ unsigned int g_device_flag[2];
}  // namespace ql

#include "dequant.cuh"
#include "embed.cuh"
#include "gemv.cuh"
#include "gemv_stream.cuh"
#include "gemm.cuh"
#include "gemm_pair.cuh"

using namespace ql;

struct GemvPlan {
    int32_t ks_cta, cl, cps, x_stride, x_bytes, smem_bytes, grid;
};

struct qlinear_s {
    Layout L;
    const uint8_t* blob;
    int device;
    int num_sms;
    int gemv_max_m;
    bool pdl;
    GemvPlan gemv[9];          // index = M (1..8)
    GemvPlan group_gemv[9];    // the same for the last group of layers launched with this one in front
    int group_rb;              // row-blocks of that group (0 = none yet)
    GemmPlan gemm;
    // streaming decode kernel
    int gemv_kernel_choice;    // 0 = cluster kernel, 1 = streaming kernel
    int stream_P, stream_stages;
    float* stream_scratch;     // device, owned: [P][2][1024] fp32 partial sums
    unsigned int* stream_counters;   // device, owned: [n_rsb][8], zero between launches
    // prefill pair kernel, K-split of skinny layers
    float* gemm_scratch;             // device, owned (nullptr if the layer can never be split)
    unsigned int* gemm_counters;     // device, owned, zero between launches
};

namespace {

constexpr int kGemvMaxSmem = 96 * 1024;

int env_int(const char* name, int dflt)
{
    const char* v = std::getenv(name);
    return (v && *v) ? std::atoi(v) : dflt;
}

// n_rb: row-blocks of the launch (one layer, or all layers of a group that shares x).
GemvPlan plan_gemv(const Layout& L, int n_rb, int M, int num_sms)
{
    const int warps_per_sm = env_int("QLINEAR_GEMV_WARPS_PER_SM", 32);
    const int force_ks = env_int("QLINEAR_GEMV_KS", 0);
    const int xdirect = env_int("QLINEAR_GEMV_XDIRECT", 1);
    const double target = (double)num_sms * warps_per_sm;
    GemvPlan best{};
    double best_score = -1e30;
    for (int ks_cta = 1; ks_cta <= 8; ks_cta *= 2)
        for (int cl = 1; cl <= (ks_cta == 8 ? 8 : 1); ++cl) {
            const int ks = ks_cta * cl;
            const int cps = (L.n_kc + ks - 1) / ks;
            if ((ks - 1) * cps >= L.n_kc && ks > 1) continue;               // would leave a slice empty
            const int span = std::min(ks_cta * cps, L.n_kc) * L.chunk_k;
            const int x_stride = span + (((span * 2) % 128) == 0 ? 32 : 0);
            // x fragments straight from global memory need K to be a whole number of chunks (no bounds checks
            // in the kernel); otherwise x is staged in shared memory with zeros beyond K
            const bool direct = xdirect && (L.K % L.chunk_k) == 0;
            const int x_bytes = direct ? 0 : ((M * x_stride * 2 + 127) / 128) * 128;
            const int smem = x_bytes + kGemvWarps * (kGemvRing * 512 + (L.grouped ? 1024 : 0));
            if (smem > kGemvMaxSmem) continue;
            const double warps = (double)n_rb * ks;
            const double eff = (double)L.n_kc / ((double)ks * cps);
            // slices of fewer than 4 chunks never reach a steady state (measured: 2-chunk slices lose to 4-chunk
            // slices on half as many warps)
            double score = -std::fabs(std::log2(warps / target)) + 2.0 * std::log2(eff) - (cps < 4 ? 1.25 : 0.0) - (cps < 2 ? 1.0 : 0.0);
            if (warps > target) score -= 2.0;                               // more CTAs than fit at once: a second wave
            if (force_ks) score = (ks == force_ks) ? 0.0 : -1e29;
            if (score > best_score) {
                best_score = score;
                const int rb_per_cta = kGemvWarps / ks_cta;
                best = GemvPlan{ks_cta, cl, cps, x_stride, x_bytes, smem, ((n_rb + rb_per_cta - 1) / rb_per_cta) * cl};
            }
        }
    return best;
}

template <typename Kern, typename Params>
cudaError_t launch(Kern kern, const Params& prm, dim3 grid, dim3 block, size_t smem, cudaStream_t st, int cluster, bool pdl)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attrs[2];
    int na = 0;
    if (cluster > 1) {
        attrs[na].id = cudaLaunchAttributeClusterDimension;
        attrs[na].val.clusterDim.x = cluster;
        attrs[na].val.clusterDim.y = 1;
        attrs[na].val.clusterDim.z = 1;
        ++na;
    }
    if (pdl) {
        attrs[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attrs[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attrs;
    cfg.numAttrs = na;
    return cudaLaunchKernelEx(&cfg, kern, prm);
}

template <int BITS, bool GROUPED, bool XDIRECT>
cudaError_t launch_gemv_x(const qlinear_s* h, const GemvParams& prm, const GemvPlan& pl, cudaStream_t st)
{
    static bool attr_set[64] = {};
    auto kern = gemv_kernel<BITS, GROUPED, XDIRECT>;
    if (h->device >= 0 && h->device < 64 && !attr_set[h->device]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemvMaxSmem);
        if (e != cudaSuccess) return e;
        attr_set[h->device] = true;
    }
    return launch(kern, prm, dim3(pl.grid), dim3(kGemvThreads), pl.smem_bytes, st, pl.cl, h->pdl);
}

template <int BITS, bool GROUPED>
cudaError_t launch_gemv(const qlinear_s* h, const GemvParams& prm, const GemvPlan& pl, cudaStream_t st)
{
    return prm.x_bytes == 0 ? launch_gemv_x<BITS, GROUPED, true>(h, prm, pl, st)
                            : launch_gemv_x<BITS, GROUPED, false>(h, prm, pl, st);
}

// One launch for n layers that read the same x (n == 1: the plain forward).
ql_status forward_gemv(qlinear_s* const* hs, int n, const void* x, void* const* ys, int M, cudaStream_t st)
{
    qlinear_s* h = hs[0];
    const Layout& L = h->L;
    GemvParams prm{};
    int n_rb = 0;
    for (int i = 0; i < n; ++i) {
        const Layout& Li = hs[i]->L;
        prm.body[i] = hs[i]->blob + Li.body_offset;
        prm.chan_scales[i] = Li.grouped ? nullptr : reinterpret_cast<const __half*>(hs[i]->blob + Li.chan_scale_offset);
        prm.y[i] = static_cast<__half*>(ys[i]);
        prm.N[i] = Li.N;
        n_rb += (Li.N + kRbRows - 1) / kRbRows;
        prm.rb_end[i] = n_rb;
    }
    prm.n_layers = n;
    GemvPlan pl;
    if (n == 1) pl = h->gemv[M];
    else {
        if (h->group_rb != n_rb) {                                       // plans of the last group this layer led
            for (int m = 1; m <= 8; ++m) h->group_gemv[m] = plan_gemv(L, n_rb, m, h->num_sms);
            h->group_rb = n_rb;
        }
        pl = h->group_gemv[M];
    }
    prm.x = static_cast<const __half*>(x);
    prm.M = M; prm.K = L.K;
    prm.n_rb = n_rb;
    prm.n_kc = L.n_kc;
    prm.block_bytes = L.block_bytes;
    prm.ks_cta = pl.ks_cta; prm.ks_cta_log2 = pl.ks_cta == 8 ? 3 : pl.ks_cta == 4 ? 2 : pl.ks_cta == 2 ? 1 : 0; prm.cl = pl.cl; prm.cps = pl.cps; prm.x_stride = pl.x_stride; prm.x_bytes = pl.x_bytes;
    cudaError_t e;
    if (L.bits == 8) e = launch_gemv<8, false>(h, prm, pl, st);
    else if (L.grouped) e = launch_gemv<4, true>(h, prm, pl, st);
    else e = launch_gemv<4, false>(h, prm, pl, st);
    return e == cudaSuccess ? QL_OK : QL_ERR_CUDA;
}

template <int BITS, bool GROUPED, int NS>
cudaError_t launch_stream_ns(const qlinear_s* h, const StreamParams& prm, cudaStream_t st)
{
    static bool attr_set[64] = {};
    auto kern = gemv_stream_kernel<BITS, GROUPED, NS>;
    if (h->device >= 0 && h->device < 64 && !attr_set[h->device]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, NS * StreamStage<BITS>::kBytes);
        if (e != cudaSuccess) return e;
        attr_set[h->device] = true;
    }
    return launch(kern, prm, dim3(prm.P), dim3(kStreamThreads), (size_t)NS * StreamStage<BITS>::kBytes, st, 1, h->pdl);
}

template <int BITS, bool GROUPED>
cudaError_t launch_stream(const qlinear_s* h, const StreamParams& prm, cudaStream_t st)
{
    switch (prm.stages) {
        case 6: return launch_stream_ns<BITS, GROUPED, 6>(h, prm, st);
        case 8: return launch_stream_ns<BITS, GROUPED, 8>(h, prm, st);
        case 12: return launch_stream_ns<BITS, GROUPED, 12>(h, prm, st);
        case 16: return launch_stream_ns<BITS, GROUPED, 16>(h, prm, st);
    }
    return cudaErrorInvalidValue;
}

ql_status forward_gemv_stream(qlinear_s* h, const void* x, void* y, int M, cudaStream_t st)
{
    const Layout& L = h->L;
    StreamParams prm{};
    prm.body = h->blob + L.body_offset;
    prm.chan_scales = L.grouped ? nullptr : reinterpret_cast<const __half*>(h->blob + L.chan_scale_offset);
    prm.x = static_cast<const __half*>(x);
    prm.y = static_cast<__half*>(y);
    prm.scratch = h->stream_scratch;
    prm.counters = h->stream_counters;
    prm.M = M; prm.N = L.N; prm.K = L.K;
    prm.n_rsb = L.n_rsb; prm.n_kc = L.n_kc; prm.block_bytes = L.block_bytes;
    prm.P = h->stream_P;
    prm.stages = h->stream_stages;
#ifdef QL_TRACE
    static int trace_seq = 0;
    prm.trace_seq = trace_seq++;
#endif
    cudaError_t e;
    if (L.bits == 8) e = launch_stream<8, false>(h, prm, st);
    else if (L.grouped) e = launch_stream<4, true>(h, prm, st);
    else e = launch_stream<4, false>(h, prm, st);
    return e == cudaSuccess ? QL_OK : QL_ERR_CUDA;
}

// ---- debug: the integers as the device unpack routines see them
template <int BITS>
__global__ void __launch_bounds__(256) debug_unpack_kernel(const uint8_t* body, int8_t* q_out, int N, int K,
                                                           int n_kc, int block_bytes)
{
    const int rsb = blockIdx.y, kc = blockIdx.x;
    const int rb = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, c = lane & 3;
    const uint8_t* blk = body + ((int64_t)rsb * n_kc + kc) * block_bytes;
    const uint4 w = *reinterpret_cast<const uint4*>(blk + rb * 512 + lane * 16);
    const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
    const int row0 = rsb * kRsbRows + rb * kRbRows + g;
    constexpr int NMMA = BITS == 4 ? 4 : 2;
#pragma unroll
    for (int i = 0; i < NMMA; ++i) {
        uint32_t a[4];
        if (BITS == 4) unpack_int4_word(ww[i], a);
        else unpack_int8_words(ww[2 * i], ww[2 * i + 1], a);
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const __half2 hv = *reinterpret_cast<const __half2*>(&a[r]);
            const int row = row0 + 8 * (r & 1);
            const int j = 2 * (r >> 1);
            const int kbase = BITS == 4 ? kc * 64 + int4_k_in_chunk(c, i, j) : kc * 32 + 8 * c + 4 * i + j;
            if (row < N && kbase < K) {
                q_out[(int64_t)row * K + kbase] = (int8_t)__half2int_rn(__low2half(hv));
                q_out[(int64_t)row * K + kbase + 1] = (int8_t)__half2int_rn(__high2half(hv));
            }
        }
    }
}

// Test aid: the bounded wait of the kernels on a barrier that nothing completes.
__global__ void __launch_bounds__(32) expire_wait_kernel()
{
    __shared__ __align__(8) unsigned long long bar;
    __shared__ volatile uint32_t abort_word;
    if (threadIdx.x == 0) {
        abort_word = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) mbar_wait<true>(smem_u32(&bar), 0, &abort_word, 0x9A0);   // gives up, records the code
}

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
        if (prev == dev) prev = -1;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

}  // namespace

extern "C" ql_status qlinear_create(const qlinear_desc* d, const void* packed_dev, int device, qlinear_t* out)
{
    if (!d || !packed_dev || !out) return QL_ERR_INVALID_ARG;
    *out = nullptr;
    Layout L;
    if (!make_layout(d->N, d->K, d->bits, d->group, &L)) return QL_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(packed_dev) % 256) return QL_ERR_INVALID_ARG;
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess) { cudaGetLastError(); return QL_ERR_CUDA; }
    if (device < 0 || device >= n_dev) return QL_ERR_INVALID_ARG;
    int major = 0, sms = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess)
        return QL_ERR_CUDA;
    if (major != 10) return QL_ERR_ARCH;
    qlinear_s* h = new (std::nothrow) qlinear_s();
    if (!h) return QL_ERR_ALLOC;
    h->L = L;
    h->blob = static_cast<const uint8_t*>(packed_dev);
    h->device = device;
    h->num_sms = sms;
    h->gemv_max_m = std::max(1, std::min(8, env_int("QLINEAR_GEMV_MAX_M", 8)));
    h->pdl = env_int("QLINEAR_PDL", 1) != 0;
    for (int M = 1; M <= 8; ++M) h->gemv[M] = plan_gemv(L, (L.N + kRbRows - 1) / kRbRows, M, sms);
    ql_status st = gemm_plan(L, sms, &h->gemm);
    if (st != QL_OK) { delete h; return st; }
    // streaming decode kernel: persistent grid, ring depth and per-handle scratch
    {
        const int stage_bytes = L.bits == 4 ? StreamStage<4>::kBytes : StreamStage<8>::kBytes;
        const int ctas_per_sm = std::max(1, std::min(4, env_int("QLINEAR_STREAM_CTAS_PER_SM", 3)));
        const int max_stages = std::min(env_int("QLINEAR_STREAM_STAGES", kStreamMaxStages), (220 * 1024 / ctas_per_sm - 1536) / stage_bytes);
        h->stream_stages = max_stages >= 16 ? 16 : max_stages >= 12 ? 12 : max_stages >= 8 ? 8 : 6;   // instantiated ring depths
        const int64_t B = (int64_t)L.n_rsb * L.n_kc;
        h->stream_P = (int)std::min<int64_t>(B, (int64_t)sms * ctas_per_sm);
        const char* kc = std::getenv("QLINEAR_GEMV_KERNEL");
        const int64_t body_bytes = B * L.block_bytes;
        h->gemv_kernel_choice = (kc && !std::strcmp(kc, "cluster")) ? 0 : (kc && !std::strcmp(kc, "stream")) ? 1
                                : (body_bytes >= (int64_t)env_int("QLINEAR_STREAM_MIN_MB", 1 << 20) * (1 << 20) ? 1 : 0);
        if (L.bits == 4 && (L.K % 64)) h->gemv_kernel_choice = 0;       // the streaming kernel reads whole 64-k slices of x
        DeviceGuard guard(device);
        const size_t sbytes = (size_t)h->stream_P * 2 * kStreamPartialFloats * sizeof(float);
        const size_t cbytes = (size_t)L.n_rsb * 8 * sizeof(unsigned int);
        if (!guard.ok || cudaMalloc(&h->stream_scratch, sbytes) != cudaSuccess) { cudaGetLastError(); delete h; return QL_ERR_CUDA; }
        if (cudaMalloc(&h->stream_counters, cbytes) != cudaSuccess || cudaMemset(h->stream_counters, 0, cbytes) != cudaSuccess) {
            cudaGetLastError(); cudaFree(h->stream_scratch); cudaFree(h->stream_counters); delete h; return QL_ERR_CUDA;
        }
        if (gemm_pair_may_split(L, sms)) {
            const size_t cb = gemm_pair_counter_count(sms) * sizeof(unsigned int);
            if (cudaMalloc(&h->gemm_scratch, gemm_pair_scratch_bytes(sms)) != cudaSuccess ||
                cudaMalloc(&h->gemm_counters, cb) != cudaSuccess || cudaMemset(h->gemm_counters, 0, cb) != cudaSuccess) {
                cudaGetLastError();
                cudaFree(h->stream_scratch); cudaFree(h->stream_counters); cudaFree(h->gemm_scratch); cudaFree(h->gemm_counters);
                delete h;
                return QL_ERR_CUDA;
            }
        }
    }
    *out = h;
    return QL_OK;
}

extern "C" int32_t qlinear_path_for(qlinear_t h, int32_t M)
{
    if (!h || M < 1) return 0;
    return M <= h->gemv_max_m ? QL_PATH_GEMV : QL_PATH_GEMM;
}

extern "C" ql_status qlinear_forward(qlinear_t h, const void* x, void* y, int32_t M, void* stream)
{
    if (!h || !x || !y || M < 1) return QL_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y)) & 15) return QL_ERR_INVALID_ARG;
    if ((int64_t)M * h->L.K > INT32_MAX || (int64_t)M * h->L.N > INT32_MAX) return QL_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) { cudaGetLastError(); return QL_ERR_CUDA; }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (M <= h->gemv_max_m) return h->gemv_kernel_choice ? forward_gemv_stream(h, x, y, M, st) : forward_gemv(&h, 1, x, &y, M, st);
    if (gemm_pair_applicable(h->L, M)) {
        GemmPairLayers set{};
        set.n = 1; set.L[0] = &h->L; set.blob[0] = h->blob; set.y[0] = y;
        return gemm_pair_forward(set, x, M, st, h->device, h->pdl, h->num_sms, h->gemm_scratch, h->gemm_counters);
    }
    return gemm_forward(h->L, h->gemm, h->blob, x, y, M, st, h->device, h->pdl, h->num_sms);
}

extern "C" ql_status qlinear_forward_group(const qlinear_t* hs, int32_t n, const void* x, void* const* ys, int32_t M, void* stream)
{
    if (!hs || !ys || !x || n < 1 || n > kGemvMaxGroup || M < 1) return QL_ERR_INVALID_ARG;
    for (int i = 0; i < n; ++i) {
        if (!hs[i] || !ys[i] || (reinterpret_cast<uintptr_t>(ys[i]) & 15)) return QL_ERR_INVALID_ARG;
        const Layout &a = hs[0]->L, &b = hs[i]->L;
        if (hs[i]->device != hs[0]->device || a.K != b.K || a.bits != b.bits || a.group != b.group) return QL_ERR_INVALID_ARG;
        if ((int64_t)M * b.N > INT32_MAX) return QL_ERR_INVALID_ARG;
    }
    if ((reinterpret_cast<uintptr_t>(x) & 15) || (int64_t)M * hs[0]->L.K > INT32_MAX) return QL_ERR_INVALID_ARG;
    // One kernel where the decode kernel serves the call; otherwise the layers run one after the other.
    if (n > 1 && M <= hs[0]->gemv_max_m && hs[0]->gemv_kernel_choice == 0) {
        DeviceGuard guard(hs[0]->device);
        if (!guard.ok) { cudaGetLastError(); return QL_ERR_CUDA; }
        return forward_gemv(const_cast<qlinear_s* const*>(hs), n, x, ys, M, static_cast<cudaStream_t>(stream));
    }
    if (n > 1 && M > hs[0]->gemv_max_m) {                                // prefill: one launch of the CTA-pair kernel
        bool pair_ok = true;
        for (int i = 0; i < n; ++i) pair_ok = pair_ok && gemm_pair_applicable(hs[i]->L, M);
        if (pair_ok) {
            DeviceGuard guard(hs[0]->device);
            if (!guard.ok) { cudaGetLastError(); return QL_ERR_CUDA; }
            GemmPairLayers set{};
            set.n = n;
            for (int i = 0; i < n; ++i) { set.L[i] = &hs[i]->L; set.blob[i] = hs[i]->blob; set.y[i] = ys[i]; }
            return gemm_pair_forward(set, x, M, static_cast<cudaStream_t>(stream), hs[0]->device, hs[0]->pdl, hs[0]->num_sms,
                                     hs[0]->gemm_scratch, hs[0]->gemm_counters);
        }
    }
    for (int i = 0; i < n; ++i) {
        ql_status s = qlinear_forward(hs[i], x, ys[i], M, stream);
        if (s != QL_OK) return s;
    }
    return QL_OK;
}

extern "C" ql_status qlinear_embed(qlinear_t h, const int32_t* ids, int32_t n, void* y, void* stream)
{
    if (!h || n < 0) return QL_ERR_INVALID_ARG;
    if (n == 0) return QL_OK;                                            // nothing to do: the pointers may be null
    if (!ids || !y) return QL_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(y) & 15) || (reinterpret_cast<uintptr_t>(ids) & 3)) return QL_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) { cudaGetLastError(); return QL_ERR_CUDA; }
    const Layout& L = h->L;
    EmbedParams prm{};
    prm.body = h->blob + L.body_offset;
    prm.chan_scales = L.grouped ? nullptr : reinterpret_cast<const __half*>(h->blob + L.chan_scale_offset);
    prm.ids = ids;
    prm.y = static_cast<__half*>(y);
    prm.n = n; prm.N = L.N; prm.K = L.K; prm.n_kc = L.n_kc; prm.block_bytes = L.block_bytes;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (L.bits == 8) embed_kernel<8, false><<<n, 128, 0, st>>>(prm);
    else if (L.grouped) embed_kernel<4, true><<<n, 128, 0, st>>>(prm);
    else embed_kernel<4, false><<<n, 128, 0, st>>>(prm);
    return cudaGetLastError() == cudaSuccess ? QL_OK : QL_ERR_CUDA;
}

extern "C" ql_status qlinear_debug_unpack_device(qlinear_t h, int8_t* q_out, void* stream)
{
    if (!h || !q_out) return QL_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) { cudaGetLastError(); return QL_ERR_CUDA; }
    const Layout& L = h->L;
    dim3 grid(L.n_kc, L.n_rsb);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (L.bits == 4)
        debug_unpack_kernel<4><<<grid, 256, 0, st>>>(h->blob + L.body_offset, q_out, L.N, L.K, L.n_kc, L.block_bytes);
    else
        debug_unpack_kernel<8><<<grid, 256, 0, st>>>(h->blob + L.body_offset, q_out, L.N, L.K, L.n_kc, L.block_bytes);
    return cudaGetLastError() == cudaSuccess ? QL_OK : QL_ERR_CUDA;
}


// ---------------------------------------------------------------------------------------------------
// qlinear_decode_static: the streaming decode kernel for callers that cannot allocate device memory
// (see include/qlinear.h).  Its partial-sum slots and counters live in one file-scope device array.
namespace {

constexpr int kStaticMaxCtas = 320;                 // CTAs of the persistent grid (2 per SM on a 148-SM part)
constexpr int kStaticMaxRsb = 4096;                 // row super-blocks, i.e. N <= 524288
constexpr size_t kStaticPartialBytes = (size_t)kStaticMaxCtas * 2 * kStreamPartialFloats * sizeof(float);   // 2.5 MiB
constexpr size_t kStaticCounterBytes = (size_t)kStaticMaxRsb * 8 * sizeof(unsigned int);                    // 128 KiB
constexpr int kStaticStages = 8;

// Every GPU that loads the library holds this array until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticPartialBytes + kStaticCounterBytes];

struct StaticDevice {
    bool ready = false;
    unsigned char* base = nullptr;                  // device address of g_static_scratch on this device
    int sms = 0;
};
StaticDevice g_static_dev[64];
std::mutex g_static_mutex;

// Once per device, with that device current: the array's name is only a host-side stand-in, the address a
// kernel may use comes from cudaGetSymbolAddress.
ql_status static_setup(int device, StaticDevice** out)
{
    if (device < 0 || device >= 64) return QL_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticDevice& d = g_static_dev[device];
    if (!d.ready) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess ||
            cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
            cudaGetLastError();
            return QL_ERR_CUDA;
        }
        if (major != 10) return QL_ERR_ARCH;
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return QL_ERR_CUDA;
        }
        d.base = static_cast<unsigned char*>(ptr);
        d.ready = true;
    }
    *out = &d;
    return QL_OK;
}

template <int BITS, bool GROUPED>
cudaError_t launch_stream_static(const StreamParams& prm, cudaStream_t st, int device)
{
    static bool attr_set[64] = {};
    auto kern = gemv_stream_kernel<BITS, GROUPED, kStaticStages>;
    const size_t smem = (size_t)kStaticStages * StreamStage<BITS>::kBytes;
    if (!attr_set[device]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        attr_set[device] = true;
    }
    return launch(kern, prm, dim3(prm.P), dim3(kStreamThreads), smem, st, 1, false);
}

}  // namespace

extern "C" ql_status qlinear_decode_static(const qlinear_desc* d, const void* packed_dev, const void* x, void* y, int32_t M,
                                           int device, void* stream)
{
    if (!d || !packed_dev || !x || !y) return QL_ERR_INVALID_ARG;
    if (M < 1 || M > 8) return QL_ERR_INVALID_ARG;                       // decode kernel only
    if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y)) & 15) return QL_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(packed_dev) % 256) return QL_ERR_INVALID_ARG;
    Layout L;
    if (!make_layout(d->N, d->K, d->bits, d->group, &L)) return QL_ERR_UNSUPPORTED;
    if (L.n_rsb > kStaticMaxRsb) return QL_ERR_UNSUPPORTED;              // beyond the static counters
    if (L.bits == 4 && (L.K % 64)) return QL_ERR_UNSUPPORTED;            // the streaming kernel reads whole 64-k slices
    DeviceGuard guard(device);
    if (!guard.ok) { cudaGetLastError(); return QL_ERR_CUDA; }
    StaticDevice* dev = nullptr;
    ql_status sst = static_setup(device, &dev);
    if (sst != QL_OK) return sst;

    const uint8_t* blob = static_cast<const uint8_t*>(packed_dev);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    StreamParams prm{};
    prm.body = blob + L.body_offset;
    prm.chan_scales = L.grouped ? nullptr : reinterpret_cast<const __half*>(blob + L.chan_scale_offset);
    prm.x = static_cast<const __half*>(x);
    prm.y = static_cast<__half*>(y);
    prm.scratch = reinterpret_cast<float*>(dev->base);
    prm.counters = reinterpret_cast<unsigned int*>(dev->base + kStaticPartialBytes);
    prm.M = M; prm.N = L.N; prm.K = L.K;
    prm.n_rsb = L.n_rsb; prm.n_kc = L.n_kc; prm.block_bytes = L.block_bytes;
    const int64_t B = (int64_t)L.n_rsb * L.n_kc;
    prm.P = (int)std::min<int64_t>(B, std::min(kStaticMaxCtas, 2 * dev->sms));
    prm.stages = kStaticStages;
    // The array keeps whatever the last call left: the counters must start at zero (they do after a call
    // that ran to completion; this also covers one that did not).
    if (cudaMemsetAsync(prm.counters, 0, (size_t)L.n_rsb * 8 * sizeof(unsigned int), st) != cudaSuccess) {
        cudaGetLastError();
        return QL_ERR_CUDA;
    }
    cudaError_t e;
    if (L.bits == 8) e = launch_stream_static<8, false>(prm, st, device);
    else if (L.grouped) e = launch_stream_static<4, true>(prm, st, device);
    else e = launch_stream_static<4, false>(prm, st, device);
    if (e != cudaSuccess) { cudaGetLastError(); return QL_ERR_CUDA; }
    return QL_OK;
}

extern "C" ql_status qlinear_debug_expire_wait(qlinear_t h, void* stream)
{
    if (!h) return QL_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) { cudaGetLastError(); return QL_ERR_CUDA; }
    expire_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>();
    return cudaGetLastError() == cudaSuccess ? QL_OK : QL_ERR_CUDA;
}

extern "C" ql_status qlinear_device_status(qlinear_t h, uint32_t* detail)
{
    if (!h) return QL_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) { cudaGetLastError(); return QL_ERR_CUDA; }
    unsigned int flag[2] = {0, 0};
    if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return QL_ERR_CUDA; }
    if (cudaMemcpyFromSymbol(flag, g_device_flag, sizeof(flag)) != cudaSuccess) { cudaGetLastError(); return QL_ERR_CUDA; }
    if (detail) *detail = flag[0];
    if (flag[0] == 0) return QL_OK;
    const unsigned int zero[2] = {0, 0};
    cudaMemcpyToSymbol(g_device_flag, zero, sizeof(zero));
    return QL_ERR_DEVICE_TIMEOUT;
}

extern "C" ql_status qlinear_destroy(qlinear_t h)
{
    if (!h) return QL_OK;
    {
        DeviceGuard guard(h->device);
        cudaFree(h->stream_scratch);
        cudaFree(h->stream_counters);
        cudaFree(h->gemm_scratch);
        cudaFree(h->gemm_counters);
    }
    delete h;
    return QL_OK;
}

extern "C" const char* qlinear_status_string(ql_status s)
{
    switch (s) {
        case QL_OK: return "ok";
        case QL_ERR_INVALID_ARG: return "invalid argument";
        case QL_ERR_UNSUPPORTED: return "unsupported shape or quantisation scheme";
        case QL_ERR_ALLOC: return "host allocation failed";
        case QL_ERR_CUDA: return "CUDA call failed";
        case QL_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel expired";
        case QL_ERR_ARCH: return "device is not compute capability 10.x (sm_100)";
    }
    return "unknown status";
}

#ifdef QL_TRACE
extern "C" int qlinear_debug_read_gemm_trace(unsigned long long* out, size_t bytes)
{
    return (int)cudaMemcpyFromSymbol(out, g_gemm_trace, bytes < sizeof(g_gemm_trace) ? bytes : sizeof(g_gemm_trace));
}
extern "C" int qlinear_debug_read_trace(unsigned long long* out, size_t bytes)
{
    return (int)cudaMemcpyFromSymbol(out, g_trace, bytes < sizeof(g_trace) ? bytes : sizeof(g_trace));
}
#endif

extern "C" uint32_t qlinear_version(void) { return (1u << 16) | 0u; }
