// C-ABI of the qlinear library: handle life cycle, stage-aware dispatch (paper Section 3.7) and the
// launchers of the decode and prefill kernels.  Single translation unit for all device code.
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
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
// Device-side alias of one word of pinned host memory (null until the first handle on the device exists): the
// same code, readable by the host without synchronising.
__device__ unsigned int* g_status_host;
}  // namespace ql

#include "dequant.cuh"
#include "embed.cuh"
#include "gemv.cuh"
#include "gemv_rows.cuh"
#include "gemv_stream.cuh"
#include "gemv_a8.cuh"
#include "kv.cuh"
#include "gemm.cuh"
#include "gemm_pair.cuh"
#include "gemm_pair_ta.cuh"
#include "norm.cuh"
#include "rope.cuh"

using namespace ql;

namespace {

int env_int(const char* name, int dflt)
{
    const char* v = std::getenv(name);
    return (v && *v) ? std::atoi(v) : dflt;
}

// Every QLINEAR_* switch, read from the environment ONCE per process (at the first call that needs one).
struct Config {
    int gemv_max_m;          // QLINEAR_GEMV_MAX_M: largest M served by the decode kernels (1..8)
    bool pdl;                // QLINEAR_PDL: programmatic dependent launch attribute on every kernel
    int warps_per_sm;        // QLINEAR_GEMV_WARPS_PER_SM: residency target of the cluster decode kernel
    bool oversubscribe;      // QLINEAR_GEMV_OVERSUBSCRIBE=0: the group-scaled int4 decode kernel never takes more CTAs than fit at once
    int force_ks;            // QLINEAR_GEMV_KS: forced K split of the cluster decode kernel (0 = planned)
    bool xdirect;            // QLINEAR_GEMV_XDIRECT: x fragments straight from global memory
    int kernel;              // QLINEAR_GEMV_KERNEL: 0 / 1 cluster kernel (default), 2 streaming kernel
    int stream_ctas_per_sm, stream_stages;
    GemmConfig gemm;
    unsigned generation;     // bumped by qlinear_debug_reload_config (tests)
};
Config g_cfg;
std::once_flag g_cfg_once;
std::atomic<unsigned> g_getenv_reads{0};

void load_config()
{
    Config c{};
    c.gemv_max_m = std::max(1, std::min(8, env_int("QLINEAR_GEMV_MAX_M", 8)));
    c.pdl = env_int("QLINEAR_PDL", 1) != 0;
    c.warps_per_sm = env_int("QLINEAR_GEMV_WARPS_PER_SM", 32);
    c.oversubscribe = env_int("QLINEAR_GEMV_OVERSUBSCRIBE", 1) != 0;
    c.force_ks = env_int("QLINEAR_GEMV_KS", 0);
    c.xdirect = env_int("QLINEAR_GEMV_XDIRECT", 1) != 0;
    const char* kc = std::getenv("QLINEAR_GEMV_KERNEL");
    c.kernel = !kc ? 0 : !std::strcmp(kc, "cluster") ? 1 : !std::strcmp(kc, "stream") ? 2 : 0;
    c.stream_ctas_per_sm = std::max(1, std::min(4, env_int("QLINEAR_STREAM_CTAS_PER_SM", 3)));
    c.stream_stages = env_int("QLINEAR_STREAM_STAGES", kStreamMaxStages);
    c.gemm.force_bn = env_int("QLINEAR_GEMM_BN", 0);
    c.gemm.force_split = env_int("QLINEAR_GEMM_SPLIT", 0);
    c.gemm.force_tb = env_int("QLINEAR_GEMM_TB", 0);
    c.gemm.pair = env_int("QLINEAR_GEMM_PAIR", 1) != 0;
    c.gemm.ta = env_int("QLINEAR_GEMM_TA", 1) != 0;
    c.generation = g_cfg.generation + 1;
    g_cfg = c;
    g_getenv_reads.fetch_add(1);
}
const Config& config()
{
    std::call_once(g_cfg_once, load_config);
    return g_cfg;
}

}  // namespace

namespace ql {
GemmConfig& gemm_config() { return const_cast<Config&>(config()).gemm; }
}  // namespace ql

namespace {

struct GemvPlan {
    int32_t ks_cta, cl, cps, x_stride, x_bytes, smem_bytes, grid;
    double max_over_mean;    // chunks of the busiest SM over the mean, as the hardware would place the grid
};

// Device memory the library owns, ONE set per device, created with the first handle on that device and shared by
// every handle there (kernels that use it run in stream order: see include/qlinear.h).
struct DeviceState {
    bool ready = false;
    int sms = 0;
    int handles = 0;
    unsigned int* status_host = nullptr;     // pinned, mapped: the code of the last expired wait (0 = none)
    float* gemm_scratch = nullptr;           // CTA-pair prefill kernel, K-split of single-round layers
    unsigned int* gemm_counters = nullptr;
    float* stream_scratch = nullptr;         // streaming decode kernel (only when QLINEAR_GEMV_KERNEL=stream)
    unsigned int* stream_counters = nullptr;
};
constexpr int kMaxDevices = 64;
constexpr int kStreamMaxRsb = 4096;          // row super-blocks the shared streaming-kernel counters cover
DeviceState g_dev[kMaxDevices];
std::mutex g_dev_mutex;

}  // namespace

struct qlinear_s {
    // Immutable after qlinear_create.
    Layout L;
    const uint8_t* blob;
    int device;
    int num_sms;
    int gemv_max_m;
    bool pdl;
    int n_rb;                  // row-blocks holding at least one real row
    GemvPlan gemv[9];          // cluster decode kernel, index = M (1..8)
    bool use_stream;
    int stream_P, stream_stages;
    CUtensorMap wmap;          // the packed body as rows of 64 bytes (prefill kernel with the weights in tensor memory)
    CUtensorMap wmap_i8;       // the same with the integer form's box (128 k per step)
    bool wmap_ok, wmap_i8_ok;
    DeviceState* dev;
};

namespace {

constexpr int kGemvMaxSmem = 96 * 1024;

// n_rb: row-blocks of the launch (one layer, or all layers of a group that shares x).
// gated: the launch needs both branches of a channel in one CTA: an even number of row-blocks per CTA, no cluster.
// a8: the int8-activation kernel keeps the quantised x of the CTA's K range, and its per-group sums, in shared memory.
GemvPlan plan_gemv(const Layout& L, int n_rb, int M, int num_sms, bool gated = false, bool a8 = false)
{
    const Config& cfg = config();
    const double target = (double)num_sms * cfg.warps_per_sm;
    GemvPlan best{};
    double best_score = -1e30;
    for (int ks_cta = 1; ks_cta <= 8; ks_cta *= 2)
        for (int cl = 1; cl <= (ks_cta == 8 ? 8 : 1); ++cl) {
            if (gated && (ks_cta > 4 || cl > 1)) continue;
            const int ks = ks_cta * cl;
            const int cps = (L.n_kc + ks - 1) / ks;
            if ((ks - 1) * cps >= L.n_kc && ks > 1) continue;               // would leave a slice empty
            const int span = std::min(ks_cta * cps, L.n_kc) * L.chunk_k;
            const int x_stride = span + (((span * 2) % 128) == 0 ? 32 : 0);
            // x fragments straight from global memory need K to be a whole number of chunks (no bounds checks
            // in the kernel); otherwise x is staged in shared memory with zeros beyond K
            const bool direct = cfg.xdirect && (L.K % L.chunk_k) == 0;
            const int a8_span = ks_cta * cps * L.chunk_k;
            const int x_bytes = a8 ? ((M * (a8_span + 32) + 15) / 16) * 16 + a8_span
                                   : direct ? 0 : ((M * x_stride * 2 + 127) / 128) * 128;
            const int smem = x_bytes + kGemvWarps * (kGemvRing * 512 + (L.grouped ? 1024 : 0));
            if (smem > kGemvMaxSmem) continue;
            const double warps = (double)n_rb * ks;
            const double eff = (double)L.n_kc / ((double)ks * cps);
            // slices of fewer than 4 chunks never reach a steady state (measured: 2-chunk slices lose to 4-chunk
            // slices on half as many warps)
            double score = -std::fabs(std::log2(warps / target)) + 2.0 * std::log2(eff) - (cps < 4 ? 1.25 : 0.0) - (cps < 2 ? 1.0 : 0.0);
            // More CTAs than fit at once mean a second wave -- except, for the group-scaled int4 kernel (bound by its
            // instruction stream, not by the memory system) at one token, up to about one and a half waves of CTAs without
            // clusters whose slices stay long: the partial second wave fills in as the first one drains, and the finer
            // units even out the end (Llama gate + up: 17.8 us with 0.76 of a wave, 17.2 us with 1.5 waves).  Measured limits
            // of the rule: the int8 and per-channel forms of the same launch lose 2 to 7 % that way, and with 2 to 8 tokens
            // the launch itself still gains but the step that contains it loses 1 to 3 % (the next launch gets its SMs later).
            if (warps > target) score += (cfg.oversubscribe && M == 1 && L.grouped && cl == 1 && warps <= 1.55 * target && cps >= 16) ? 0.25 : -2.0;
            // a cluster launch and its two cluster-wide barriers cost a microsecond or two (the CTAs of a cluster start
            // together and leave together): more than a launch of a few MB gains from the extra warps (V-cache product of 8
            // heads at 1280 positions: 4.2 us with clusters of 5, 3.1 us without; one 2304 x 2304 int8 layer: 4.0 / 3.7 us).
            // Larger launches keep their clusters: timed alone they look better without (Llama o, 16.8 MB: 5.9 / 4.6 us),
            // but inside the step the under-filled grid costs the launches around it more than it saves.
            if (cl > 1 && (double)n_rb * L.n_kc * 512.0 < 6.0e6) score -= 0.75;
            if (cfg.force_ks && !gated) score = (ks == cfg.force_ks) ? 0.0 : -1e29;
            if (score > best_score) {
                best_score = score;
                const int rb_per_cta = kGemvWarps / ks_cta;
                const int grid = ((n_rb + rb_per_cta - 1) / rb_per_cta) * cl;
                // CTAs spread over the SMs one by one: the busiest SM holds ceil(grid / SMs) of them
                const double per_sm = (double)grid / num_sms;
                best = GemvPlan{ks_cta, cl, cps, x_stride, x_bytes, smem, grid,
                                grid <= 4 * num_sms ? std::ceil(per_sm) / per_sm / eff : 2.0};
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

// cudaFuncSetAttribute once per (kernel instantiation, device); `flags` is that instantiation's table.
template <typename Kern>
cudaError_t ensure_smem_attr(Kern kern, std::atomic<bool>* flags, int device, int bytes)
{
    if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
    if (flags[device].load(std::memory_order_acquire)) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) flags[device].store(true, std::memory_order_release);
    return e;
}

template <int BITS, bool GROUPED, bool XDIRECT, bool GATED = false, bool XSCALE = false, int NG = kGemvMaxGroup>
cudaError_t launch_gemv_x(const qlinear_s* h, const GemvParamsT<NG>& prm, const GemvPlan& pl, cudaStream_t st)
{
    static std::atomic<bool> attr_set[kMaxDevices];
    auto kern = gemv_kernel<BITS, GROUPED, XDIRECT, GATED, XSCALE, NG>;
    cudaError_t e = ensure_smem_attr(kern, attr_set, h->device, kGemvMaxSmem);
    if (e != cudaSuccess) return e;
    return launch(kern, prm, dim3(pl.grid), dim3(kGemvThreads), pl.smem_bytes, st, pl.cl, h->pdl);
}

template <int BITS, bool GROUPED>
cudaError_t launch_gemv(const qlinear_s* h, const GemvParams& prm, const GemvPlan& pl, cudaStream_t st, bool gated = false, bool xscale = false)
{
    if constexpr (BITS == 8 && !GROUPED) {
        if (xscale) return launch_gemv_x<8, false, true, false, true>(h, prm, pl, st);   // (int8, direct x: checked by the caller)
    }
    if (gated) return launch_gemv_x<BITS, GROUPED, true, true>(h, prm, pl, st);     // (planned only with direct x)
    return prm.x_bytes == 0 ? launch_gemv_x<BITS, GROUPED, true>(h, prm, pl, st)
                            : launch_gemv_x<BITS, GROUPED, false>(h, prm, pl, st);
}
// The wide form (5 to 8 layers, each with its own input read straight from global memory): int8 layers, the KV heads of
// an attention layer.
cudaError_t launch_gemv_wide(const qlinear_s* h, const GemvParamsT<kGemvMaxBatch>& prm, const GemvPlan& pl, cudaStream_t st, bool xscale)
{
    return xscale ? launch_gemv_x<8, false, true, false, true, kGemvMaxBatch>(h, prm, pl, st)
                  : launch_gemv_x<8, false, true, false, false, kGemvMaxBatch>(h, prm, pl, st);
}

template <int NG>
void fill_gemv_params(GemvParamsT<NG>& prm, qlinear_s* const* hs, int n, const void* x, void* const* ys, int M, int n_rb, const GemvPlan& pl,
                      int act, const void* const* xs, const void* const* xscales)
{
    const Layout& L = hs[0]->L;
    const bool gated = act >= 0;
    int acc = 0;
    for (int i = 0; i < n; ++i) {
        const Layout& Li = hs[i]->L;
        prm.body[i] = hs[i]->blob + Li.body_offset;
        prm.chan_scales[i] = Li.grouped ? nullptr : reinterpret_cast<const __half*>(hs[i]->blob + Li.chan_scale_offset);
        prm.y[i] = static_cast<__half*>(ys[gated ? 0 : i]);
        prm.N[i] = Li.N;
        acc += hs[i]->n_rb;
        prm.rb_end[i] = acc;
    }
    prm.n_layers = n;
    prm.act = gated ? act : 0;
    prm.x = static_cast<const __half*>(xs ? xs[0] : x);
    for (int i = 0; i < NG; ++i) {
        prm.xl[i] = static_cast<const __half*>(xs ? xs[i < n ? i : 0] : x);
        prm.xscale[i] = static_cast<const __half*>(xscales ? xscales[i < n ? i : 0] : nullptr);
    }
    prm.M = M; prm.K = L.K;
    prm.n_rb = n_rb;
    prm.n_kc = L.n_kc;
    prm.block_bytes = L.block_bytes;
    prm.ks_cta = pl.ks_cta; prm.ks_cta_log2 = pl.ks_cta == 8 ? 3 : pl.ks_cta == 4 ? 2 : pl.ks_cta == 2 ? 1 : 0; prm.cl = pl.cl; prm.cps = pl.cps; prm.x_stride = pl.x_stride; prm.x_bytes = pl.x_bytes;
}

// The persistent form for int8 layers with many rows and a short K (gemv_rows.cuh): every layer with its own input.
template <int NKC>
cudaError_t launch_gemv_rows(const qlinear_s* h, const GemvRowsParams& prm, cudaStream_t st)
{
    static std::atomic<bool> attr_set[kMaxDevices];
    auto kern = gemv_rows_kernel<NKC>;
    const int smem = kGemvWarps * 2 * NKC * 512;
    cudaError_t e = ensure_smem_attr(kern, attr_set, h->device, smem);
    if (e != cudaSuccess) return e;
    const int grid = std::min(prm.n_rsb, h->num_sms * (NKC <= 4 ? 4 : 3));
    return launch(kern, prm, dim3(grid), dim3(kGemvThreads), smem, st, 1, h->pdl);
}

// One launch for n layers that read the same x (n == 1: the plain forward).  The plan of a group is made per
// call (integer arithmetic only); nothing is written to a handle.
// act >= 0: the gated form (n == 2: gate, up; ys[0] the output; the row-blocks of the two layers alternate).
// xs != nullptr: the batched form, layer i reads xs[i] (x is then ignored); needs the kernel form that reads x straight
// from global memory; int8 layers may come up to kGemvMaxBatch at a time.  xscales != nullptr (with xs, int8 layers):
// layer i's input is multiplied by xscales[i][0 .. K).
ql_status forward_gemv(qlinear_s* const* hs, int n, const void* x, void* const* ys, int M, cudaStream_t st, int act = -1,
                       const void* const* xs = nullptr, const void* const* xscales = nullptr)
{
    const qlinear_s* h = hs[0];
    const Layout& L = h->L;
    int n_rb = 0;
    for (int i = 0; i < n; ++i) n_rb += hs[i]->n_rb;
    const bool gated = act >= 0;
    if (gated) n_rb = 2 * hs[0]->n_rb;
    // many rows, short K (the score product over a long KV cache): more than one wave of row super-blocks
    if (xs && !xscales && !gated && n <= kGemvMaxBatch && L.bits == 8 && (L.K % 32) == 0 && (L.n_kc == 2 || L.n_kc == 4 || L.n_kc == 8)) {
        GemvRowsParams rp{};
        int n_rsb = 0;
        for (int i = 0; i < n; ++i) {
            const Layout& Li = hs[i]->L;
            rp.body[i] = hs[i]->blob + Li.body_offset;
            rp.chan_scales[i] = reinterpret_cast<const __half*>(hs[i]->blob + Li.chan_scale_offset);
            rp.y[i] = static_cast<__half*>(ys[i]);
            rp.xl[i] = static_cast<const __half*>(xs[i]);
            rp.N[i] = Li.N;
            n_rsb += Li.n_rsb;
            rp.rsb_end[i] = n_rsb;
        }
        if (n_rsb > 4 * h->num_sms) {
            rp.n_layers = n; rp.M = M; rp.K = L.K; rp.n_rsb = n_rsb; rp.block_bytes = L.block_bytes;
            const cudaError_t e = L.n_kc == 2 ? launch_gemv_rows<2>(h, rp, st) : L.n_kc == 4 ? launch_gemv_rows<4>(h, rp, st) : launch_gemv_rows<8>(h, rp, st);
            return e == cudaSuccess ? QL_OK : QL_ERR_CUDA;
        }
    }
    const GemvPlan pl = gated ? plan_gemv(L, n_rb, M, h->num_sms, true) : n == 1 ? h->gemv[M] : plan_gemv(L, n_rb, M, h->num_sms);
    if ((gated || xs) && (pl.grid <= 0 || pl.x_bytes != 0)) return QL_ERR_UNSUPPORTED;
    if (xscales && (!xs || L.bits != 8)) return QL_ERR_UNSUPPORTED;
    if (n > kGemvMaxGroup && (n > kGemvMaxBatch || !xs || L.bits != 8)) return QL_ERR_UNSUPPORTED;
    cudaError_t e;
    if (pl.grid <= 0) return QL_ERR_UNSUPPORTED;
    if (n > kGemvMaxGroup) {
        GemvParamsT<kGemvMaxBatch> wide{};
        fill_gemv_params(wide, hs, n, x, ys, M, n_rb, pl, act, xs, xscales);
        return launch_gemv_wide(h, wide, pl, st, xscales != nullptr) == cudaSuccess ? QL_OK : QL_ERR_CUDA;
    }
    GemvParams prm{};
    fill_gemv_params(prm, hs, n, x, ys, M, n_rb, pl, act, xs, xscales);
    if (L.bits == 8) e = launch_gemv<8, false>(h, prm, pl, st, gated, xscales != nullptr);
    else if (L.grouped) e = launch_gemv<4, true>(h, prm, pl, st, gated);
    else e = launch_gemv<4, false>(h, prm, pl, st, gated);
    return e == cudaSuccess ? QL_OK : QL_ERR_CUDA;
}

// y = act(g) * u, element-wise (the unfused form of the gating, for shapes the fused kernels do not take).
__global__ void __launch_bounds__(256) gate_mul_kernel(const __half* g, const __half* u, __half* y, int64_t n, int act)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n; i += (int64_t)gridDim.x * 256)
        y[i] = __float2half_rn(gate_activation(__half2float(g[i]), act) * __half2float(u[i]));
}

template <int BITS, bool GROUPED, int NS>
cudaError_t launch_stream_ns(const qlinear_s* h, const StreamParams& prm, cudaStream_t st)
{
    static std::atomic<bool> attr_set[kMaxDevices];
    auto kern = gemv_stream_kernel<BITS, GROUPED, NS>;
    cudaError_t e = ensure_smem_attr(kern, attr_set, h->device, NS * StreamStage<BITS>::kBytes);
    if (e != cudaSuccess) return e;
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

ql_status forward_gemv_stream(const qlinear_s* h, const void* x, void* y, int M, cudaStream_t st)
{
    const Layout& L = h->L;
    StreamParams prm{};
    prm.body = h->blob + L.body_offset;
    prm.chan_scales = L.grouped ? nullptr : reinterpret_cast<const __half*>(h->blob + L.chan_scale_offset);
    prm.x = static_cast<const __half*>(x);
    prm.y = static_cast<__half*>(y);
    prm.scratch = h->dev->stream_scratch;
    prm.counters = h->dev->stream_counters;
    prm.M = M; prm.N = L.N; prm.K = L.K;
    prm.n_rsb = L.n_rsb; prm.n_kc = L.n_kc; prm.block_bytes = L.block_bytes;
    prm.P = h->stream_P;
    prm.stages = h->stream_stages;
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
    __shared__ volatile uint32_t abort_word[3];                          // [0] abort, [2] "dependency resolved"
    if (threadIdx.x == 0) {
        abort_word[0] = 0;
        abort_word[1] = 0;
        abort_word[2] = 1;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) mbar_wait<true>(smem_u32(&bar), 0, abort_word, 0x9A0);   // gives up, records the code
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

namespace {

// Creates the device's shared state on first use (the device must be current).  Called under g_dev_mutex.
ql_status device_state_init(int device, int sms, DeviceState* d)
{
    if (d->ready) return QL_OK;
    const Config& cfg = config();
    d->sms = sms;
    const size_t cb = gemm_pair_counter_count(sms) * sizeof(unsigned int);
    bool ok = cudaHostAlloc(reinterpret_cast<void**>(&d->status_host), 64, cudaHostAllocMapped | cudaHostAllocPortable) == cudaSuccess;
    unsigned int* status_dev = nullptr;
    if (ok) {
        d->status_host[0] = 0;
        ok = cudaHostGetDevicePointer(reinterpret_cast<void**>(&status_dev), d->status_host, 0) == cudaSuccess &&
             cudaMemcpyToSymbol(g_status_host, &status_dev, sizeof(status_dev)) == cudaSuccess;
    }
    ok = ok && cudaMalloc(&d->gemm_scratch, gemm_pair_scratch_bytes(sms)) == cudaSuccess &&
         cudaMalloc(&d->gemm_counters, cb) == cudaSuccess && cudaMemset(d->gemm_counters, 0, cb) == cudaSuccess;
    if (ok && cfg.kernel == 2) {
        const size_t sbytes = (size_t)sms * 4 * 2 * kStreamPartialFloats * sizeof(float);
        const size_t cbytes = (size_t)kStreamMaxRsb * 8 * sizeof(unsigned int);
        ok = cudaMalloc(&d->stream_scratch, sbytes) == cudaSuccess && cudaMalloc(&d->stream_counters, cbytes) == cudaSuccess &&
             cudaMemset(d->stream_counters, 0, cbytes) == cudaSuccess;
    }
    if (!ok) {
        cudaGetLastError();
        unsigned int* null_ptr = nullptr;
        cudaMemcpyToSymbol(g_status_host, &null_ptr, sizeof(null_ptr));
        cudaFreeHost(d->status_host); cudaFree(d->gemm_scratch); cudaFree(d->gemm_counters);
        cudaFree(d->stream_scratch); cudaFree(d->stream_counters);
        cudaGetLastError();
        *d = DeviceState{};
        return QL_ERR_CUDA;
    }
    d->ready = true;
    return QL_OK;
}

// An earlier kernel on this device gave up a bounded wait: the host sees the code without synchronising.
inline bool device_timed_out(const qlinear_s* h)
{
    return *reinterpret_cast<volatile unsigned int*>(h->dev->status_host) != 0;
}

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
    if (device < 0 || device >= n_dev || device >= kMaxDevices) return QL_ERR_INVALID_ARG;
    int major = 0, sms = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess)
        return QL_ERR_CUDA;
    if (major != 10) return QL_ERR_ARCH;
    const Config& cfg = config();
    qlinear_s* h = new (std::nothrow) qlinear_s();
    if (!h) return QL_ERR_ALLOC;
    h->L = L;
    h->blob = static_cast<const uint8_t*>(packed_dev);
    h->device = device;
    h->num_sms = sms;
    h->gemv_max_m = cfg.gemv_max_m;
    h->pdl = cfg.pdl;
    h->n_rb = (L.N + kRbRows - 1) / kRbRows;
    h->wmap_ok = w_tensor_map(L, h->blob, &h->wmap);
    h->wmap_i8_ok = !L.grouped && (L.K % 128) == 0 && w_tensor_map(L, h->blob, &h->wmap_i8, true);
    for (int M = 1; M <= 8; ++M) {
        h->gemv[M] = plan_gemv(L, h->n_rb, M, sms);
        if (h->gemv[M].grid <= 0 && M <= h->gemv_max_m) { delete h; return QL_ERR_UNSUPPORTED; }   // no decode plan fits this shape
    }
    {
        // streaming decode kernel (QLINEAR_GEMV_KERNEL=stream): persistent grid and ring depth
        const int stage_bytes = L.bits == 4 ? StreamStage<4>::kBytes : StreamStage<8>::kBytes;
        const int max_stages = std::min(cfg.stream_stages, (220 * 1024 / cfg.stream_ctas_per_sm - 1536) / stage_bytes);
        h->stream_stages = max_stages >= 16 ? 16 : max_stages >= 12 ? 12 : max_stages >= 8 ? 8 : 6;   // instantiated ring depths
        const int64_t B = (int64_t)L.n_rsb * L.n_kc;
        h->stream_P = (int)std::min<int64_t>(B, (int64_t)sms * cfg.stream_ctas_per_sm);
        // the streaming kernel reads whole 64-k slices of x and shares counters sized for kStreamMaxRsb row super-blocks
        h->use_stream = cfg.kernel == 2 && !(L.bits == 4 && (L.K % 64)) && L.n_rsb <= kStreamMaxRsb;
    }
    {
        DeviceGuard guard(device);
        std::lock_guard<std::mutex> lock(g_dev_mutex);
        ql_status st = guard.ok ? device_state_init(device, sms, &g_dev[device]) : QL_ERR_CUDA;
        if (st != QL_OK) { cudaGetLastError(); delete h; return st; }
        h->dev = &g_dev[device];
        ++h->dev->handles;
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
    if (device_timed_out(h)) return QL_ERR_DEVICE_TIMEOUT;
    DeviceGuard guard(h->device);
    if (!guard.ok) { cudaGetLastError(); return QL_ERR_CUDA; }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (M <= h->gemv_max_m) return h->use_stream ? forward_gemv_stream(h, x, y, M, st) : forward_gemv(&h, 1, x, &y, M, st);
    {
        GemmPairLayers set{};
        set.n = 1; set.L[0] = &h->L; set.blob[0] = h->blob; set.y[0] = y; set.wmap[0] = h->wmap_ok ? &h->wmap : nullptr;
        const ql_status s = gemm_pair_forward_auto(set, x, M, st, h->device, h->pdl, h->num_sms, h->dev->gemm_scratch, h->dev->gemm_counters);
        if (s != QL_ERR_UNSUPPORTED) return s;                           // (an odd number of row super-blocks: the single-CTA kernel)
    }
    return gemm_forward(h->L, h->blob, x, y, M, st, h->device, h->pdl, h->num_sms);
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
    if (device_timed_out(hs[0])) return QL_ERR_DEVICE_TIMEOUT;
    // One kernel where the decode kernel serves the call; otherwise the layers run one after the other.
    if (n > 1 && M <= hs[0]->gemv_max_m && !hs[0]->use_stream) {
        DeviceGuard guard(hs[0]->device);
        if (!guard.ok) { cudaGetLastError(); return QL_ERR_CUDA; }
        return forward_gemv(const_cast<qlinear_s* const*>(hs), n, x, ys, M, static_cast<cudaStream_t>(stream));
    }
    if (n > 1 && M > hs[0]->gemv_max_m) {                                // prefill: one launch of the CTA-pair kernel
        bool pair_ok = true;
        for (int i = 0; i < n; ++i) pair_ok = pair_ok && (hs[i]->L.n_rsb % 2) == 0 && (gemm_pair_applicable(hs[i]->L, M) || (hs[i]->wmap_ok && gemm_config().ta));
        if (pair_ok) {
            DeviceGuard guard(hs[0]->device);
            if (!guard.ok) { cudaGetLastError(); return QL_ERR_CUDA; }
            GemmPairLayers set{};
            set.n = n;
            for (int i = 0; i < n; ++i) {
                set.L[i] = &hs[i]->L; set.blob[i] = hs[i]->blob; set.y[i] = ys[i];
                set.wmap[i] = hs[i]->wmap_ok ? &hs[i]->wmap : nullptr;
            }
            const ql_status s = gemm_pair_forward_auto(set, x, M, static_cast<cudaStream_t>(stream), hs[0]->device, hs[0]->pdl, hs[0]->num_sms,
                                                       hs[0]->dev->gemm_scratch, hs[0]->dev->gemm_counters);
            if (s != QL_ERR_UNSUPPORTED) return s;
        }
    }
    for (int i = 0; i < n; ++i) {
        ql_status s = qlinear_forward(hs[i], x, ys[i], M, stream);
        if (s != QL_OK) return s;
    }
    return QL_OK;
}

extern "C" ql_status qlinear_forward_batch(const qlinear_t* hs, int32_t n, const void* const* xs, void* const* ys, int32_t M, void* stream)
{
    if (!hs || !xs || !ys || n < 1 || n > kGemvMaxBatch || M < 1) return QL_ERR_INVALID_ARG;
    for (int i = 0; i < n; ++i) {
        if (!hs[i] || !xs[i] || !ys[i] || ((reinterpret_cast<uintptr_t>(xs[i]) | reinterpret_cast<uintptr_t>(ys[i])) & 15)) return QL_ERR_INVALID_ARG;
        const Layout &a = hs[0]->L, &b = hs[i]->L;
        if (hs[i]->device != hs[0]->device || a.K != b.K || a.bits != b.bits || a.group != b.group) return QL_ERR_INVALID_ARG;
        if ((int64_t)M * b.N > INT32_MAX || (int64_t)M * b.K > INT32_MAX) return QL_ERR_INVALID_ARG;
    }
    if (device_timed_out(hs[0])) return QL_ERR_DEVICE_TIMEOUT;
    if (n > 1 && M <= hs[0]->gemv_max_m && !hs[0]->use_stream) {         // one decode launch for all of them
        DeviceGuard guard(hs[0]->device);
        if (!guard.ok) { cudaGetLastError(); return QL_ERR_CUDA; }
        const ql_status s = forward_gemv(const_cast<qlinear_s* const*>(hs), n, nullptr, ys, M, static_cast<cudaStream_t>(stream), -1, xs);
        if (s != QL_ERR_UNSUPPORTED) return s;
    }
    for (int i = 0; i < n; ++i) {                                        // anything else: one call per layer
        const ql_status s = qlinear_forward(hs[i], xs[i], ys[i], M, stream);
        if (s != QL_OK) return s;
    }
    return QL_OK;
}

extern "C" ql_status qlinear_forward_gated(qlinear_t hg, qlinear_t hu, const void* x, void* y, int32_t M, int32_t act, void* stream)
{
    if (!hg || !hu || !x || !y || M < 1) return QL_ERR_INVALID_ARG;
    if (act != QL_ACT_IDENTITY && act != QL_ACT_SILU && act != QL_ACT_GELU_TANH) return QL_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y)) & 15) return QL_ERR_INVALID_ARG;
    const Layout &a = hg->L, &b = hu->L;
    if (hg->device != hu->device || a.N != b.N || a.K != b.K || a.bits != b.bits || a.group != b.group) return QL_ERR_INVALID_ARG;
    if ((int64_t)M * a.K > INT32_MAX || (int64_t)M * a.N > INT32_MAX) return QL_ERR_INVALID_ARG;
    if (device_timed_out(hg)) return QL_ERR_DEVICE_TIMEOUT;
    DeviceGuard guard(hg->device);
    if (!guard.ok) { cudaGetLastError(); return QL_ERR_CUDA; }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    qlinear_s* hs[2] = {hg, hu};
    if (M <= hg->gemv_max_m && !hg->use_stream) {                        // decode: both branches in one launch
        void* ys[2] = {y, y};
        const ql_status s = forward_gemv(hs, 2, x, ys, M, st, act);
        if (s != QL_ERR_UNSUPPORTED) return s;
    } else if (M > hg->gemv_max_m && gemm_pair_applicable(a, M)) {       // prefill: both accumulators of the CTA-pair kernel
        GemmPairLayers set{};
        set.n = 2;
        set.L[0] = &hg->L; set.blob[0] = hg->blob; set.y[0] = y; set.wmap[0] = hg->wmap_ok ? &hg->wmap : nullptr;
        set.L[1] = &hu->L; set.blob[1] = hu->blob; set.y[1] = y; set.wmap[1] = hu->wmap_ok ? &hu->wmap : nullptr;
        if (gemm_pair_ta_applicable(set, M, hg->num_sms, true)) return gemm_pair_ta_forward_gated(set, x, M, act, st, hg->device, hg->pdl, hg->num_sms);
        return gemm_pair_forward_gated(set, x, M, act, st, hg->device, hg->pdl, hg->num_sms);
    }
    // Unfused: the two projections into the device's shared scratch, then the element-wise product.
    const int64_t n = (int64_t)M * a.N;
    if ((size_t)n * 2 * sizeof(__half) > gemm_pair_scratch_bytes(hg->num_sms)) return QL_ERR_UNSUPPORTED;
    __half* g = reinterpret_cast<__half*>(hg->dev->gemm_scratch);
    __half* u = g + ((n + 7) & ~(int64_t)7);
    void* ys[2] = {g, u};
    ql_status s = qlinear_forward_group(hs, 2, x, ys, M, stream);
    if (s != QL_OK) return s;
    const int blocks = (int)std::min<int64_t>((n + 255) / 256, (int64_t)hg->num_sms * 8);
    gate_mul_kernel<<<blocks, 256, 0, st>>>(g, u, static_cast<__half*>(y), n, act);
    return cudaGetLastError() == cudaSuccess ? QL_OK : QL_ERR_CUDA;
}

namespace {
template <int BITS, bool GROUPED>
cudaError_t launch_a8(const qlinear_s* h, const GemvA8Params& prm, const GemvPlan& pl, cudaStream_t st)
{
    static std::atomic<bool> attr_set[kMaxDevices];
    auto kern = gemv_a8_kernel<BITS, GROUPED>;
    cudaError_t e = ensure_smem_attr(kern, attr_set, h->device, kGemvMaxSmem);
    if (e != cudaSuccess) return e;
    return launch(kern, prm, dim3(pl.grid), dim3(kGemvThreads), pl.smem_bytes, st, pl.cl, h->pdl);
}
}  // namespace

extern "C" ql_status qlinear_forward_a8(qlinear_t h, const void* x, void* y, int32_t M, void* stream)
{
    if (!h || !x || !y || M < 1) return QL_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y)) & 15) return QL_ERR_INVALID_ARG;
    if (device_timed_out(h)) return QL_ERR_DEVICE_TIMEOUT;
    const Layout& L = h->L;
    if (M > h->gemv_max_m) {
        // Prefill stage (Section 3.7): the quantisation kernel, then the integer matmul with output dequantisation.
        // Built for the per-channel schemes on the CTA-pair kernel; the quantised activations live in the device's
        // shared scratch (calls must be ordered against other users of it).
        if (L.grouped || (L.K % 128) || !gemm_pair_applicable(L, M)) return QL_ERR_UNSUPPORTED;
        const size_t xq_bytes = (((size_t)M * L.K + 255) / 256) * 256;
        const size_t arr = (size_t)((M + 255) / 256) * 256 * 4;             // per-token arrays padded to whole 256-token tiles
        if (xq_bytes + 2 * arr > gemm_pair_scratch_bytes(h->num_sms)) return QL_ERR_UNSUPPORTED;
        DeviceGuard guard(h->device);
        if (!guard.ok) { cudaGetLastError(); return QL_ERR_CUDA; }
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        unsigned char* base = reinterpret_cast<unsigned char*>(h->dev->gemm_scratch);
        signed char* xq = reinterpret_cast<signed char*>(base);
        float* sx = reinterpret_cast<float*>(base + xq_bytes);
        int32_t* rs = reinterpret_cast<int32_t*>(base + xq_bytes + arr);
        quantize_activations_kernel<<<M, 256, 0, st>>>(static_cast<const __half*>(x), xq, sx, rs, M, L.K);
        if (cudaGetLastError() != cudaSuccess) return QL_ERR_CUDA;
        GemmPairLayers set{};
        set.n = 1; set.L[0] = &h->L; set.blob[0] = h->blob; set.y[0] = y; set.wmap[0] = h->wmap_i8_ok ? &h->wmap_i8 : nullptr;
        if (gemm_pair_ta_i8_applicable(set, M, h->num_sms)) return gemm_pair_ta_forward_i8(set, xq, sx, rs, M, st, h->device, h->pdl, h->num_sms);
        return gemm_pair_forward_i8(set, xq, sx, rs, M, st, h->device, h->pdl, h->num_sms);
    }
    const GemvPlan pl = plan_gemv(L, h->n_rb, M, h->num_sms, false, true);
    if (pl.grid <= 0) return QL_ERR_UNSUPPORTED;
    DeviceGuard guard(h->device);
    if (!guard.ok) { cudaGetLastError(); return QL_ERR_CUDA; }
    GemvA8Params prm{};
    prm.body = h->blob + L.body_offset;
    prm.chan_scales = L.grouped ? nullptr : reinterpret_cast<const __half*>(h->blob + L.chan_scale_offset);
    prm.x = static_cast<const __half*>(x);
    prm.y = static_cast<__half*>(y);
    prm.M = M; prm.N = L.N; prm.K = L.K;
    prm.n_rb = h->n_rb; prm.n_kc = L.n_kc; prm.block_bytes = L.block_bytes;
    prm.ks_cta = pl.ks_cta; prm.ks_cta_log2 = pl.ks_cta == 8 ? 3 : pl.ks_cta == 4 ? 2 : pl.ks_cta == 2 ? 1 : 0; prm.cl = pl.cl; prm.cps = pl.cps;
    const int span = pl.ks_cta * pl.cps * L.chunk_k;
    prm.xq_stride = span + 32;
    prm.xq_bytes = ((M * prm.xq_stride + 15) / 16) * 16;
    prm.sg_bytes = span;                                                 // 32 bytes per 32-k group
    cudaError_t e;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (L.bits == 8) e = launch_a8<8, false>(h, prm, pl, st);
    else if (L.grouped) e = launch_a8<4, true>(h, prm, pl, st);
    else e = launch_a8<4, false>(h, prm, pl, st);
    return e == cudaSuccess ? QL_OK : QL_ERR_CUDA;
}

extern "C" ql_status qlinear_quantize_activations(const void* x, int8_t* xq, float* scale, int32_t M, int32_t K, int device, void* stream)
{
    if (!x || !xq || !scale || M < 1 || K < 32 || (K % 32)) return QL_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(xq)) & 15) return QL_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(scale) & 3) return QL_ERR_INVALID_ARG;
    if (device < 0 || device >= kMaxDevices) return QL_ERR_INVALID_ARG;
    DeviceGuard guard(device);
    if (!guard.ok) { cudaGetLastError(); return QL_ERR_CUDA; }
    quantize_activations_kernel<<<M, 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<const __half*>(x),
                                                                                reinterpret_cast<signed char*>(xq), scale, nullptr, M, K);
    return cudaGetLastError() == cudaSuccess ? QL_OK : QL_ERR_CUDA;
}

extern "C" ql_status qlinear_kv_append_heads(const qlinear_t* hk, const qlinear_t* hv, int32_t n_heads, const void* k_new, const void* v_new,
                                             int64_t head_stride, int64_t token_stride, void* const* v_scales, int32_t pos, int32_t n_new,
                                             void* stream)
{
    if (!hk || !hv || !v_scales || n_heads < 1 || n_heads > kKvMaxHeads || !k_new || !v_new || pos < 0 || n_new < 0) return QL_ERR_INVALID_ARG;
    if (head_stride < 0 || token_stride < 0 || ((head_stride | token_stride) & 7)) return QL_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(k_new) | reinterpret_cast<uintptr_t>(v_new)) & 15) return QL_ERR_INVALID_ARG;
    for (int i = 0; i < n_heads; ++i) {
        if (!hk[i] || !hv[i] || !v_scales[i] || (reinterpret_cast<uintptr_t>(v_scales[i]) & 15)) return QL_ERR_INVALID_ARG;
        const Layout &K = hk[i]->L, &V = hv[i]->L;
        if (hk[i]->device != hk[0]->device || hv[i]->device != hk[0]->device) return QL_ERR_INVALID_ARG;
        if (K.bits != 8 || V.bits != 8 || K.N != V.K || K.K != V.N || K.N != hk[0]->L.N || K.K != hk[0]->L.K) return QL_ERR_INVALID_ARG;
    }
    const Layout &K = hk[0]->L, &V = hv[0]->L;
    if ((int64_t)pos + n_new > K.N || K.K > 1024) return QL_ERR_INVALID_ARG;
    if (n_new == 0) return QL_OK;
    DeviceGuard guard(hk[0]->device);
    if (!guard.ok) { cudaGetLastError(); return QL_ERR_CUDA; }
    KvAppendParams prm{};
    for (int i = 0; i < n_heads; ++i) {
        uint8_t* kb = const_cast<uint8_t*>(hk[i]->blob);                 // the caches are the one kind of blob the library writes
        uint8_t* vb = const_cast<uint8_t*>(hv[i]->blob);
        prm.k_body[i] = kb + K.body_offset;
        prm.k_scales[i] = reinterpret_cast<__half*>(kb + K.chan_scale_offset);
        prm.v_body[i] = vb + V.body_offset;
        prm.v_scale[i] = static_cast<__half*>(v_scales[i]);
    }
    prm.k_new = static_cast<const __half*>(k_new);
    prm.v_new = static_cast<const __half*>(v_new);
    prm.head_stride = head_stride; prm.token_stride = token_stride;
    prm.d_h = K.K; prm.cache_size = K.N; prm.pos = pos; prm.n_new = n_new;
    prm.k_n_kc = K.n_kc; prm.v_n_kc = V.n_kc;
    const cudaError_t e = launch(kv_append_kernel, prm, dim3(n_new, n_heads), dim3(128), 0, static_cast<cudaStream_t>(stream), 1, hk[0]->pdl);
    return e == cudaSuccess ? QL_OK : QL_ERR_CUDA;
}

extern "C" ql_status qlinear_kv_append(qlinear_t hk, qlinear_t hv, const void* k_new, const void* v_new, void* v_scale,
                                       int32_t pos, int32_t n_new, void* stream)
{
    if (!hk || !hv) return QL_ERR_INVALID_ARG;
    return qlinear_kv_append_heads(&hk, &hv, 1, k_new, v_new, 0, hk->L.K, &v_scale, pos, n_new, stream);
}

extern "C" ql_status qlinear_kv_scores(qlinear_t hk, const void* q_rows, void* scores, int32_t R, void* stream)
{
    if (!hk || hk->L.bits != 8) return QL_ERR_INVALID_ARG;
    return qlinear_forward(hk, q_rows, scores, R, stream);
}

extern "C" ql_status qlinear_kv_scores_heads(const qlinear_t* hk, int32_t n_heads, const void* q_rows, void* scores, int32_t R, void* stream)
{
    if (!hk || n_heads < 1 || n_heads > kKvMaxHeads || !q_rows || !scores || R < 1) return QL_ERR_INVALID_ARG;
    for (int i = 0; i < n_heads; ++i)
        if (!hk[i] || hk[i]->L.bits != 8 || hk[i]->L.N != hk[0]->L.N || hk[i]->L.K != hk[0]->L.K) return QL_ERR_INVALID_ARG;
    const int64_t xs_stride = (int64_t)R * hk[0]->L.K, ys_stride = (int64_t)R * hk[0]->L.N;
    if ((xs_stride | ys_stride) & 7) return QL_ERR_INVALID_ARG;          // every head's rows start on a 16-byte boundary
    for (int h0 = 0; h0 < n_heads; h0 += kGemvMaxBatch) {
        const int n = std::min(kGemvMaxBatch, n_heads - h0);
        const void* xs[kGemvMaxBatch];
        void* ys[kGemvMaxBatch];
        for (int i = 0; i < n; ++i) {
            xs[i] = static_cast<const __half*>(q_rows) + (h0 + i) * xs_stride;
            ys[i] = static_cast<__half*>(scores) + (h0 + i) * ys_stride;
        }
        const ql_status s = qlinear_forward_batch(hk + h0, n, xs, ys, R, stream);
        if (s != QL_OK) return s;
    }
    return QL_OK;
}

extern "C" ql_status qlinear_kv_output_heads(const qlinear_t* hv, int32_t n_heads, const void* prob, const void* const* v_scales, void* out,
                                             int32_t R, void* stream)
{
    if (!hv || !v_scales || n_heads < 1 || n_heads > kKvMaxHeads || !prob || !out || R < 1) return QL_ERR_INVALID_ARG;
    for (int i = 0; i < n_heads; ++i) {
        if (!hv[i] || !v_scales[i] || (reinterpret_cast<uintptr_t>(v_scales[i]) & 15)) return QL_ERR_INVALID_ARG;
        if (hv[i]->L.bits != 8 || hv[i]->L.N != hv[0]->L.N || hv[i]->L.K != hv[0]->L.K || hv[i]->device != hv[0]->device) return QL_ERR_INVALID_ARG;
    }
    const Layout& V = hv[0]->L;
    const int64_t xs_stride = (int64_t)R * V.K, ys_stride = (int64_t)R * V.N;
    if ((xs_stride | ys_stride) & 7) return QL_ERR_INVALID_ARG;
    if (((reinterpret_cast<uintptr_t>(prob) | reinterpret_cast<uintptr_t>(out)) & 15) || xs_stride > INT32_MAX) return QL_ERR_INVALID_ARG;
    if (R > hv[0]->gemv_max_m || hv[0]->use_stream) return QL_ERR_UNSUPPORTED;          // the fused form exists in the decode kernel
    if (device_timed_out(hv[0])) return QL_ERR_DEVICE_TIMEOUT;
    DeviceGuard guard(hv[0]->device);
    if (!guard.ok) { cudaGetLastError(); return QL_ERR_CUDA; }
    for (int h0 = 0; h0 < n_heads; h0 += kGemvMaxBatch) {
        const int n = std::min(kGemvMaxBatch, n_heads - h0);
        const void* xs[kGemvMaxBatch];
        void* ys[kGemvMaxBatch];
        for (int i = 0; i < n; ++i) {
            xs[i] = static_cast<const __half*>(prob) + (h0 + i) * xs_stride;
            ys[i] = static_cast<__half*>(out) + (h0 + i) * ys_stride;
        }
        const ql_status s = forward_gemv(const_cast<qlinear_s* const*>(hv + h0), n, nullptr, ys, R, static_cast<cudaStream_t>(stream), -1, xs, v_scales + h0);
        if (s != QL_OK) return s;
    }
    return QL_OK;
}

extern "C" ql_status qlinear_kv_output(qlinear_t hv, const void* prob, const void* v_scale, void* tmp, void* out, int32_t R, void* stream)
{
    if (!hv || !prob || !v_scale || !tmp || !out || R < 1 || hv->L.bits != 8) return QL_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(tmp) | reinterpret_cast<uintptr_t>(out)) & 15) return QL_ERR_INVALID_ARG;
    const int T = hv->L.K;
    if ((int64_t)R * T > INT32_MAX) return QL_ERR_INVALID_ARG;
    // decode-sized products whose cache length is a whole number of chunks: the scales are applied inside the kernel
    if (!((reinterpret_cast<uintptr_t>(prob) | reinterpret_cast<uintptr_t>(v_scale)) & 15)) {
        const ql_status s = qlinear_kv_output_heads(&hv, 1, prob, &v_scale, out, R, stream);
        if (s != QL_ERR_UNSUPPORTED) return s;
    }
    {
        DeviceGuard guard(hv->device);
        if (!guard.ok) { cudaGetLastError(); return QL_ERR_CUDA; }
        const int64_t n = (int64_t)R * T;
        const int blocks = (int)std::min<int64_t>((n + 255) / 256, (int64_t)hv->num_sms * 8);
        kv_scale_probs_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<const __half*>(prob),
                                                                                     static_cast<const __half*>(v_scale), static_cast<__half*>(tmp), n, T);
        if (cudaGetLastError() != cudaSuccess) return QL_ERR_CUDA;
    }
    return qlinear_forward(hv, tmp, out, R, stream);
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

extern "C" ql_status qlinear_residual_rmsnorm(const void* x, const void* residual, const void* gamma, float eps, float gamma_offset,
                                              void* h_out, void* y_out, int32_t M, int32_t K, int32_t device, void* stream)
{
    if (!x || !gamma || !y_out || M < 0 || K < 8 || (K % 8) || device < 0) return QL_ERR_INVALID_ARG;
    if (!(eps >= 0.f) || y_out == h_out) return QL_ERR_INVALID_ARG;
    const uintptr_t all = reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(residual) | reinterpret_cast<uintptr_t>(gamma) |
                          reinterpret_cast<uintptr_t>(h_out) | reinterpret_cast<uintptr_t>(y_out);
    if (all & 15) return QL_ERR_INVALID_ARG;
    if (M == 0) return QL_OK;
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device >= n_dev) { cudaGetLastError(); return QL_ERR_INVALID_ARG; }
    DeviceGuard guard(device);
    if (!guard.ok) { cudaGetLastError(); return QL_ERR_CUDA; }
    NormParams prm{};
    prm.x = static_cast<const __half*>(x);
    prm.r = static_cast<const __half*>(residual);
    prm.g = static_cast<const __half*>(gamma);
    prm.h_out = static_cast<__half*>(h_out);
    prm.y_out = static_cast<__half*>(y_out);
    prm.eps = eps; prm.offset = gamma_offset; prm.M = M; prm.K = K;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int vpt = (K / 8 + kNormThreads - 1) / kNormThreads;           // 8-value vectors per thread
    const bool pdl = config().pdl;
    cudaError_t e;
    if (vpt <= 1) e = launch(residual_rmsnorm_kernel<1>, prm, dim3(M), dim3(kNormThreads), 0, st, 1, pdl);
    else if (vpt <= 2) e = launch(residual_rmsnorm_kernel<2>, prm, dim3(M), dim3(kNormThreads), 0, st, 1, pdl);
    else if (vpt <= 4) e = launch(residual_rmsnorm_kernel<4>, prm, dim3(M), dim3(kNormThreads), 0, st, 1, pdl);
    else if (vpt <= 8) e = launch(residual_rmsnorm_kernel<8>, prm, dim3(M), dim3(kNormThreads), 0, st, 1, pdl);
    else e = launch(residual_rmsnorm_kernel<0>, prm, dim3(M), dim3(kNormThreads), 0, st, 1, pdl);
    if (e != cudaSuccess) cudaGetLastError();
    return e == cudaSuccess ? QL_OK : QL_ERR_CUDA;
}

extern "C" ql_status qlinear_rope_qkv(const void* q, const void* k, const void* v, const int32_t* pos, const float* cos_t, const float* sin_t,
                                      int32_t n_pos, void* q_out, void* k_out, void* v_out, int32_t B, int32_t S, int32_t h_q, int32_t h_kv,
                                      int32_t d_h, int32_t device, void* stream)
{
    if (!q || !k || !v || !pos || !cos_t || !sin_t || !q_out || !k_out || !v_out) return QL_ERR_INVALID_ARG;
    if (B < 0 || S < 0 || h_q < 1 || h_kv < 1 || (h_q % h_kv) || d_h < 16 || (d_h % 16) || n_pos < 1 || device < 0) return QL_ERR_INVALID_ARG;
    if ((int64_t)B * S > INT32_MAX || (int64_t)B * S * h_q * d_h > ((int64_t)1 << 40)) return QL_ERR_INVALID_ARG;
    const uintptr_t all = reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k) | reinterpret_cast<uintptr_t>(v) | reinterpret_cast<uintptr_t>(cos_t) |
                          reinterpret_cast<uintptr_t>(sin_t) | reinterpret_cast<uintptr_t>(q_out) | reinterpret_cast<uintptr_t>(k_out) | reinterpret_cast<uintptr_t>(v_out);
    if ((all & 15) || (reinterpret_cast<uintptr_t>(pos) & 3)) return QL_ERR_INVALID_ARG;
    if (q_out == q || k_out == k || v_out == v) return QL_ERR_INVALID_ARG;   // the layout changes: not in place
    if ((int64_t)B * S == 0) return QL_OK;
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device >= n_dev) { cudaGetLastError(); return QL_ERR_INVALID_ARG; }
    DeviceGuard guard(device);
    if (!guard.ok) { cudaGetLastError(); return QL_ERR_CUDA; }
    RopeParams prm{};
    prm.q = static_cast<const __half*>(q); prm.k = static_cast<const __half*>(k); prm.v = static_cast<const __half*>(v);
    prm.pos = pos; prm.cos_t = cos_t; prm.sin_t = sin_t;
    prm.q_out = static_cast<__half*>(q_out); prm.k_out = static_cast<__half*>(k_out); prm.v_out = static_cast<__half*>(v_out);
    prm.B = B; prm.S = S; prm.h_q = h_q; prm.h_kv = h_kv; prm.d_h = d_h; prm.n_pos = n_pos;
    // threads: the work items of a token (8-element vectors of half a head) spread evenly over the fewest passes
    const int items = (h_q + h_kv) * (d_h / 16) + h_kv * (d_h / 8);
    const int passes = (items + kRopeThreads - 1) / kRopeThreads;
    const int threads = std::min(kRopeThreads, (((items + passes - 1) / passes) + 31) / 32 * 32);
    const cudaError_t e = launch(rope_qkv_kernel, prm, dim3(B * S), dim3(threads), 0, static_cast<cudaStream_t>(stream), 1, config().pdl);
    if (e != cudaSuccess) cudaGetLastError();
    return e == cudaSuccess ? QL_OK : QL_ERR_CUDA;
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
    static std::atomic<bool> attr_set[kMaxDevices];
    auto kern = gemv_stream_kernel<BITS, GROUPED, kStaticStages>;
    const size_t smem = (size_t)kStaticStages * StreamStage<BITS>::kBytes;
    cudaError_t e = ensure_smem_attr(kern, attr_set, device, (int)smem);
    if (e != cudaSuccess) return e;
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
    if (device < 0 || device >= kMaxDevices) return QL_ERR_INVALID_ARG;
    {
        int n_dev = 0;
        if (cudaGetDeviceCount(&n_dev) != cudaSuccess) { cudaGetLastError(); return QL_ERR_CUDA; }
        if (device >= n_dev) return QL_ERR_INVALID_ARG;
    }
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

// A kernel that does nothing but take part in programmatic dependent launch: what a launch costs on this machine.
__global__ void null_kernel(unsigned int* sink)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (sink && threadIdx.x == 0 && blockIdx.x == 0x7fffffff) *sink = 1;   // (never true: keeps the kernel from being empty code)
}

extern "C" ql_status qlinear_debug_null_launch(qlinear_t h, int32_t grid, int32_t block, void* stream)
{
    if (!h || grid < 1 || block < 1 || block > 1024) return QL_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) { cudaGetLastError(); return QL_ERR_CUDA; }
    const cudaError_t e = launch(null_kernel, static_cast<unsigned int*>(nullptr), dim3(grid), dim3(block), 0, static_cast<cudaStream_t>(stream), 1, h->pdl);
    return e == cudaSuccess ? QL_OK : QL_ERR_CUDA;
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
    // Clear the condition, and with it whatever an abandoned launch left in the shared arrival counters.
    const unsigned int zero[2] = {0, 0};
    cudaMemcpyToSymbol(g_device_flag, zero, sizeof(zero));
    h->dev->status_host[0] = 0;
    cudaMemset(h->dev->gemm_counters, 0, gemm_pair_counter_count(h->dev->sms) * sizeof(unsigned int));
    if (h->dev->stream_counters) cudaMemset(h->dev->stream_counters, 0, (size_t)kStreamMaxRsb * 8 * sizeof(unsigned int));
    cudaDeviceSynchronize();
    return QL_ERR_DEVICE_TIMEOUT;
}

extern "C" ql_status qlinear_destroy(qlinear_t h)
{
    if (!h) return QL_OK;
    {
        std::lock_guard<std::mutex> lock(g_dev_mutex);
        --h->dev->handles;                   // the device's shared state stays for the next handle (a few tens of MB)
    }
    delete h;
    return QL_OK;
}

extern "C" int32_t qlinear_debug_plan(qlinear_t h, int32_t M, int32_t* out, int32_t n_out)
{
    if (!h || M < 1 || M > 8 || !out) return 0;
    const int32_t v[8] = {h->use_stream ? 3 : 1, h->gemv[M].grid, h->gemv[M].cl, h->gemv[M].ks_cta, h->gemv[M].cps,
                          (int32_t)(1000 * h->gemv[M].max_over_mean), h->n_rb, h->L.n_kc};
    int n = n_out < 8 ? n_out : 8;
    for (int i = 0; i < n; ++i) out[i] = v[i];
    return n;
}

extern "C" uint32_t qlinear_debug_config_reads(void) { config(); return g_getenv_reads.load(); }

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


extern "C" uint32_t qlinear_version(void) { return (1u << 16) | 0u; }
