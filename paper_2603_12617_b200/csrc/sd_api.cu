// Host side of the C ABI declared in include/sd_verify.h: argument checks, workspace layout,
// choice of launch shape, the per-device scratch cache and the host-memory entry point.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>

#include "sd_kernels.cuh"
#include "sd_greedy.cuh"
#include "sd_errpos.cuh"
#include "sd_lmhead.cuh"
#include "sd_vocab_parallel.cuh"

namespace {

using namespace sdv;

constexpr int kMaxDevices = 64;
constexpr size_t kAlign = 256;
template <int DT> constexpr int stream_smem() { return RingStages<DT>::value * kStageBytes + (int)sizeof(StreamShared); }
constexpr int kStreamSmem = kRingStages * kStageBytes + (int)sizeof(StreamShared);
static_assert(kStreamSmem <= 227 * 1024, "ring does not fit the shared memory of a block");
constexpr int kL2PersistMiB = 0;
constexpr long long kL2BudgetMiB = 80;             // row pairs in flight between their two passes should fit this

// Tuning options: defaults, overridden once per process by the environment, then by sd_set_option.
struct Options {
    long long v[SD_OPT_COUNT];
};
std::once_flag g_opt_once;
std::mutex g_opt_mu;
Options g_opt;

void init_options() {
    std::call_once(g_opt_once, [] {
        static const struct { int id; const char* env; long long dflt; } table[] = {
            {SD_OPT_L2_PERSIST_MIB, "SD_VERIFY_L2_PERSIST_MIB", kL2PersistMiB},
            {SD_OPT_CLUSTER, "SD_VERIFY_CLUSTER", 0},
            {SD_OPT_LAG, "SD_VERIFY_LAG", -1},
            {SD_OPT_L2_BUDGET_MIB, "SD_VERIFY_L2_MIB", kL2BudgetMiB},
            {SD_OPT_FORCE_GENERIC, "SD_VERIFY_FORCE_GENERIC", 0},
            {SD_OPT_GREEDY_BLOCKS_PER_SM, "SD_GREEDY_BLOCKS_PER_SM", 4},
            {SD_OPT_WAIT_POLLS, "SD_VERIFY_WAIT_POLLS", (long long)kWaitLimit},
            {SD_OPT_PREFETCH, "SD_VERIFY_PREFETCH", 0},
        };
        for (const auto& t : table) {
            const char* e = getenv(t.env);
            g_opt.v[t.id] = (e && *e) ? atoll(e) : t.dflt;
        }
    });
}
long long option(int id) {
    init_options();
    std::lock_guard<std::mutex> lock(g_opt_mu);
    return g_opt.v[id];
}

thread_local char tl_cuda_error[256] = "";
thread_local int tl_info[6] = {0, 0, 0, 0, 0, 0};

int cuda_fail(cudaError_t e, const char* where) {
    snprintf(tl_cuda_error, sizeof tl_cuda_error, "%s: %s", where, cudaGetErrorString(e));
    return SD_ERR_CUDA;
}
#define SD_CUDA(call)                                         \
    do {                                                      \
        cudaError_t e_ = (call);                              \
        if (e_ != cudaSuccess) return cuda_fail(e_, #call);   \
    } while (0)

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
int elem_bytes(int dtype) { return dtype == SD_DTYPE_F32 ? 4 : 2; }
int vec_elems(int dtype) { return 16 / elem_bytes(dtype); }

struct WorkspaceLayout {
    size_t ticket, wstatus, sticky, accept, rowc, region_sums, hint_part, total;
    int NRmax;   // room for region sums per row: enough for either path at any cluster size
};

bool shape_ok(int B, int k, int V) {
    if (B < 1 || k < 1 || V < 1 || k > SD_MAX_K) return false;
    const long double n = (long double)B * (long double)(k + 1) * (long double)V;
    return n < 4.0e18L && (long double)B * (k + 1) < 2.0e9L;
}

WorkspaceLayout workspace_layout(int B, int k, int V, int dtype, bool with_hint = false) {
    WorkspaceLayout L;
    // room for region sums per row: enough for either path (the fast path's regions are 64 vectors,
    // 256 fp32 or 512 bf16 entries; the generic path's 512 entries)
    const int fast_elems = kRegionVecs * vec_elems(dtype);
    const int per = fast_elems < kGenericRegionElems ? fast_elems : kGenericRegionElems;
    L.NRmax = (V + per - 1) / per;
    size_t off = 0;
    L.ticket = off;      off = align_up(off + (size_t)B * 4, kAlign);
    L.wstatus = off;     off = align_up(off + (size_t)B * 4, kAlign);
    L.sticky = off;      off = align_up(off + 4, kAlign);
    L.accept = off;      off = align_up(off + (size_t)B * k, kAlign);
    L.rowc = off;        off = align_up(off + (size_t)B * (k + 1) * sizeof(RowConst), kAlign);
    L.region_sums = off; off = align_up(off + (size_t)B * (k + 1) * L.NRmax * 4, kAlign);
    L.hint_part = off;
    if (with_hint) off = align_up(off + (size_t)B * (k + 1) * kMaxCluster * 8, kAlign);
    L.total = off;
    return L;
}

struct StageSet {
    unsigned char* base = nullptr;
    size_t bytes = 0;
    cudaEvent_t in_ready = nullptr, comp_done = nullptr, out_done = nullptr;
};

struct DeviceState {
    DeviceState() { for (auto& row : max_clusters) for (int& v : row) v = -1; }
    std::mutex mu;
    bool probed = false;
    int cc_major = 0;
    int sm_count = 0;
    // grow-only scratch of the 13-argument entry points
    void* ws = nullptr;
    size_t ws_bytes = 0;
    // Leading bytes of ws known to be zero.  Every entry point wants the head of its own layout
    // zero (tickets, status words, error flag; keys of the greedy path), leaves that head zero and
    // writes whatever it likes behind it -- and where the head ends depends on the shape.  So a call
    // whose head is longer than this clears it first, and afterwards its own head is what is known.
    size_t ws_zero_bytes = 0;
    bool attr_set[2][4] = {};   // shared-memory / cluster attributes of the fast kernels
    int max_clusters[2][kMaxCluster + 1];   // resident clusters of 1..8 blocks, -1 = not asked yet
    // last launch-shape decision of the fast path
    int dec_dtype = -1, dec_V = 0, dec_forced = 0, dec_C = 0, dec_G = 0, dec_lag = 0, dec_use_lag = 0, dec_per = 0;
    long long dec_units = 0;
    double dec_l2 = 0.0;
    // output-layer gradient
    uint32_t* gemm_error = nullptr;
    bool gemm_attr = false;
    // host-memory entry point
    StageSet stage[2];
    cudaStream_t s_h2d = nullptr, s_comp = nullptr, s_d2h = nullptr;
};
DeviceState g_dev[kMaxDevices];

int current_device(int* dev, DeviceState** st) {
    cudaError_t e = cudaGetDevice(dev);
    if (e != cudaSuccess) {
        cuda_fail(e, "cudaGetDevice");
        return SD_ERR_NO_DEVICE;
    }
    if (*dev < 0 || *dev >= kMaxDevices) return SD_ERR_NO_DEVICE;
    DeviceState& d = g_dev[*dev];
    std::lock_guard<std::mutex> lock(d.mu);
    if (!d.probed) {
        cudaDeviceProp prop;
        e = cudaGetDeviceProperties(&prop, *dev);
        if (e != cudaSuccess) {
            cuda_fail(e, "cudaGetDeviceProperties");
            return SD_ERR_NO_DEVICE;
        }
        d.cc_major = prop.major;
        d.sm_count = prop.multiProcessorCount;
        // Optional: part of L2 set aside for lines fetched with the evict_last policy (pass 1 of the
        // fast path fetches with it what pass 2 reads again).  Off by default: with pass 2 walking a
        // row pair backwards it measured no better than no set-aside (0.509 ms against 0.511 ms on the
        // largest workload; 64 MiB and more: 0.67 ms and worse), and the caller's context stays as it was.
        {
            const long long mib = option(SD_OPT_L2_PERSIST_MIB);
            size_t want = (size_t)(mib > 0 ? mib : 0) << 20;
            if (want > (size_t)prop.persistingL2CacheMaxSize) want = (size_t)prop.persistingL2CacheMaxSize;
            if (want > 0 && cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, want) != cudaSuccess)
                (void)cudaGetLastError();   // not fatal: the path is only slower without it
        }
        d.probed = true;
    }
    if (d.cc_major != 10) {
        snprintf(tl_cuda_error, sizeof tl_cuda_error, "device %d has compute capability %d.x, need 10.x", *dev,
                 d.cc_major);
        return SD_ERR_NO_DEVICE;
    }
    *st = &d;
    return SD_OK;
}

// Launches the fast path with G clusters of C blocks, or (query_only) asks how many such
// clusters the device can hold at once.
template <int DT, bool ENS = false, bool STATS = false, bool HINT = false>
int launch_stream(DeviceState& d, const Params& P, int C, int G, int lag, cudaStream_t stream, bool query_only,
                  int* max_clusters) {
    auto kern = sd_stream_kernel<DT, ENS, STATS, HINT>;
    constexpr int kVariant = ENS ? 1 : STATS ? 2 : HINT ? 3 : 0;
    if (!d.attr_set[DT][kVariant]) {
        SD_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, stream_smem<DT>()));
        SD_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
        d.attr_set[DT][kVariant] = true;
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3((unsigned)(G * C), 1, 1);
    cfg.blockDim = dim3(kStreamThreads, 1, 1);
    cfg.dynamicSmemBytes = (size_t)stream_smem<DT>();
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)C;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (query_only) {
        int n = 0;
        cudaError_t e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            n = 0;
        }
        *max_clusters = n;
        return SD_OK;
    }
    const int prefetch = option(SD_OPT_PREFETCH) != 0 ? 1 : 0;
    SD_CUDA(cudaLaunchKernelEx(&cfg, kern, P, lag, prefetch));
    tl_info[0] = 1; tl_info[1] = C; tl_info[2] = kStreamThreads; tl_info[3] = stream_smem<DT>();
    tl_info[4] = G * C; tl_info[5] = 1;
    return SD_OK;
}

template <int DT>
int launch_generic(const Params& P, cudaStream_t stream) {
    const long long units = (long long)P.B * (P.k + 1);
    sd_generic_kernel<DT><<<(unsigned)units, kGenericThreads, 0, stream>>>(P);
    SD_CUDA(cudaGetLastError());
    tl_info[0] = 0; tl_info[1] = 1; tl_info[2] = kGenericThreads; tl_info[3] = 0;
    tl_info[4] = (int)units; tl_info[5] = 1;
    return SD_OK;
}

// Launch shape of the fast path: cluster size C (0 if the fast path cannot run), number of
// clusters G, vectors per sampling region, and how many stages of pass 1 of the next unit a
// consumer warp takes before pass 2 of a unit.
//
// A row is cut into stages and block r of a cluster of C takes every C-th share of them.  A
// block's slice lives in L2 between its two passes, so the row pairs the resident clusters work on
// at the same time should fit the part of L2 that holds on to them (about 80 MiB of the 126 MiB,
// measured: beyond it the second pass goes back to HBM).  Among the cluster sizes that fit, take
// the one that keeps most blocks busy (resident clusters, but no more clusters than units; 128
// busy blocks or more count alike), then the smaller cluster: larger slices spread the per-unit
// costs (exchange, row report) over more bytes and small clusters pack the GPU best (resident
// blocks: 148 for C = 1 and 2, 135 for 3, 132 for 4 and 6, 130 for 5, 112 for 7, 120 for 8).  If none fits, the
// largest cluster.
int choose_stream(DeviceState& d, int V, long long units, int dtype, int* G_out, int* per_out, int* lag_out) {
    const int forced = (int)option(SD_OPT_CLUSTER);
    const double l2_budget = (double)option(SD_OPT_L2_BUDGET_MIB) * 1048576.0;
    const int lag = (int)option(SD_OPT_LAG);       // stages of the next unit before pass 2 of a unit
    if (d.dec_dtype == dtype && d.dec_V == V && d.dec_units == units && d.dec_forced == forced &&
        d.dec_l2 == l2_budget && d.dec_lag == lag) {
        *G_out = d.dec_G;
        *per_out = d.dec_per;
        *lag_out = d.dec_use_lag;
        return d.dec_C;
    }
    const int NV = V / vec_elems(dtype);
    int best_C = 0, best_G = 0, best_per = 0;
    long long best_busy = -1;
    bool best_fits = false;
    Params dummy;
    memset(&dummy, 0, sizeof dummy);
    for (int C = 1; C <= kMaxCluster; ++C) {
        const int ci = C;
        if (forced > 0 && C != forced) continue;
        const int regions_row = (NV + kRegionVecs - 1) / kRegionVecs;
        const int regions_blk = (regions_row + C - 1) / C;
        if (d.max_clusters[dtype][ci] < 0) {
            int n = 0;
            int rc = dtype == SD_DTYPE_F32 ? launch_stream<SD_DTYPE_F32>(d, dummy, C, 1, 0, nullptr, true, &n)
                                           : launch_stream<SD_DTYPE_BF16>(d, dummy, C, 1, 0, nullptr, true, &n);
            d.max_clusters[dtype][ci] = (rc == SD_OK) ? n : 0;
        }
        const int resident = d.max_clusters[dtype][ci];
        if (resident < 1) continue;
        const int G = (int)(units < resident ? units : resident);
        const int used = (regions_row + regions_blk - 1) / regions_blk;   // blocks with work
        long long busy = (long long)G * (used < C ? used : C);
        if (busy > 128) busy = 128;
        const double in_flight = (double)G * (double)NV * 16.0 * 2.0;
        const bool fits = in_flight <= l2_budget;
        // a shape that fits L2 beats one that does not; then more busy blocks; then the smaller cluster
        const bool better = best_C == 0 || (fits && !best_fits) || (fits == best_fits && busy > best_busy) ||
                            (!fits && !best_fits);
        if (better) { best_C = C; best_G = G; best_per = kRegionVecs; best_busy = busy; best_fits = fits; }
    }
    // Stages of the next row pair that go before the second pass over a row pair: with few row
    // pairs per cluster every wait for an exchange shows (and the first and the last cannot hide),
    // so all of the next pair's first pass goes first; with many, the data between the passes is
    // what costs (L2 holds less of it), and the second pass follows the first at once.
    int use_lag = lag;
    if (lag == -1) use_lag = (best_G > 0 && units <= 8LL * best_G) ? 1 << 20 : 0;
    d.dec_dtype = dtype; d.dec_V = V; d.dec_units = units; d.dec_forced = forced; d.dec_l2 = l2_budget;
    d.dec_C = best_C; d.dec_G = best_G; d.dec_lag = lag; d.dec_use_lag = use_lag; d.dec_per = best_per;
    *G_out = best_G;
    *per_out = best_per;
    *lag_out = use_lag;
    return best_C;
}

uint32_t wait_polls() {
    const long long v = option(SD_OPT_WAIT_POLLS);
    return (uint32_t)(v < 1 ? 1 : v > (long long)kWaitLimit ? (long long)kWaitLimit : v);
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

int check_args(const void* T, const void* D, const int32_t* x, const float* u, float tau, int B, int k, int V,
               int dtype, const int32_t* accept_len, const int32_t* tokens, const float* loss, const void* grad,
               const float* acc_prob, const uint32_t* status) {
    if (dtype != SD_DTYPE_F32 && dtype != SD_DTYPE_BF16) return SD_ERR_DTYPE;
    if (!T || !D || !x || !u || !accept_len || !tokens) return SD_ERR_NULL;
    if (!shape_ok(B, k, V)) return SD_ERR_SHAPE;
    if (!(tau > 0.f) || !isfinite(tau)) return SD_ERR_TEMPERATURE;
    const size_t es = (size_t)elem_bytes(dtype);
    if (!aligned(T, es) || !aligned(D, es) || (grad && !aligned(grad, es))) return SD_ERR_ALIGN;
    if (!aligned(x, 4) || !aligned(u, 4) || !aligned(accept_len, 4) || !aligned(tokens, 4) ||
        (loss && !aligned(loss, 4)) || (acc_prob && !aligned(acc_prob, 4)) || (status && !aligned(status, 4)))
        return SD_ERR_ALIGN;
    return SD_OK;
}

// Enqueue the step on `stream` with scratch `ws` (device, layout L).  clean: tickets/status are zero.
int run_device(DeviceState& d, const void* T, const void* D, const int32_t* x, const float* u, float tau, int B,
               int k, int V, int dtype, int32_t* accept_len, int32_t* tokens, float* loss, void* grad,
               float* acc_prob, uint32_t* status, unsigned char* ws, const WorkspaceLayout& L, bool clean,
               cudaStream_t stream, const void* hint = nullptr, float* hint_err = nullptr) {
    Params P;
    memset(&P, 0, sizeof P);
    P.T = T; P.D = D; P.x = x; P.u = u;
    P.B = B; P.k = k; P.V = V;
    P.c = (float)(1.4426950408889634 / (double)tau);
    P.tau = tau;
    P.inv_tau = 1.0 / (double)tau;
    P.accept_len = accept_len; P.tokens = tokens; P.loss = loss; P.grad = grad;
    P.acc_prob = acc_prob; P.status = status;
    P.ticket = reinterpret_cast<uint32_t*>(ws + L.ticket);
    P.wstatus = reinterpret_cast<uint32_t*>(ws + L.wstatus);
    P.sticky = reinterpret_cast<uint32_t*>(ws + L.sticky);
    P.accept = ws + L.accept;
    P.rowc = reinterpret_cast<RowConst*>(ws + L.rowc);
    P.region_sums = reinterpret_cast<float*>(ws + L.region_sums);
    P.wait_polls = wait_polls();
    P.hint = hint;
    P.hint_err = hint_err;
    P.hint_part = hint ? reinterpret_cast<double*>(ws + L.hint_part) : nullptr;

    if (!clean) SD_CUDA(cudaMemsetAsync(ws, 0, L.accept, stream));   // tickets, status words, sticky flag
    if (status) SD_CUDA(cudaMemsetAsync(status, 0, (size_t)B * 4, stream));   // bits are ORed in on the device

    const size_t row_bytes = (size_t)V * elem_bytes(dtype);
    const bool fast = (row_bytes % 16 == 0) && aligned(T, 16) && aligned(D, 16) && (!grad || aligned(grad, 16)) &&
                      (!hint || aligned(hint, 16)) && option(SD_OPT_FORCE_GENERIC) == 0;
    int C = 0, G = 0, lag = 0, per = 0;
    if (fast) C = choose_stream(d, V, (long long)B * (k + 1), dtype, &G, &per, &lag);
    int rc;
    if (C > 0) {
        P.blocks_per_unit = C;
        P.RE = per * vec_elems(dtype);
        P.NR = (V + P.RE - 1) / P.RE;
        if (hint)
            rc = dtype == SD_DTYPE_F32 ? launch_stream<SD_DTYPE_F32, false, false, true>(d, P, C, G, lag, stream, false, nullptr)
                                       : launch_stream<SD_DTYPE_BF16, false, false, true>(d, P, C, G, lag, stream, false, nullptr);
        else
            rc = dtype == SD_DTYPE_F32 ? launch_stream<SD_DTYPE_F32>(d, P, C, G, lag, stream, false, nullptr)
                                       : launch_stream<SD_DTYPE_BF16>(d, P, C, G, lag, stream, false, nullptr);
    } else {
        P.blocks_per_unit = 1;
        P.RE = kGenericRegionElems;
        P.NR = (V + P.RE - 1) / P.RE;
        rc = dtype == SD_DTYPE_F32 ? launch_generic<SD_DTYPE_F32>(P, stream)
                                   : launch_generic<SD_DTYPE_BF16>(P, stream);
    }
    return rc;
}

int run_cached(const void* T, const void* D, const int32_t* x, const float* u, float tau, int B, int k, int V,
               int dtype, int32_t* accept_len, int32_t* tokens, float* loss, void* grad, void* stream) {
    int rc = check_args(T, D, x, u, tau, B, k, V, dtype, accept_len, tokens, loss, grad, nullptr, nullptr);
    if (rc != SD_OK) return rc;
    int dev;
    DeviceState* d = nullptr;
    rc = current_device(&dev, &d);
    if (rc != SD_OK) return rc;
    const WorkspaceLayout L = workspace_layout(B, k, V, dtype);
    std::lock_guard<std::mutex> lock(d->mu);
    if (d->ws_bytes < L.total) {
        if (d->ws) {
            SD_CUDA(cudaDeviceSynchronize());
            SD_CUDA(cudaFree(d->ws));
            d->ws = nullptr;
            d->ws_bytes = 0;
        }
        const size_t want = align_up(L.total + L.total / 4, 1 << 20);
        SD_CUDA(cudaMalloc(&d->ws, want));
        d->ws_bytes = want;
        d->ws_zero_bytes = 0;
    }
    // the head of this layout (tickets, status words, error flag) must be zero on entry; the kernel
    // leaves it zero again and dirties everything behind it
    const bool clean = d->ws_zero_bytes >= L.accept;
    d->ws_zero_bytes = 0;
    rc = run_device(*d, T, D, x, u, tau, B, k, V, dtype, accept_len, tokens, loss, grad, nullptr, nullptr,
                    static_cast<unsigned char*>(d->ws), L, clean, static_cast<cudaStream_t>(stream));
    if (rc == SD_OK) d->ws_zero_bytes = L.accept;   // a failed launch may leave anything behind
    return rc;
}

// ---- scratch that nobody allocates --------------------------------------------------------
// For callers that must not allocate device memory (see sd_verify_feedback_static in the header):
// the scratch of the step lives in the library's own image.  Every GPU that loads the library
// holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[SD_STATIC_SCRATCH_BYTES];

// In host code the name g_static_scratch is only a handle of the symbol, not a device address:
// the address on a given GPU comes from cudaGetSymbolAddress, asked once per device while that
// device is current.
std::mutex g_static_mu;
unsigned char* g_static_ptr[kMaxDevices] = {};

int static_scratch(int dev, unsigned char** out) {
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {
        void* ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress(g_static_scratch)");
        if (!ptr || !aligned(ptr, kAlign)) {
            snprintf(tl_cuda_error, sizeof tl_cuda_error, "static scratch has no usable device address");
            return SD_ERR_CUDA;
        }
        g_static_ptr[dev] = static_cast<unsigned char*>(ptr);
    }
    *out = g_static_ptr[dev];
    return SD_OK;
}

// ---- tensor maps for the output-layer gradient ---------------------------------------------
// cuTensorMapEncodeTiled lives in the driver; its address comes from the runtime, so the library
// links against nothing but the CUDA runtime.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            (void)cudaGetLastError();
    });
    return fn;
}
// Map of a row-major bf16 matrix [rows, cols] (device memory of this GPU) for boxes of
// box_rows x 64 columns in the 128-byte swizzle; entries outside the matrix read as zero.
int bf16_matrix_map(CUtensorMap* map, const void* base, int rows, int cols, int box_rows) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) {
        snprintf(tl_cuda_error, sizeof tl_cuda_error, "cuTensorMapEncodeTiled is not available from this driver");
        return SD_ERR_CUDA;
    }
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kGemmChunk, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(tl_cuda_error, sizeof tl_cuda_error, "cuTensorMapEncodeTiled failed with code %d", (int)r);
        return SD_ERR_CUDA;
    }
    return SD_OK;
}

}  // namespace

extern "C" {

int sd_verify_feedback(const float* target_logits, const float* draft_logits, const int32_t* draft_tokens,
                       const float* uniforms, float temperature, int B, int k, int V, int32_t* out_accept_len,
                       int32_t* out_tokens, float* out_loss, float* out_grad_draft, void* stream) {
    return run_cached(target_logits, draft_logits, draft_tokens, uniforms, temperature, B, k, V, SD_DTYPE_F32,
                      out_accept_len, out_tokens, out_loss, out_grad_draft, stream);
}

int sd_verify_feedback_bf16(const uint16_t* target_logits, const uint16_t* draft_logits,
                            const int32_t* draft_tokens, const float* uniforms, float temperature, int B, int k,
                            int V, int32_t* out_accept_len, int32_t* out_tokens, float* out_loss,
                            uint16_t* out_grad_draft, void* stream) {
    return run_cached(target_logits, draft_logits, draft_tokens, uniforms, temperature, B, k, V, SD_DTYPE_BF16,
                      out_accept_len, out_tokens, out_loss, out_grad_draft, stream);
}

size_t sd_workspace_bytes(int B, int k, int V, int dtype) {
    if ((dtype != SD_DTYPE_F32 && dtype != SD_DTYPE_BF16) || !shape_ok(B, k, V)) return 0;
    return workspace_layout(B, k, V, dtype).total;
}

int sd_verify_feedback_ex(const void* target_logits, const void* draft_logits, const int32_t* draft_tokens,
                          const float* uniforms, float temperature, int B, int k, int V, int dtype,
                          int32_t* out_accept_len, int32_t* out_tokens, float* out_loss, void* out_grad_draft,
                          float* out_acc_prob, uint32_t* out_status, void* workspace, size_t workspace_bytes,
                          void* stream) {
    int rc = check_args(target_logits, draft_logits, draft_tokens, uniforms, temperature, B, k, V, dtype,
                        out_accept_len, out_tokens, out_loss, out_grad_draft, out_acc_prob, out_status);
    if (rc != SD_OK) return rc;
    const WorkspaceLayout L = workspace_layout(B, k, V, dtype);
    if (!workspace || !aligned(workspace, kAlign) || workspace_bytes < L.total) return SD_ERR_WORKSPACE;
    int dev;
    DeviceState* d = nullptr;
    rc = current_device(&dev, &d);
    if (rc != SD_OK) return rc;
    std::lock_guard<std::mutex> lock(d->mu);
    return run_device(*d, target_logits, draft_logits, draft_tokens, uniforms, temperature, B, k, V, dtype,
                      out_accept_len, out_tokens, out_loss, out_grad_draft, out_acc_prob, out_status,
                      static_cast<unsigned char*>(workspace), L, false, static_cast<cudaStream_t>(stream));
}

size_t sd_hint_workspace_bytes(int B, int k, int V, int dtype) {
    if ((dtype != SD_DTYPE_F32 && dtype != SD_DTYPE_BF16) || !shape_ok(B, k, V)) return 0;
    return workspace_layout(B, k, V, dtype, true).total;
}

int sd_verify_feedback_hint(const void* target_logits, const void* draft_logits, const int32_t* draft_tokens,
                            const float* uniforms, float temperature, int B, int k, int V, int dtype, const void* hint,
                            int32_t* out_accept_len, int32_t* out_tokens, float* out_loss, void* out_grad_draft,
                            float* out_hint_err, uint32_t* out_status, void* workspace, size_t workspace_bytes,
                            void* stream) {
    int rc = check_args(target_logits, draft_logits, draft_tokens, uniforms, temperature, B, k, V, dtype,
                        out_accept_len, out_tokens, out_loss, out_grad_draft, nullptr, out_status);
    if (rc != SD_OK) return rc;
    if (!hint || !out_hint_err) return SD_ERR_NULL;
    if (!aligned(hint, (size_t)elem_bytes(dtype)) || !aligned(out_hint_err, 4)) return SD_ERR_ALIGN;
    const WorkspaceLayout L = workspace_layout(B, k, V, dtype, true);
    if (!workspace || !aligned(workspace, kAlign) || workspace_bytes < L.total) return SD_ERR_WORKSPACE;
    int dev;
    DeviceState* d = nullptr;
    rc = current_device(&dev, &d);
    if (rc != SD_OK) return rc;
    std::lock_guard<std::mutex> lock(d->mu);
    return run_device(*d, target_logits, draft_logits, draft_tokens, uniforms, temperature, B, k, V, dtype,
                      out_accept_len, out_tokens, out_loss, out_grad_draft, nullptr, out_status,
                      static_cast<unsigned char*>(workspace), L, false, static_cast<cudaStream_t>(stream), hint,
                      out_hint_err);
}

int sd_verify_feedback_static(const void* target_logits, const void* draft_logits, const int32_t* draft_tokens,
                              const float* uniforms, float temperature, int B, int k, int V, int dtype,
                              int32_t* out_accept_len, int32_t* out_tokens, float* out_loss, void* out_grad_draft,
                              float* out_acc_prob, uint32_t* out_status, void* stream) {
    int rc = check_args(target_logits, draft_logits, draft_tokens, uniforms, temperature, B, k, V, dtype,
                        out_accept_len, out_tokens, out_loss, out_grad_draft, out_acc_prob, out_status);
    if (rc != SD_OK) return rc;
    const WorkspaceLayout L = workspace_layout(B, k, V, dtype);
    if (L.total > (size_t)SD_STATIC_SCRATCH_BYTES) {
        snprintf(tl_cuda_error, sizeof tl_cuda_error,
                 "this shape needs %zu bytes of scratch, the built-in scratch has %d: use sd_verify_feedback_ex",
                 L.total, SD_STATIC_SCRATCH_BYTES);
        return SD_ERR_WORKSPACE;
    }
    int dev;
    DeviceState* d = nullptr;
    rc = current_device(&dev, &d);
    if (rc != SD_OK) return rc;
    unsigned char* scratch = nullptr;
    rc = static_scratch(dev, &scratch);   // first call on this device: looks the address up
    if (rc != SD_OK) return rc;
    std::lock_guard<std::mutex> lock(d->mu);
    // clean = false: the tickets, status words and error flag at the head of the scratch are zeroed
    // on the stream before the kernel, whatever the previous call left there
    return run_device(*d, target_logits, draft_logits, draft_tokens, uniforms, temperature, B, k, V, dtype,
                      out_accept_len, out_tokens, out_loss, out_grad_draft, out_acc_prob, out_status, scratch, L, false,
                      static_cast<cudaStream_t>(stream));
}

// ---- online ensemble -------------------------------------------------------------------------
int sd_ensemble_feedback(const void* target_logits, const void* const* draft_logits, int n_learners,
                         float temperature, float epsilon, int B, int k, int V, int dtype,
                         const double* cum_loss_in, float* out_loss, void* const* out_grad,
                         double* out_round_loss, double* out_cum_loss, float* out_weights, uint32_t* out_status,
                         void* workspace, size_t workspace_bytes, void* stream) {
    if (dtype != SD_DTYPE_F32 && dtype != SD_DTYPE_BF16) return SD_ERR_DTYPE;
    if (!target_logits || !draft_logits || !out_loss || !out_round_loss || !out_cum_loss || !out_weights)
        return SD_ERR_NULL;
    if (n_learners < 1 || n_learners > SD_MAX_LEARNERS || !shape_ok(B, k, V)) return SD_ERR_SHAPE;
    if ((long double)B * k * n_learners >= 2.0e9L) return SD_ERR_SHAPE;
    if (!(temperature > 0.f) || !isfinite(temperature)) return SD_ERR_TEMPERATURE;
    if (!(epsilon >= 0.f) || !isfinite(epsilon)) return SD_ERR_TEMPERATURE;
    const size_t row_bytes = (size_t)V * elem_bytes(dtype);
    if (row_bytes % 16 != 0 || !aligned(target_logits, 16)) return SD_ERR_ALIGN;
    for (int n = 0; n < n_learners; ++n) {
        if (!draft_logits[n]) return SD_ERR_NULL;
        if (!aligned(draft_logits[n], 16) || (out_grad && out_grad[n] && !aligned(out_grad[n], 16))) return SD_ERR_ALIGN;
    }
    if (!aligned(out_loss, 4) || !aligned(out_round_loss, 8) || !aligned(out_cum_loss, 8) || !aligned(out_weights, 4) ||
        (cum_loss_in && !aligned(cum_loss_in, 8)) || (out_status && !aligned(out_status, 4)))
        return SD_ERR_ALIGN;
    if (workspace && (!aligned(workspace, kAlign) || workspace_bytes < SD_ENSEMBLE_SCRATCH_BYTES)) return SD_ERR_WORKSPACE;
    int dev;
    DeviceState* d = nullptr;
    int rc = current_device(&dev, &d);
    if (rc != SD_OK) return rc;
    std::lock_guard<std::mutex> lock(d->mu);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    if (!ws) {
        if (!d->ws) {
            const size_t want = 1 << 20;
            SD_CUDA(cudaMalloc(&d->ws, want));
            d->ws_bytes = want;
            d->ws_zero_bytes = 0;
        }
        ws = static_cast<unsigned char*>(d->ws);
        d->ws_zero_bytes = 0;      // the flag word of this call sits where other entry points expect zeros
    }
    SD_CUDA(cudaMemsetAsync(ws, 0, SD_ENSEMBLE_SCRATCH_BYTES, st));
    if (out_status) SD_CUDA(cudaMemsetAsync(out_status, 0, (size_t)B * 4, st));

    Params P;
    memset(&P, 0, sizeof P);
    P.T = target_logits;
    P.B = B; P.k = k; P.V = V;
    P.c = (float)(1.4426950408889634 / (double)temperature);
    P.tau = temperature;
    P.inv_tau = 1.0 / (double)temperature;
    P.loss = out_loss;
    P.status = out_status;
    P.sticky = reinterpret_cast<uint32_t*>(ws);
    P.learners = n_learners;
    P.wait_polls = wait_polls();
    for (int n = 0; n < n_learners; ++n) {
        P.Dn[n] = draft_logits[n];
        P.Gn[n] = out_grad ? out_grad[n] : nullptr;
    }
    int G = 0, lag = 0, per = 0;
    const int C = choose_stream(*d, V, (long long)B * k * n_learners, dtype, &G, &per, &lag);
    if (C <= 0) return SD_ERR_CUDA;
    P.blocks_per_unit = C;
    P.RE = per * vec_elems(dtype);
    P.NR = (V + P.RE - 1) / P.RE;
    rc = dtype == SD_DTYPE_F32 ? launch_stream<SD_DTYPE_F32, true>(*d, P, C, G, lag, st, false, nullptr)
                               : launch_stream<SD_DTYPE_BF16, true>(*d, P, C, G, lag, st, false, nullptr);
    if (rc != SD_OK) return rc;
    sd_hedge_kernel<<<1, 256, 0, st>>>(out_loss, n_learners, (long long)B * k, (double)epsilon, cum_loss_in,
                                       out_round_loss, out_cum_loss, out_weights, P.sticky, out_status, B);
    SD_CUDA(cudaGetLastError());
    tl_info[0] = 3; tl_info[5] = 2;
    return SD_OK;
}

// ---- error-position feedback -------------------------------------------------------------------
int sd_verify_error_feedback(const void* target_logits, const void* draft_logits, const int32_t* draft_tokens,
                             const float* uniforms, float temperature, int B, int k, int V, int dtype,
                             int32_t* out_accept_len, int32_t* out_tokens, float* out_loss, void* out_error_grad,
                             uint32_t* out_status, void* workspace, size_t workspace_bytes, void* stream) {
    int rc = check_args(target_logits, draft_logits, draft_tokens, uniforms, temperature, B, k, V, dtype,
                        out_accept_len, out_tokens, out_loss, out_error_grad, nullptr, out_status);
    if (rc != SD_OK) return rc;
    const size_t row_bytes = (size_t)V * elem_bytes(dtype);
    if (row_bytes % 16 != 0 || !aligned(target_logits, 16) || !aligned(draft_logits, 16) ||
        (out_error_grad && !aligned(out_error_grad, 16)))
        return SD_ERR_ALIGN;
    const WorkspaceLayout L = workspace_layout(B, k, V, dtype);
    if (workspace && (!aligned(workspace, kAlign) || workspace_bytes < L.total)) return SD_ERR_WORKSPACE;
    int dev;
    DeviceState* d = nullptr;
    rc = current_device(&dev, &d);
    if (rc != SD_OK) return rc;
    std::lock_guard<std::mutex> lock(d->mu);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    if (!ws) {
        // the library's own scratch, shared with the other entry points and grown on demand
        if (d->ws_bytes < L.total) {
            if (d->ws) {
                SD_CUDA(cudaDeviceSynchronize());
                SD_CUDA(cudaFree(d->ws));
                d->ws = nullptr;
                d->ws_bytes = 0;
            }
            const size_t want = align_up(L.total + L.total / 4, 1 << 20);
            SD_CUDA(cudaMalloc(&d->ws, want));
            d->ws_bytes = want;
        }
        ws = static_cast<unsigned char*>(d->ws);
        d->ws_zero_bytes = 0;     // cleared below for this call; what it leaves behind is not tracked
    }
    Params P;
    memset(&P, 0, sizeof P);
    P.T = target_logits; P.D = draft_logits; P.x = draft_tokens; P.u = uniforms;
    P.B = B; P.k = k; P.V = V;
    P.c = (float)(1.4426950408889634 / (double)temperature);
    P.tau = temperature;
    P.inv_tau = 1.0 / (double)temperature;
    P.accept_len = out_accept_len; P.tokens = out_tokens; P.loss = out_loss; P.grad = out_error_grad;
    P.status = out_status;
    P.ticket = reinterpret_cast<uint32_t*>(ws + L.ticket);
    P.wstatus = reinterpret_cast<uint32_t*>(ws + L.wstatus);
    P.sticky = reinterpret_cast<uint32_t*>(ws + L.sticky);
    P.accept = ws + L.accept;
    P.rowc = reinterpret_cast<RowConst*>(ws + L.rowc);
    P.region_sums = reinterpret_cast<float*>(ws + L.region_sums);
    P.wait_polls = wait_polls();
    SD_CUDA(cudaMemsetAsync(ws, 0, L.accept, st));   // tickets, status words, sticky flag
    if (out_status) SD_CUDA(cudaMemsetAsync(out_status, 0, (size_t)B * 4, st));   // bits are ORed in on the device
    int G = 0, lag = 0, per = 0;
    const int C = choose_stream(*d, V, (long long)B * (k + 1), dtype, &G, &per, &lag);
    if (C <= 0) return SD_ERR_CUDA;
    P.blocks_per_unit = C;
    P.RE = per * vec_elems(dtype);
    P.NR = (V + P.RE - 1) / P.RE;
    rc = dtype == SD_DTYPE_F32 ? launch_stream<SD_DTYPE_F32, false, true>(*d, P, C, G, lag, st, false, nullptr)
                               : launch_stream<SD_DTYPE_BF16, false, true>(*d, P, C, G, lag, st, false, nullptr);
    if (rc != SD_OK) return rc;
    const int slices = (P.NR + kErrSliceRegions - 1) / kErrSliceRegions;
    const unsigned grid = (unsigned)B * (unsigned)slices;
    if (dtype == SD_DTYPE_F32) sd_errpos_kernel<SD_DTYPE_F32><<<grid, kErrThreads, 0, st>>>(P, slices);
    else                       sd_errpos_kernel<SD_DTYPE_BF16><<<grid, kErrThreads, 0, st>>>(P, slices);
    SD_CUDA(cudaGetLastError());
    tl_info[0] = 4; tl_info[5] = 2;
    return SD_OK;
}

size_t sd_greedy_workspace_bytes(int B, int k) {
    if (B < 1 || k < 1 || k > SD_MAX_K || (long double)B * (k + 1) >= 2.0e9L) return 0;
    return kAlign + align_up((size_t)B * (k + 1) * 8, kAlign);   // ticket word, keys
}

int sd_verify_greedy(const void* target_logits, const int32_t* draft_tokens, int B, int k, int V, int dtype,
                     int32_t* out_accept_len, int32_t* out_tokens, int32_t* out_argmax, void* workspace,
                     size_t workspace_bytes, void* stream) {
    if (dtype != SD_DTYPE_F32 && dtype != SD_DTYPE_BF16) return SD_ERR_DTYPE;
    if (!target_logits || !draft_tokens || !out_accept_len || !out_tokens) return SD_ERR_NULL;
    if (!shape_ok(B, k, V)) return SD_ERR_SHAPE;
    const size_t es = (size_t)elem_bytes(dtype);
    if (!aligned(target_logits, es) || !aligned(draft_tokens, 4) || !aligned(out_accept_len, 4) ||
        !aligned(out_tokens, 4) || (out_argmax && !aligned(out_argmax, 4)))
        return SD_ERR_ALIGN;
    const size_t need = sd_greedy_workspace_bytes(B, k);
    if (workspace && (!aligned(workspace, kAlign) || workspace_bytes < need)) return SD_ERR_WORKSPACE;
    int dev;
    DeviceState* d = nullptr;
    int rc = current_device(&dev, &d);
    if (rc != SD_OK) return rc;
    std::lock_guard<std::mutex> lock(d->mu);
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // The kernel wants its ticket word and keys zero and leaves them zero.  A caller's workspace is
    // cleared every call; the library's own scratch (shared with sd_verify_feedback, grown on
    // demand) only when something else has written there since.
    bool clean = false;
    if (!ws) {
        if (d->ws_bytes < need) {
            if (d->ws) {
                SD_CUDA(cudaDeviceSynchronize());
                SD_CUDA(cudaFree(d->ws));
                d->ws = nullptr;
                d->ws_bytes = 0;
            }
            const size_t want = align_up(need + need / 4, 1 << 20);
            SD_CUDA(cudaMalloc(&d->ws, want));
            d->ws_bytes = want;
            SD_CUDA(cudaMemset(d->ws, 0, want));
            SD_CUDA(cudaDeviceSynchronize());
            d->ws_zero_bytes = want;
        }
        ws = static_cast<unsigned char*>(d->ws);
        clean = d->ws_zero_bytes >= need;
    }
    if (!clean) SD_CUDA(cudaMemsetAsync(ws, 0, need, st));
    GreedyParams P;
    memset(&P, 0, sizeof P);
    P.T = target_logits; P.x = draft_tokens;
    P.B = B; P.k = k; P.V = V;
    P.accept_len = out_accept_len; P.tokens = out_tokens; P.argmax = out_argmax;
    P.ticket = reinterpret_cast<uint32_t*>(ws);
    P.keys = reinterpret_cast<unsigned long long*>(ws + kAlign);
    const int item_elems = kGreedyItemVecs * vec_elems(dtype);
    P.items_per_row = (V + item_elems - 1) / item_elems;
    P.vectorised = (((size_t)V * es) % 16 == 0 && aligned(target_logits, 16)) ? 1 : 0;
    const long long items = (long long)B * (k + 1) * P.items_per_row;
    // blocks per SM: 4 of 256 threads, 8 loads of 16 bytes in flight per thread, measured best among 2..8
    // on the largest workload (more blocks disturb the DRAM page locality of the streams);
    // option SD_OPT_GREEDY_BLOCKS_PER_SM (1..8) overrides it
    int per_sm = (int)option(SD_OPT_GREEDY_BLOCKS_PER_SM);
    if (per_sm < 1 || per_sm > 8) per_sm = 4;
    const long long cap = (long long)d->sm_count * per_sm;
    const unsigned grid = (unsigned)(items < cap ? items : cap);
    if (dtype == SD_DTYPE_F32) sd_greedy_kernel<SD_DTYPE_F32><<<grid, kGreedyThreads, 0, st>>>(P);
    else                       sd_greedy_kernel<SD_DTYPE_BF16><<<grid, kGreedyThreads, 0, st>>>(P);
    const cudaError_t launched = cudaGetLastError();
    if (!workspace) d->ws_zero_bytes = launched == cudaSuccess ? (clean ? d->ws_zero_bytes : need) : 0;
    SD_CUDA(launched);
    tl_info[0] = 2; tl_info[1] = 1; tl_info[2] = kGreedyThreads; tl_info[3] = 0;
    tl_info[4] = (int)grid; tl_info[5] = 1;
    return SD_OK;
}

int sd_verify_feedback_host(const void* target_logits, const void* draft_logits, const int32_t* draft_tokens,
                            const float* uniforms, float temperature, int B, int k, int V, int dtype,
                            int32_t* out_accept_len, int32_t* out_tokens, float* out_loss, void* out_grad_draft,
                            float* out_acc_prob, uint32_t* out_status) {
    int rc = check_args(target_logits, draft_logits, draft_tokens, uniforms, temperature, B, k, V, dtype,
                        out_accept_len, out_tokens, out_loss, out_grad_draft, out_acc_prob, out_status);
    if (rc != SD_OK) return rc;
    int dev;
    DeviceState* d = nullptr;
    rc = current_device(&dev, &d);
    if (rc != SD_OK) return rc;
    std::lock_guard<std::mutex> lock(d->mu);

    const size_t es = (size_t)elem_bytes(dtype);
    const size_t t_seq = (size_t)(k + 1) * V * es, d_seq = (size_t)k * V * es;
    // sequences per slice: about 96 MiB of logits and gradient in flight per buffer set
    const size_t per_seq = t_seq + 2 * d_seq;
    int S = (int)((96u << 20) / per_seq);
    if (S < 1) S = 1;
    if (S > B) S = B;
    const int nslices = (B + S - 1) / S;

    // one device arena per buffer set
    const WorkspaceLayout L = workspace_layout(S, k, V, dtype);
    size_t off = 0;
    const size_t oT = off;   off = align_up(off + (size_t)S * t_seq, kAlign);
    const size_t oD = off;   off = align_up(off + (size_t)S * d_seq, kAlign);
    const size_t oG = off;   off = align_up(off + (size_t)S * d_seq, kAlign);
    const size_t oX = off;   off = align_up(off + (size_t)S * k * 4, kAlign);
    const size_t oU = off;   off = align_up(off + (size_t)S * (k + 1) * 4, kAlign);
    const size_t oN = off;   off = align_up(off + (size_t)S * 4, kAlign);
    const size_t oTok = off; off = align_up(off + (size_t)S * (k + 1) * 4, kAlign);
    const size_t oL = off;   off = align_up(off + (size_t)S * k * 4, kAlign);
    const size_t oA = off;   off = align_up(off + (size_t)S * k * 4, kAlign);
    const size_t oS = off;   off = align_up(off + (size_t)S * 4, kAlign);
    const size_t oW = off;   off = align_up(off + L.total, kAlign);
    const size_t arena = off;

    if (!d->s_h2d) {
        SD_CUDA(cudaStreamCreateWithFlags(&d->s_h2d, cudaStreamNonBlocking));
        SD_CUDA(cudaStreamCreateWithFlags(&d->s_comp, cudaStreamNonBlocking));
        SD_CUDA(cudaStreamCreateWithFlags(&d->s_d2h, cudaStreamNonBlocking));
    }
    const int nsets = nslices > 1 ? 2 : 1;
    for (int s = 0; s < nsets; ++s) {
        StageSet& st = d->stage[s];
        if (!st.in_ready) {
            SD_CUDA(cudaEventCreateWithFlags(&st.in_ready, cudaEventDisableTiming));
            SD_CUDA(cudaEventCreateWithFlags(&st.comp_done, cudaEventDisableTiming));
            SD_CUDA(cudaEventCreateWithFlags(&st.out_done, cudaEventDisableTiming));
        }
        if (st.bytes < arena) {
            if (st.base) {
                SD_CUDA(cudaDeviceSynchronize());
                SD_CUDA(cudaFree(st.base));
                st.base = nullptr;
                st.bytes = 0;
            }
            SD_CUDA(cudaMalloc(reinterpret_cast<void**>(&st.base), arena));
            st.bytes = arena;
        }
    }

    const unsigned char* hT = static_cast<const unsigned char*>(target_logits);
    const unsigned char* hD = static_cast<const unsigned char*>(draft_logits);
    unsigned char* hG = static_cast<unsigned char*>(out_grad_draft);
    int kernels = 0;
    for (int s = 0; s < nslices; ++s) {
        StageSet& st = d->stage[s % nsets];
        const int b0 = s * S, nb = (B - b0 < S) ? (B - b0) : S;
        unsigned char* a = st.base;
        if (s >= nsets) {
            // the buffer set is free once slice s-2 has been computed and copied out
            SD_CUDA(cudaStreamWaitEvent(d->s_h2d, st.out_done, 0));
        }
        SD_CUDA(cudaMemcpyAsync(a + oT, hT + (size_t)b0 * t_seq, (size_t)nb * t_seq, cudaMemcpyHostToDevice, d->s_h2d));
        SD_CUDA(cudaMemcpyAsync(a + oD, hD + (size_t)b0 * d_seq, (size_t)nb * d_seq, cudaMemcpyHostToDevice, d->s_h2d));
        SD_CUDA(cudaMemcpyAsync(a + oX, draft_tokens + (size_t)b0 * k, (size_t)nb * k * 4, cudaMemcpyHostToDevice, d->s_h2d));
        SD_CUDA(cudaMemcpyAsync(a + oU, uniforms + (size_t)b0 * (k + 1), (size_t)nb * (k + 1) * 4, cudaMemcpyHostToDevice, d->s_h2d));
        SD_CUDA(cudaEventRecord(st.in_ready, d->s_h2d));
        SD_CUDA(cudaStreamWaitEvent(d->s_comp, st.in_ready, 0));
        const WorkspaceLayout Ls = workspace_layout(nb, k, V, dtype);
        rc = run_device(*d, a + oT, a + oD, reinterpret_cast<int32_t*>(a + oX), reinterpret_cast<float*>(a + oU),
                        temperature, nb, k, V, dtype, reinterpret_cast<int32_t*>(a + oN),
                        reinterpret_cast<int32_t*>(a + oTok), out_loss ? reinterpret_cast<float*>(a + oL) : nullptr,
                        out_grad_draft ? a + oG : nullptr, out_acc_prob ? reinterpret_cast<float*>(a + oA) : nullptr,
                        out_status ? reinterpret_cast<uint32_t*>(a + oS) : nullptr, a + oW, Ls, false, d->s_comp);
        if (rc != SD_OK) break;
        kernels += 1;
        SD_CUDA(cudaEventRecord(st.comp_done, d->s_comp));
        SD_CUDA(cudaStreamWaitEvent(d->s_d2h, st.comp_done, 0));
        SD_CUDA(cudaMemcpyAsync(out_accept_len + b0, a + oN, (size_t)nb * 4, cudaMemcpyDeviceToHost, d->s_d2h));
        SD_CUDA(cudaMemcpyAsync(out_tokens + (size_t)b0 * (k + 1), a + oTok, (size_t)nb * (k + 1) * 4, cudaMemcpyDeviceToHost, d->s_d2h));
        if (out_loss)
            SD_CUDA(cudaMemcpyAsync(out_loss + (size_t)b0 * k, a + oL, (size_t)nb * k * 4, cudaMemcpyDeviceToHost, d->s_d2h));
        if (out_grad_draft)
            SD_CUDA(cudaMemcpyAsync(hG + (size_t)b0 * d_seq, a + oG, (size_t)nb * d_seq, cudaMemcpyDeviceToHost, d->s_d2h));
        if (out_acc_prob)
            SD_CUDA(cudaMemcpyAsync(out_acc_prob + (size_t)b0 * k, a + oA, (size_t)nb * k * 4, cudaMemcpyDeviceToHost, d->s_d2h));
        if (out_status)
            SD_CUDA(cudaMemcpyAsync(out_status + b0, a + oS, (size_t)nb * 4, cudaMemcpyDeviceToHost, d->s_d2h));
        SD_CUDA(cudaEventRecord(st.out_done, d->s_d2h));
    }
    cudaError_t e1 = cudaStreamSynchronize(d->s_h2d);
    cudaError_t e2 = cudaStreamSynchronize(d->s_comp);
    cudaError_t e3 = cudaStreamSynchronize(d->s_d2h);
    if (rc != SD_OK) return rc;
    if (e1 != cudaSuccess) return cuda_fail(e1, "cudaStreamSynchronize(h2d)");
    if (e2 != cudaSuccess) return cuda_fail(e2, "cudaStreamSynchronize(compute)");
    if (e3 != cudaSuccess) return cuda_fail(e3, "cudaStreamSynchronize(d2h)");
    tl_info[5] = kernels;
    return SD_OK;
}

// ---- vocabulary-parallel step ------------------------------------------------------------------
namespace {
struct VpLayout { size_t rowc, region_sums, total; int NR; };
VpLayout vp_layout(int B, int k, int Vs, int dtype) {
    VpLayout L;
    const int NV = Vs / vec_elems(dtype);
    L.NR = (NV + kRegionVecs - 1) / kRegionVecs;
    size_t off = 0;
    L.rowc = off;        off = align_up(off + (size_t)B * (k + 1) * sizeof(RowConst), kAlign);
    L.region_sums = off; off = align_up(off + (size_t)B * 2 * L.NR * 4, kAlign);
    L.total = off;
    return L;
}
int vp_check(const void* T, const void* D, const int32_t* x, float tau, int B, int k, int Vs, int v_offset, int V_total,
             int dtype, const void* ws, size_t ws_bytes) {
    if (dtype != SD_DTYPE_F32 && dtype != SD_DTYPE_BF16) return SD_ERR_DTYPE;
    if (!T || !D || !x) return SD_ERR_NULL;
    if (!shape_ok(B, k, Vs) || V_total < Vs || v_offset < 0 || v_offset > V_total - Vs) return SD_ERR_SHAPE;
    if (!(tau > 0.f) || !isfinite(tau)) return SD_ERR_TEMPERATURE;
    if (((size_t)Vs * elem_bytes(dtype)) % 16 != 0 || !aligned(T, 16) || !aligned(D, 16) || !aligned(x, 4)) return SD_ERR_ALIGN;
    if (!ws || !aligned(ws, kAlign) || ws_bytes < vp_layout(B, k, Vs, dtype).total) return SD_ERR_WORKSPACE;
    return SD_OK;
}
VpParams vp_params(const void* T, const void* D, const int32_t* x, const float* u, float tau, int B, int k, int Vs,
                   int v_offset, int V_total, int dtype, int G, int rank, unsigned char* ws) {
    VpParams P;
    memset(&P, 0, sizeof P);
    const VpLayout L = vp_layout(B, k, Vs, dtype);
    P.T = T; P.D = D; P.x = x; P.u = u;
    P.B = B; P.k = k; P.Vs = Vs; P.v_offset = v_offset; P.V_total = V_total;
    P.G = G; P.rank = rank;
    P.c = (float)(1.4426950408889634 / (double)tau);
    P.tau = tau;
    P.inv_tau = 1.0 / (double)tau;
    P.NR = L.NR;
    P.rowc = reinterpret_cast<RowConst*>(ws + L.rowc);
    P.region_sums = reinterpret_cast<float*>(ws + L.region_sums);
    return P;
}
}  // namespace

size_t sd_vp_workspace_bytes(int B, int k, int V_shard, int dtype) {
    if ((dtype != SD_DTYPE_F32 && dtype != SD_DTYPE_BF16) || !shape_ok(B, k, V_shard)) return 0;
    return vp_layout(B, k, V_shard, dtype).total;
}

int sd_vp_partial(const void* target_shard, const void* draft_shard, const int32_t* draft_tokens, float temperature,
                  int B, int k, int V_shard, int v_offset, int V_total, int dtype, void* out_records, void* workspace,
                  size_t workspace_bytes, void* stream) {
    int rc = vp_check(target_shard, draft_shard, draft_tokens, temperature, B, k, V_shard, v_offset, V_total, dtype,
                      workspace, workspace_bytes);
    if (rc != SD_OK) return rc;
    if (!out_records) return SD_ERR_NULL;
    if (!aligned(out_records, 16)) return SD_ERR_ALIGN;
    int dev;
    DeviceState* ds = nullptr;
    rc = current_device(&dev, &ds);
    if (rc != SD_OK) return rc;
    VpParams P = vp_params(target_shard, draft_shard, draft_tokens, nullptr, temperature, B, k, V_shard, v_offset, V_total,
                           dtype, 1, 0, static_cast<unsigned char*>(workspace));
    P.records = static_cast<VpRecord*>(out_records);
    const unsigned units = (unsigned)B * (unsigned)(k + 1);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (dtype == SD_DTYPE_F32) sd_vp_stats_kernel<SD_DTYPE_F32><<<units, kVpThreads, 0, st>>>(P);
    else                       sd_vp_stats_kernel<SD_DTYPE_BF16><<<units, kVpThreads, 0, st>>>(P);
    SD_CUDA(cudaGetLastError());
    tl_info[0] = 6; tl_info[1] = 1; tl_info[2] = kVpThreads; tl_info[3] = 0; tl_info[4] = (int)units; tl_info[5] = 1;
    return SD_OK;
}

int sd_vp_finish(const void* target_shard, const void* draft_shard, const int32_t* draft_tokens, const float* uniforms,
                 float temperature, int B, int k, int V_shard, int v_offset, int V_total, int dtype,
                 const void* all_records, int n_ranks, int rank, int32_t* out_accept_len, float* out_loss,
                 void* out_grad_shard, double* out_local_mass, uint32_t* out_status, void* workspace,
                 size_t workspace_bytes, void* stream) {
    int rc = vp_check(target_shard, draft_shard, draft_tokens, temperature, B, k, V_shard, v_offset, V_total, dtype,
                      workspace, workspace_bytes);
    if (rc != SD_OK) return rc;
    if (!uniforms || !all_records || !out_accept_len || !out_local_mass) return SD_ERR_NULL;
    if (n_ranks < 1 || rank < 0 || rank >= n_ranks) return SD_ERR_SHAPE;
    if (!aligned(all_records, 16) || !aligned(uniforms, 4) || !aligned(out_accept_len, 4) || !aligned(out_local_mass, 8) ||
        (out_loss && !aligned(out_loss, 4)) || (out_grad_shard && !aligned(out_grad_shard, 16)) ||
        (out_status && !aligned(out_status, 4)))
        return SD_ERR_ALIGN;
    int dev;
    DeviceState* ds = nullptr;
    rc = current_device(&dev, &ds);
    if (rc != SD_OK) return rc;
    VpParams P = vp_params(target_shard, draft_shard, draft_tokens, uniforms, temperature, B, k, V_shard, v_offset, V_total,
                           dtype, n_ranks, rank, static_cast<unsigned char*>(workspace));
    P.all = static_cast<const VpRecord*>(all_records);
    P.accept_len = out_accept_len;
    P.loss = out_loss;
    P.grad = out_grad_shard;
    P.status = out_status;
    P.local_mass = out_local_mass;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    sd_vp_rows_kernel<<<(unsigned)B, 96, 0, st>>>(P);
    const int slices = (P.NR + kVpSliceRegions - 1) / kVpSliceRegions;
    const unsigned grid = (unsigned)B * (unsigned)(k + 1) * (unsigned)slices;
    if (dtype == SD_DTYPE_F32) sd_vp_grad_kernel<SD_DTYPE_F32><<<grid, kVpThreads, 0, st>>>(P, slices);
    else                       sd_vp_grad_kernel<SD_DTYPE_BF16><<<grid, kVpThreads, 0, st>>>(P, slices);
    sd_vp_mass_kernel<<<(unsigned)B, 32, 0, st>>>(P);
    SD_CUDA(cudaGetLastError());
    tl_info[0] = 6; tl_info[1] = 1; tl_info[2] = kVpThreads; tl_info[3] = 0; tl_info[4] = (int)grid; tl_info[5] = 3;
    return SD_OK;
}

int sd_vp_draw(const void* target_shard, const void* draft_shard, const int32_t* draft_tokens, const float* uniforms,
               float temperature, int B, int k, int V_shard, int v_offset, int V_total, int dtype,
               const int32_t* accept_len, const double* all_masses, int n_ranks, int rank, int32_t* out_tokens,
               uint32_t* out_status, void* workspace, size_t workspace_bytes, void* stream) {
    int rc = vp_check(target_shard, draft_shard, draft_tokens, temperature, B, k, V_shard, v_offset, V_total, dtype,
                      workspace, workspace_bytes);
    if (rc != SD_OK) return rc;
    if (!uniforms || !accept_len || !all_masses || !out_tokens) return SD_ERR_NULL;
    if (n_ranks < 1 || rank < 0 || rank >= n_ranks) return SD_ERR_SHAPE;
    if (!aligned(all_masses, 8) || !aligned(out_tokens, 4) || !aligned(accept_len, 4) || (out_status && !aligned(out_status, 4)))
        return SD_ERR_ALIGN;
    int dev;
    DeviceState* ds = nullptr;
    rc = current_device(&dev, &ds);
    if (rc != SD_OK) return rc;
    VpParams P = vp_params(target_shard, draft_shard, draft_tokens, uniforms, temperature, B, k, V_shard, v_offset, V_total,
                           dtype, n_ranks, rank, static_cast<unsigned char*>(workspace));
    P.accept_len = const_cast<int32_t*>(accept_len);
    P.all_mass = all_masses;
    P.tokens = out_tokens;
    P.status = out_status;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (dtype == SD_DTYPE_F32) sd_vp_draw_kernel<SD_DTYPE_F32><<<(unsigned)B, 32, 0, st>>>(P);
    else                       sd_vp_draw_kernel<SD_DTYPE_BF16><<<(unsigned)B, 32, 0, st>>>(P);
    SD_CUDA(cudaGetLastError());
    tl_info[0] = 6; tl_info[5] = 1;
    return SD_OK;
}

// ---- the output layer's gradient ----------------------------------------------------------------
int sd_lmhead_grad(const uint16_t* grad_logits, const uint16_t* hidden, int R, int V, int d, float* out_dW,
                   uint32_t* out_status, void* stream) {
    if (!grad_logits || !hidden || !out_dW) return SD_ERR_NULL;
    if (R < 1 || V < 1 || d < 1 || (long double)V * d >= 4.0e18L) return SD_ERR_SHAPE;
    if (V % 8 != 0 || d % 8 != 0) return SD_ERR_ALIGN;            // rows of whole 16-byte vectors (TMA strides)
    if (!aligned(grad_logits, 16) || !aligned(hidden, 16) || !aligned(out_dW, 16) || (out_status && !aligned(out_status, 4)))
        return SD_ERR_ALIGN;
    int dev;
    DeviceState* ds = nullptr;
    int rc = current_device(&dev, &ds);
    if (rc != SD_OK) return rc;
    std::lock_guard<std::mutex> lock(ds->mu);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!ds->gemm_error) SD_CUDA(cudaMalloc(reinterpret_cast<void**>(&ds->gemm_error), 256));
    uint32_t* err = out_status ? out_status : ds->gemm_error;
    SD_CUDA(cudaMemsetAsync(err, 0, 4, st));
    CUtensorMap map_g, map_x;
    rc = bf16_matrix_map(&map_g, grad_logits, R, V, kGemmBK);
    if (rc != SD_OK) return rc;
    rc = bf16_matrix_map(&map_x, hidden, R, d, kGemmBK);
    if (rc != SD_OK) return rc;
    if (!ds->gemm_attr) {
        SD_CUDA(cudaFuncSetAttribute(sd_lmhead_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmem));
        ds->gemm_attr = true;
    }
    GemmParams P;
    P.R = R; P.V = V; P.d = d;
    P.out = out_dW;
    P.error = err;
    const long long tiles = (long long)((V + kGemmBM - 1) / kGemmBM) * ((d + kGemmBN - 1) / kGemmBN);
    const unsigned grid = (unsigned)(tiles < ds->sm_count ? tiles : ds->sm_count);
    sd_lmhead_kernel<<<grid, kGemmThreads, kGemmSmem, st>>>(map_g, map_x, P);
    SD_CUDA(cudaGetLastError());
    tl_info[0] = 5; tl_info[1] = 1; tl_info[2] = kGemmThreads; tl_info[3] = kGemmSmem; tl_info[4] = (int)grid; tl_info[5] = 1;
    return SD_OK;
}

int sd_set_option(int option_id, long long value) {
    if (option_id < 0 || option_id >= SD_OPT_COUNT) return SD_ERR_SHAPE;
    init_options();
    std::lock_guard<std::mutex> lock(g_opt_mu);
    g_opt.v[option_id] = value;
    return SD_OK;
}

long long sd_get_option(int option_id) {
    if (option_id < 0 || option_id >= SD_OPT_COUNT) return -1;
    return option(option_id);
}

void sd_launch_info(int* path, int* cluster_size, int* threads, int* smem_bytes, int* blocks, int* kernels) {
    if (path) *path = tl_info[0];
    if (cluster_size) *cluster_size = tl_info[1];
    if (threads) *threads = tl_info[2];
    if (smem_bytes) *smem_bytes = tl_info[3];
    if (blocks) *blocks = tl_info[4];
    if (kernels) *kernels = tl_info[5];
}

void sd_release_cached_buffers(void) {
    for (int i = 0; i < kMaxDevices; ++i) {
        DeviceState& d = g_dev[i];
        std::lock_guard<std::mutex> lock(d.mu);
        if (!d.probed || (!d.ws && !d.gemm_error && !d.stage[0].base && !d.stage[1].base)) continue;
        int prev = -1;
        if (cudaGetDevice(&prev) != cudaSuccess) continue;
        if (cudaSetDevice(i) != cudaSuccess) continue;
        cudaDeviceSynchronize();
        if (d.ws) { cudaFree(d.ws); d.ws = nullptr; d.ws_bytes = 0; d.ws_zero_bytes = 0; }
        if (d.gemm_error) { cudaFree(d.gemm_error); d.gemm_error = nullptr; }
        for (StageSet& st : d.stage)
            if (st.base) { cudaFree(st.base); st.base = nullptr; st.bytes = 0; }
        cudaSetDevice(prev);
    }
}

const char* sd_strerror(int code) {
    switch (code) {
        case SD_OK: return "ok";
        case SD_ERR_NULL: return "a required pointer is NULL";
        case SD_ERR_SHAPE: return "B, k or V out of range";
        case SD_ERR_TEMPERATURE: return "temperature must be a finite number > 0";
        case SD_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case SD_ERR_DTYPE: return "unknown dtype";
        case SD_ERR_CUDA: return "a CUDA call failed (see sd_last_cuda_error)";
        case SD_ERR_NO_DEVICE: return "no current CUDA device of compute capability 10.x";
        case SD_ERR_ALIGN: return "a pointer is not aligned to its element type";
        default: return "unknown error code";
    }
}

const char* sd_last_cuda_error(void) { return tl_cuda_error; }

int sd_bounds_report(unsigned long long* out4) {
    if (!out4) return SD_ERR_NULL;
#ifdef SD_BOUNDS_CHECK
    int dev;
    DeviceState* ds = nullptr;
    int rc = current_device(&dev, &ds);
    if (rc != SD_OK) return rc;
    SD_CUDA(cudaDeviceSynchronize());
    SD_CUDA(cudaMemcpyFromSymbol(out4, g_sd_bounds, 4 * sizeof(unsigned long long)));
    const unsigned long long zero[4] = {0, 0, 0, 0};
    SD_CUDA(cudaMemcpyToSymbol(g_sd_bounds, zero, sizeof zero));
    return SD_OK;
#else
    out4[0] = ~0ull;
    out4[1] = out4[2] = out4[3] = 0;
    return SD_OK;
#endif
}

int sd_version(void) { return SD_VERSION; }

}  // extern "C"
