// SVIP speculative-decoding epilogues for sm_100a: the host side and the C ABI (see include/svip.h).
//
// The kernels live in the headers included below:
//   svip_device.cuh    the streaming core: row geometry, cp.async ring, online reduction, warp / block
//                      scans, picking the segment that holds a sample
//   svip_draft.cuh     draft_step_kernel (Algorithm 1 inner loop + Eq. 7) and row_stats_kernel (softmax
//                      normalisers or argmax of target rows; of draft rows when the caller has no q_stats)
//   svip_verify.cuh    verify_finish_kernel (Algorithms 2 and 4 + the loop of Algorithm 1: ratio tests by
//                      one warp, first rejection, residual or bonus token) and verify_greedy_kernel
//                      (Algorithms 3 and 5)
//   svip_analysis.cuh  pair_stats_kernel (Eq. 1-6)
//   svip_policy.cuh    vocabulary-parallel combine, draft-length policies, ragged packing
//   svip_select.cuh    row_threshold_kernel (top-k / nucleus truncation)
//   svip_tree.cuh      verify_tree_kernel (several candidates per position: recursive rejection sampling)
#include "svip_device.cuh"

#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <mutex>
#include <new>

#include "svip.h"

#include "svip_draft.cuh"
#include "svip_verify.cuh"
#include "svip_analysis.cuh"
#include "svip_policy.cuh"

#include "svip_select.cuh"
#include "svip_tree.cuh"

// ==================================================================== host side / C ABI

// -DSVIP_NVTX: a named range around every entry point's host work, for timelines.
#ifdef SVIP_NVTX
#include <nvtx3/nvToolsExt.h>
namespace {
struct NvtxRange {
    explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
};
}  // namespace
#define SVIP_RANGE(name) NvtxRange svip_nvtx_range_(name)
#else
#define SVIP_RANGE(name) do { } while (0)
#endif

using namespace svip;

struct svip_ctx {
    int device;
    int max_rows;
    int num_sms;
    int cluster_override;
    long launches;
    int last_cuda;
    int capturing;
    float2* p_stats;
    float2* q_stats;
    int32_t* p_argmax;
    unsigned* status;
    int* loop_iter;            // device: iteration counter of the drafting loop being replayed
    cudaStream_t loop_stream;  // records the body of a drafting loop
    int loop_open;             // a loop body is being recorded
    int loop_decided;          // the body already holds the kernel that decides the loop
    int loop_failed;           // a loop of the graph being recorded is not closed properly
    LoopCtl loop;
    const int32_t* loop_n_active;
    int profiling;
    int prof_used;
    cudaEvent_t* prof_start;
    cudaEvent_t* prof_stop;
};

constexpr int kProfilePairs = 4096;

struct svip_graph {
    cudaGraphExec_t exec;
    cudaGraph_t graph;
};

namespace {

// SVIP_NO_PDL=1 in the environment launches every kernel fully serialized (for A/B timing).
const bool g_use_pdl = [] {
    const char* v = std::getenv("SVIP_NO_PDL");
    return !(v && v[0] == '1');
}();

// Set while the calling thread records the body of a drafting loop: kernels inside a conditional
// node are launched without the programmatic-serialization attribute.
thread_local bool t_plain_launches = false;

int cuda_fail(svip_ctx* ctx, cudaError_t e) {
    if (ctx) ctx->last_cuda = static_cast<int>(e);
    return SVIP_ERR_CUDA;
}

// Every kernel goes through here: optional cluster dimension, dynamic shared memory, and the
// programmatic-serialization attribute that lets the kernel be scheduled while its predecessor in
// the stream drains (the kernels wait for the predecessor themselves, see pdl_wait()).
template <class... KArgs, class... Args>
cudaError_t launch_ex(void (*kernel)(KArgs...), unsigned grid, unsigned block, int S, size_t dyn_smem,
                      cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(block, 1, 1);
    cfg.dynamicSmemBytes = dyn_smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n = 0;
    if (S > 0) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = S;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    if (g_use_pdl && !t_plain_launches) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

template <class Args>
cudaError_t launch_clustered(void (*kernel)(Args), long units, int S, const Args& args, cudaStream_t st,
                             size_t dyn_smem) {
    return launch_ex(kernel, static_cast<unsigned>(units * S), kThreads, S, dyn_smem, st, args);
}

// Blocks per row.  Small launches are latency-bound: spread a row over as many blocks (1..8, any
// size) as still lets the whole grid sit on the GPU at once (two blocks per SM) while every thread
// keeps a vector; a second wave of clusters would double the time of such a launch.
int pick_cluster(const svip_ctx* ctx, long rows, int V, int dtype) {
    if (ctx->cluster_override > 0) return ctx->cluster_override;
    long nvec = (static_cast<long>(V) * (dtype == SVIP_BF16 ? 2 : 4) + 15) / 16;
    // measured: grids up to about 7/4 blocks per SM run as one wave next to the blocks of the
    // following launch that programmatic launch makes resident early; fuller grids run as two
    long by_grid = rows > 0 ? (7L * ctx->num_sms / 4) / rows : kMaxCluster;
    long by_work = nvec / kThreads;
    long S = by_grid < by_work ? by_grid : by_work;
    if (S > kMaxCluster) S = kMaxCluster;
    if (S < 1) S = 1;
    // measured: clusters of 5 and 7 blocks are placed badly (48 rows of 304 KB: 11.4 us with 5 blocks per row,
    // 9.8 with 4); the next smaller even size is used instead
    if (S == 5 || S == 7) S -= 1;
    // many long rows (more than a wave of blocks anyway): rows above 512 KB are cut so that the
    // two blocks of an SM finish close together (measured on 256 x 1 MB: 64 -> 55 us)
    const long row_bytes = nvec * 16;
    if (S == 1 && rows > ctx->num_sms && row_bytes > (512L << 10)) {
        S = (row_bytes + (512L << 10) - 1) / (512L << 10);
        if (S > 4) S = 4;
    }
    return static_cast<int>(S);
}

// Bytes from the start of the first row to the end of the last one.
[[maybe_unused]] size_t rows_extent(long n_rows, long row_stride, int V, size_t esz) {
    if (n_rows < 1) return 0;
    return (static_cast<size_t>(n_rows - 1) * static_cast<size_t>(row_stride) + static_cast<size_t>(V)) * esz;
}

// -DSVIP_DEBUG_BOUNDS: the extents of the (up to two) logits buffers of a call go into constant memory
// ahead of its kernels, which then refuse loads outside them (see debug_ok).  The vector loads start at the
// 16-byte boundary below a row and end at the one above it, hence the rounding.
#ifdef SVIP_DEBUG_BOUNDS
cudaError_t debug_ranges(const svip_ctx* ctx, cudaStream_t st, const void* p0, size_t bytes0, const void* p1 = nullptr,
                         size_t bytes1 = 0) {
    DebugRange r[2];
    const void* p[2] = {p0, p1};
    const size_t n[2] = {bytes0, bytes1};
    for (int i = 0; i < 2; ++i) {
        const unsigned long long a = reinterpret_cast<unsigned long long>(p[i]);
        r[i].lo = p[i] ? (a & ~15ull) : 0;
        r[i].hi = p[i] ? ((a + n[i] + 15ull) & ~15ull) : 0;
        if (p[i] && n[i] == ~static_cast<size_t>(0)) { r[i].lo = 0; r[i].hi = ~0ull; }   // extent not known
    }
    if (ctx->capturing) { r[0].lo = 0; r[0].hi = ~0ull; }   // no copies from host memory into a graph
    if (ctx->capturing) return cudaSuccess;
    return cudaMemcpyToSymbolAsync(g_debug_range, r, sizeof r, 0, cudaMemcpyHostToDevice, st);
}
#define SVIP_DEBUG_RANGES(...) do { if (debug_ranges(__VA_ARGS__) != cudaSuccess) return SVIP_ERR_CUDA; } while (0)
#else
#define SVIP_DEBUG_RANGES(...) do { } while (0)
#endif

// The candidate path of the threshold kernel reads every row twice.  A launch that fits in L2 finds its rows
// there the second time; a larger one takes its first bound from the first half of every warp segment instead
// of all of it (measured on 256 x 256000 fp32 rows, top-k 50: a half or a third 86 us per launch, all 97, a
// quarter 102 and an eighth 144, because the looser bound lets more candidates in than the counting finish holds).
int threshold_sample_den(long rows, int V, int dtype) {
    const long bytes = rows * static_cast<long>(V) * (dtype == SVIP_BF16 ? 2 : 4);
    return bytes > (48L << 20) ? 2 : 1;
}

bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

float scale_for(float T) { return static_cast<float>(1.4426950408889634 / (T > 0.f ? static_cast<double>(T) : 1.0)); }

}  // namespace

extern "C" {

const char* svip_strerror(int status) {
    switch (status) {
        case SVIP_OK: return "ok";
        case SVIP_ERR_INVALID_ARG: return "invalid argument";
        case SVIP_ERR_UNSUPPORTED: return "unsupported dtype or device";
        case SVIP_ERR_WORKSPACE: return "more rows than the context's workspace holds";
        case SVIP_ERR_CUDA: return "CUDA runtime error";
        case SVIP_ERR_STATE: return "call not valid in the context's current state";
        default: return "unknown status";
    }
}

int svip_version(void) { return 200; }

int svip_last_cuda_error(const svip_ctx* ctx) { return ctx ? ctx->last_cuda : 0; }

int svip_create(svip_ctx** out, int device, int max_rows) {
    if (!out || max_rows < 1 || device < 0) return SVIP_ERR_INVALID_ARG;
    int prev = 0;
    if (cudaGetDevice(&prev) != cudaSuccess) { cudaGetLastError(); return SVIP_ERR_CUDA; }
    if (cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return SVIP_ERR_CUDA; }
    int rc = SVIP_OK;
    svip_ctx* c = new (std::nothrow) svip_ctx();
    if (!c) { cudaSetDevice(prev); return SVIP_ERR_CUDA; }
    c->device = device;
    c->max_rows = max_rows;
    int major = 0, sms = 0;
    cudaError_t e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
    if (e != cudaSuccess) rc = SVIP_ERR_CUDA;
    else if (major != 10) rc = SVIP_ERR_UNSUPPORTED;
    c->num_sms = sms;
    if (rc == SVIP_OK) {
        // the cp.async rings need more dynamic shared memory than the default limit
        const void* ringed[] = {
            (const void*)draft_step_kernel<kBF16, true, 2>, (const void*)draft_step_kernel<kBF16, false, 2>,
            (const void*)draft_step_kernel<kF32, true, 2>,  (const void*)draft_step_kernel<kF32, false, 2>,
            (const void*)draft_step_kernel<kBF16, true, 3>, (const void*)draft_step_kernel<kBF16, false, 3>,
            (const void*)draft_step_kernel<kF32, true, 3>,  (const void*)draft_step_kernel<kF32, false, 3>,
            (const void*)draft_step_kernel<kBF16, true, 2, true>, (const void*)draft_step_kernel<kBF16, false, 2, true>,
            (const void*)draft_step_kernel<kF32, true, 2, true>,  (const void*)draft_step_kernel<kF32, false, 2, true>,
            (const void*)row_stats_kernel<kBF16, 0>,     (const void*)row_stats_kernel<kBF16, 1>,
            (const void*)row_stats_kernel<kF32, 0>,      (const void*)row_stats_kernel<kF32, 1>,
            (const void*)verify_finish_kernel<kBF16>,    (const void*)verify_finish_kernel<kF32>,
            (const void*)row_stats_kernel<kBF16, 2>,     (const void*)row_stats_kernel<kF32, 2>,
            (const void*)row_threshold_kernel<kBF16>,    (const void*)row_threshold_kernel<kF32>,
            (const void*)row_threshold_kernel<kBF16, true>, (const void*)row_threshold_kernel<kF32, true>,
            (const void*)draft_step_kernel<kBF16, false, 2, false, true>, (const void*)draft_step_kernel<kF32, false, 2, false, true>,
            (const void*)row_stats_kernel<kBF16, 1, true>, (const void*)row_stats_kernel<kF32, 1, true>,
            (const void*)verify_finish_kernel<kBF16, true>, (const void*)verify_finish_kernel<kF32, true>,
            (const void*)pair_stats_kernel<kBF16>, (const void*)pair_stats_kernel<kF32>,
            (const void*)pair_stats_kernel<kBF16, true>, (const void*)pair_stats_kernel<kF32, true>,
            (const void*)verify_scan_kernel<kBF16, false>, (const void*)verify_scan_kernel<kF32, false>,
            (const void*)verify_scan_kernel<kBF16, true>, (const void*)verify_scan_kernel<kF32, true>};
        for (const void* k : ringed)
            if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, kRingBytes) != cudaSuccess)
                rc = SVIP_ERR_CUDA;
    }
    if (rc == SVIP_OK) {
        size_t n = static_cast<size_t>(max_rows);
        if (cudaMalloc(&c->p_stats, n * sizeof(float2)) != cudaSuccess ||
            cudaMalloc(&c->q_stats, n * sizeof(float2)) != cudaSuccess ||
            cudaMalloc(&c->p_argmax, n * sizeof(int32_t)) != cudaSuccess ||
            cudaMalloc(&c->status, sizeof(unsigned)) != cudaSuccess ||
            cudaMemset(c->status, 0, sizeof(unsigned)) != cudaSuccess ||
            cudaMalloc(&c->loop_iter, sizeof(int)) != cudaSuccess ||
            cudaMemset(c->loop_iter, 0, sizeof(int)) != cudaSuccess) {
            rc = SVIP_ERR_CUDA;
        }
    }
    if (rc != SVIP_OK) {
        cudaGetLastError();
        cudaFree(c->p_stats); cudaFree(c->q_stats); cudaFree(c->p_argmax); cudaFree(c->status);
        cudaFree(c->loop_iter);
        delete c;
    } else {
        *out = c;
    }
    cudaSetDevice(prev);
    return rc;
}

int svip_destroy(svip_ctx* ctx) {
    if (!ctx) return SVIP_ERR_INVALID_ARG;
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(ctx->device);
    cudaFree(ctx->p_stats); cudaFree(ctx->q_stats); cudaFree(ctx->p_argmax); cudaFree(ctx->status);
    cudaFree(ctx->loop_iter);
    if (ctx->loop_stream) cudaStreamDestroy(ctx->loop_stream);
    if (ctx->prof_start) {
        for (int k = 0; k < kProfilePairs; ++k) {
            cudaEventDestroy(ctx->prof_start[k]);
            cudaEventDestroy(ctx->prof_stop[k]);
        }
        delete[] ctx->prof_start;
        delete[] ctx->prof_stop;
    }
    cudaSetDevice(prev);
    delete ctx;
    return SVIP_OK;
}

int svip_set_cluster_size(svip_ctx* ctx, int cluster_size) {
    if (!ctx) return SVIP_ERR_INVALID_ARG;
    if (cluster_size < 0 || cluster_size > kMaxCluster) return SVIP_ERR_INVALID_ARG;
    ctx->cluster_override = cluster_size;
    return SVIP_OK;
}

long svip_launch_count(const svip_ctx* ctx) { return ctx ? ctx->launches : 0; }

int svip_read_status(svip_ctx* ctx, unsigned* flags, void* stream) {
    if (!ctx || !flags) return SVIP_ERR_INVALID_ARG;
    if (ctx->capturing) return SVIP_ERR_STATE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned v = 0;
    cudaError_t e = cudaMemcpyAsync(&v, ctx->status, sizeof v, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->status, 0, sizeof v, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
#ifdef SVIP_DEBUG_BOUNDS
    unsigned oob = 0, zero = 0;
    e = cudaMemcpyFromSymbol(&oob, g_debug_oob, sizeof oob);
    if (e == cudaSuccess) e = cudaMemcpyToSymbol(g_debug_oob, &zero, sizeof zero);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    if (oob) v |= SVIP_STATUS_DEBUG_OOB;
#endif
    *flags = v;
    return SVIP_OK;
}

static int draft_impl(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V, long row_stride,
                      long pos_stride, const int32_t* pos, long slot_stride, float T, float thresh,
                      const float* uniforms, const uint8_t* active, const float* thr, int32_t* token,
                      float* entropy, uint8_t* stop, float* row_stats, void* stream);

int svip_draft_step(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V, long row_stride,
                    float T, float thresh, const float* uniforms, int32_t* token, float* entropy,
                    uint8_t* stop, float* row_stats, void* stream) {
    return svip_draft_step_masked(ctx, logits, dtype, B, V, row_stride, T, thresh, uniforms, nullptr, token,
                                  entropy, stop, row_stats, stream);
}

int svip_draft_step_masked(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V, long row_stride,
                           float T, float thresh, const float* uniforms, const uint8_t* active,
                           int32_t* token, float* entropy, uint8_t* stop, float* row_stats, void* stream) {
    return svip_draft_step_at(ctx, logits, dtype, B, V, row_stride, 0, nullptr, 0, T, thresh, uniforms, active,
                              token, entropy, stop, row_stats, stream);
}

int svip_draft_step_at(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V, long row_stride,
                       long pos_stride, const int32_t* pos, long slot_stride, float T, float thresh,
                       const float* uniforms, const uint8_t* active, int32_t* token, float* entropy,
                       uint8_t* stop, float* row_stats, void* stream) {
    return draft_impl(ctx, logits, dtype, B, V, row_stride, pos_stride, pos, slot_stride, T, thresh, uniforms, active,
                      nullptr, token, entropy, stop, row_stats, stream);
}

int svip_draft_step_filtered(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V, long row_stride,
                             float T, float thresh, const float* uniforms, const uint8_t* active, const float* thr,
                             int32_t* token, float* entropy, uint8_t* stop, float* row_stats, void* stream) {
    if (!thr || !(T > 0.f)) return SVIP_ERR_INVALID_ARG;
    return draft_impl(ctx, logits, dtype, B, V, row_stride, 0, nullptr, 0, T, thresh, uniforms, active, thr, token,
                      entropy, stop, row_stats, stream);
}

static int draft_impl(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V, long row_stride,
                      long pos_stride, const int32_t* pos, long slot_stride, float T, float thresh,
                      const float* uniforms, const uint8_t* active, const float* thr, int32_t* token,
                      float* entropy, uint8_t* stop, float* row_stats, void* stream) {
    if (!ctx || !logits || !token || !entropy || !stop) return SVIP_ERR_INVALID_ARG;
    if (pos_stride < 0 || slot_stride < 0) return SVIP_ERR_INVALID_ARG;
    if (dtype != SVIP_F32 && dtype != SVIP_BF16) return SVIP_ERR_UNSUPPORTED;
    if (B < 0 || V < 1 || V > 0x7fffffe0 || row_stride < 0) return SVIP_ERR_INVALID_ARG;
    if (!(T >= 0.f) || std::isinf(T) || std::isnan(thresh)) return SVIP_ERR_INVALID_ARG;
    if (T > 0.f && !uniforms) return SVIP_ERR_INVALID_ARG;
    if (!aligned_to(logits, dtype == SVIP_BF16 ? 2 : 4)) return SVIP_ERR_INVALID_ARG;
    if (B == 0) return SVIP_OK;
    SVIP_RANGE("svip_draft_step");
    SVIP_DEBUG_RANGES(ctx, static_cast<cudaStream_t>(stream), logits,
                      pos ? ~static_cast<size_t>(0) : rows_extent(B, row_stride, V, dtype == SVIP_BF16 ? 2 : 4));
    DraftArgs a;
    a.logits = logits; a.row_stride = row_stride; a.V = V; a.c = scale_for(T); a.thresh = thresh;
    a.greedy = T > 0.f ? 0 : 1; a.uniforms = uniforms; a.token = token; a.entropy = entropy;
    a.stop = stop; a.row_stats = row_stats; a.status = ctx->status; a.active = active;
    a.ext_target = nullptr; a.token_offset = 0;
    a.pos = pos; a.pos_stride = pos_stride; a.slot_stride = slot_stride; a.thr = thr;
    int S = pick_cluster(ctx, B, V, dtype);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool waves = static_cast<long>(B) * S > 2L * ctx->num_sms;
    void (*k)(DraftArgs);
    if (dtype == SVIP_BF16)
        k = a.greedy ? (waves ? draft_step_kernel<kBF16, true, 3> : draft_step_kernel<kBF16, true, 2>)
                     : (waves ? draft_step_kernel<kBF16, false, 3> : draft_step_kernel<kBF16, false, 2>);
    else
        k = a.greedy ? (waves ? draft_step_kernel<kF32, true, 3> : draft_step_kernel<kF32, true, 2>)
                     : (waves ? draft_step_kernel<kF32, false, 3> : draft_step_kernel<kF32, false, 2>);
    if (pos) {
        if (dtype == SVIP_BF16) k = a.greedy ? draft_step_kernel<kBF16, true, 2, true> : draft_step_kernel<kBF16, false, 2, true>;
        else k = a.greedy ? draft_step_kernel<kF32, true, 2, true> : draft_step_kernel<kF32, false, 2, true>;
    }
    if (thr) k = dtype == SVIP_BF16 ? draft_step_kernel<kBF16, false, 2, false, true> : draft_step_kernel<kF32, false, 2, false, true>;
    cudaError_t e = launch_clustered(k, B, S, a, st, kRingBytes);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return SVIP_OK;
}

int svip_row_threshold(svip_ctx* ctx, const void* logits, svip_dtype dtype, int n_rows, int V, long row_stride,
                       float T, int top_k, float top_p, float* thr, float* stats, void* stream) {
    if (!ctx || !logits || !thr) return SVIP_ERR_INVALID_ARG;
    if (dtype != SVIP_F32 && dtype != SVIP_BF16) return SVIP_ERR_UNSUPPORTED;
    if (n_rows < 0 || V < 1 || V > 0x7fffffe0 || row_stride < 0 || top_k < 0) return SVIP_ERR_INVALID_ARG;
    if (!(T > 0.f) || std::isinf(T) || !(top_p > 0.f)) return SVIP_ERR_INVALID_ARG;
    if (!aligned_to(logits, dtype == SVIP_BF16 ? 2 : 4)) return SVIP_ERR_INVALID_ARG;
    if (n_rows == 0) return SVIP_OK;
    SVIP_RANGE("svip_row_threshold");
    SVIP_DEBUG_RANGES(ctx, static_cast<cudaStream_t>(stream), logits, rows_extent(n_rows, row_stride, V, dtype == SVIP_BF16 ? 2 : 4));
    ThresholdArgs a;
    a.logits = logits; a.row_stride = row_stride; a.V = V; a.c = scale_for(T);
    a.top_k = (top_k >= 1 && top_k < V) ? top_k : 0; a.top_p = top_p; a.thr = thr;
    a.stats = reinterpret_cast<float2*>(stats);
    if (stats && !aligned_to(stats, 8)) return SVIP_ERR_INVALID_ARG;
    a.uniforms = nullptr; a.active = nullptr; a.thresh = 0.f; a.token = nullptr; a.entropy = nullptr;
    a.stop = nullptr; a.status = ctx->status;
    a.sample_den = threshold_sample_den(n_rows, V, dtype);
    const int S = pick_cluster(ctx, n_rows, V, dtype);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = dtype == SVIP_BF16 ? launch_clustered(row_threshold_kernel<kBF16>, n_rows, S, a, st, kRingBytes)
                                       : launch_clustered(row_threshold_kernel<kF32>, n_rows, S, a, st, kRingBytes);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return SVIP_OK;
}

int svip_draft_step_truncated(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V, long row_stride,
                              float T, float thresh, int top_k, float top_p, const float* uniforms,
                              const uint8_t* active, float* thr, int32_t* token, float* entropy, uint8_t* stop,
                              float* row_stats, void* stream) {
    if (!ctx || !logits || !thr || !token || !entropy || !stop || !uniforms) return SVIP_ERR_INVALID_ARG;
    if (dtype != SVIP_F32 && dtype != SVIP_BF16) return SVIP_ERR_UNSUPPORTED;
    if (B < 0 || V < 1 || V > 0x7fffffe0 || row_stride < 0 || top_k < 0) return SVIP_ERR_INVALID_ARG;
    if (!(T > 0.f) || std::isinf(T) || !(top_p > 0.f) || std::isnan(thresh)) return SVIP_ERR_INVALID_ARG;
    if (!aligned_to(logits, dtype == SVIP_BF16 ? 2 : 4)) return SVIP_ERR_INVALID_ARG;
    if (row_stats && !aligned_to(row_stats, 8)) return SVIP_ERR_INVALID_ARG;
    if (B == 0) return SVIP_OK;
    SVIP_RANGE("svip_draft_step_truncated");
    SVIP_DEBUG_RANGES(ctx, static_cast<cudaStream_t>(stream), logits, rows_extent(B, row_stride, V, dtype == SVIP_BF16 ? 2 : 4));
    ThresholdArgs a;
    a.logits = logits; a.row_stride = row_stride; a.V = V; a.c = scale_for(T);
    a.top_k = (top_k >= 1 && top_k < V) ? top_k : 0; a.top_p = top_p; a.thr = thr;
    a.stats = reinterpret_cast<float2*>(row_stats);
    a.uniforms = uniforms; a.active = active; a.thresh = thresh; a.token = token; a.entropy = entropy;
    a.stop = stop; a.status = ctx->status;
    a.sample_den = threshold_sample_den(B, V, dtype);
    const int S = pick_cluster(ctx, B, V, dtype);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = dtype == SVIP_BF16
        ? launch_clustered(row_threshold_kernel<kBF16, true>, B, S, a, st, kRingBytes)
        : launch_clustered(row_threshold_kernel<kF32, true>, B, S, a, st, kRingBytes);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return SVIP_OK;
}

int svip_pack_ragged(svip_ctx* ctx, const int32_t* draft_len, int B, int K_max, int32_t* cu_rows,
                     int32_t* row_seq, int32_t* row_pos, void* stream) {
    if (!ctx || !draft_len || !cu_rows) return SVIP_ERR_INVALID_ARG;
    if (B < 1 || B > 65536 || K_max < 1) return SVIP_ERR_INVALID_ARG;
    if (static_cast<long>(B) * (static_cast<long>(K_max) + 1) >= 0x7fffffffL) return SVIP_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = launch_ex(pack_ragged_kernel, 1, kPackThreads, 0, 0, st, draft_len, B, K_max, cu_rows, row_seq,
                              row_pos, ctx->status);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return SVIP_OK;
}

// The verification round; q_thr / p_thr are both NULL (plain distributions) or both given
// (distributions truncated at those per-row thresholds).
static int verify_impl(svip_ctx* ctx, const int32_t* draft_tokens, const void* q_logits, long q_row_stride,
                       const float* q_stats, long q_seq_stride, long q_pos_stride, const void* target_logits,
                       long t_row_stride, svip_dtype dtype, const int32_t* cu_rows, int B, int K,
                       int n_target_rows, int V, float T, const float* uniforms, int32_t* n_accepted,
                       int32_t* next_token, void* stream, const float* q_thr, const float* p_thr,
                       const float* p_stats_user, bool early_exit = false) {
    if (!ctx || !draft_tokens || !target_logits || !n_accepted || !next_token) return SVIP_ERR_INVALID_ARG;
    const bool truncated = q_thr != nullptr;
    if (dtype != SVIP_F32 && dtype != SVIP_BF16) return SVIP_ERR_UNSUPPORTED;
    if (B < 0 || K < 1 || V < 1 || V > 0x7fffffe0 || t_row_stride < 0 || q_row_stride < 0) return SVIP_ERR_INVALID_ARG;
    if (!(T >= 0.f) || std::isinf(T)) return SVIP_ERR_INVALID_ARG;
    const bool sampling = T > 0.f;
    if (sampling && (!q_logits || !uniforms)) return SVIP_ERR_INVALID_ARG;
    if (q_seq_stride < 0 && q_seq_stride != SVIP_Q_PACKED) return SVIP_ERR_INVALID_ARG;
    if (q_seq_stride >= 0 && q_pos_stride < 0) return SVIP_ERR_INVALID_ARG;
    const size_t esz = dtype == SVIP_BF16 ? 2 : 4;
    if (!aligned_to(target_logits, esz) || (q_logits && !aligned_to(q_logits, esz))) return SVIP_ERR_INVALID_ARG;
    if (static_cast<long>(B) * (static_cast<long>(K) + 1) >= 0x7fffffffL) return SVIP_ERR_INVALID_ARG;
    if (B == 0) return n_target_rows == 0 ? SVIP_OK : SVIP_ERR_INVALID_ARG;
    if (n_target_rows < 2 * B || n_target_rows > B * (K + 1)) return SVIP_ERR_INVALID_ARG;
    if (!cu_rows && n_target_rows != B * (K + 1)) return SVIP_ERR_INVALID_ARG;
    if (n_target_rows > ctx->max_rows) return SVIP_ERR_WORKSPACE;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const float c = scale_for(T);
    cudaError_t e;
    SVIP_RANGE("svip_verify");
    {
        [[maybe_unused]] const long q_rows =
            q_seq_stride < 0 ? n_target_rows - B : (B - 1) * q_seq_stride + (static_cast<long>(K) - 1) * q_pos_stride + 1;
        SVIP_DEBUG_RANGES(ctx, st, target_logits, rows_extent(n_target_rows, t_row_stride, V, esz), q_logits,
                          rows_extent(q_rows, q_row_stride, V, esz));
    }

    StatsArgs s;
    s.logits = target_logits; s.row_stride = t_row_stride; s.V = V; s.c = c; s.draft_rows = 0; s.K = K;
    s.cu = cu_rows; s.q_seq_stride = q_seq_stride; s.q_pos_stride = q_pos_stride;
    s.out_stats = ctx->p_stats; s.out_argmax = sampling ? nullptr : ctx->p_argmax; s.status = ctx->status;
    s.out_partial = nullptr; s.idx_offset = 0; s.thr = p_thr;
    int S = pick_cluster(ctx, n_target_rows, V, dtype);
    const bool timed = ctx->profiling && !ctx->capturing && ctx->prof_used < kProfilePairs;
    if (early_exit) {
        // the draft rows' normalisers first (the accept test of a position needs them), then one cluster
        // per sequence walks the target rows up to the first rejection
        if (sampling && !q_stats) {
            StatsArgs d = s;
            d.logits = q_logits; d.row_stride = q_row_stride; d.draft_rows = 1;
            d.out_stats = ctx->q_stats; d.out_argmax = nullptr; d.thr = nullptr;
            const int Sd = pick_cluster(ctx, n_target_rows - B, V, dtype);
            e = dtype == SVIP_BF16 ? launch_clustered(row_stats_kernel<kBF16, 1>, static_cast<long>(B) * K, Sd, d, st, kRingBytes)
                                   : launch_clustered(row_stats_kernel<kF32, 1>, static_cast<long>(B) * K, Sd, d, st, kRingBytes);
            if (e != cudaSuccess) return cuda_fail(ctx, e);
            ctx->launches += 1;
        }
        FinishArgs w;
        w.draft_tokens = draft_tokens; w.q_logits = q_logits; w.q_row_stride = q_row_stride;
        w.q_stats_user = reinterpret_cast<const float2*>(q_stats); w.q_stats_ws = ctx->q_stats;
        w.q_seq_stride = q_seq_stride; w.q_pos_stride = q_pos_stride; w.t_logits = target_logits;
        w.t_row_stride = t_row_stride; w.p_stats = ctx->p_stats; w.p_stats_out = ctx->p_stats;
        w.cu = cu_rows; w.K = K; w.V = V; w.c = c;
        w.uniforms = uniforms; w.n_accepted = n_accepted; w.next_token = next_token; w.status = ctx->status;
        w.p_thr = nullptr; w.q_thr = nullptr; w.n_acc_in = nullptr;
        // one cluster per sequence, cut as for the finish kernel (measured on 256 sequences of 1 MB rows: 2 or 4
        // blocks per sequence are equally fast, 8 are slower; on 32 sequences of 304 KB rows 8 are fastest)
        int Sw = pick_cluster(ctx, B, V, dtype);
        if (ctx->cluster_override == 0) {
            const long row_bytes = static_cast<long>(V) * static_cast<long>(esz);
            while (Sw < 4 && 2 * row_bytes / Sw > (512L << 10)) Sw *= 2;
        }
        if (timed) cudaEventRecord(ctx->prof_start[ctx->prof_used], st);
        if (sampling)
            e = dtype == SVIP_BF16 ? launch_clustered(verify_scan_kernel<kBF16, false>, B, Sw, w, st, kRingBytes)
                                   : launch_clustered(verify_scan_kernel<kF32, false>, B, Sw, w, st, kRingBytes);
        else
            e = dtype == SVIP_BF16 ? launch_clustered(verify_scan_kernel<kBF16, true>, B, Sw, w, st, kRingBytes)
                                   : launch_clustered(verify_scan_kernel<kF32, true>, B, Sw, w, st, kRingBytes);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        ctx->launches += 1;
        if (timed) cudaEventRecord(ctx->prof_stop[ctx->prof_used++], st);
        return SVIP_OK;
    } else {
    if (timed) cudaEventRecord(ctx->prof_start[ctx->prof_used], st);
    if (p_stats_user)
        e = cudaSuccess;   // the caller already holds (m, Z) of every target row
    else if (truncated)
        e = dtype == SVIP_BF16 ? launch_clustered(row_stats_kernel<kBF16, 1, true>, n_target_rows, S, s, st, kRingBytes)
                               : launch_clustered(row_stats_kernel<kF32, 1, true>, n_target_rows, S, s, st, kRingBytes);
    else if (sampling)
        e = dtype == SVIP_BF16 ? launch_clustered(row_stats_kernel<kBF16, 1>, n_target_rows, S, s, st, kRingBytes)
                               : launch_clustered(row_stats_kernel<kF32, 1>, n_target_rows, S, s, st, kRingBytes);
    else
        e = dtype == SVIP_BF16 ? launch_clustered(row_stats_kernel<kBF16, 0>, n_target_rows, S, s, st, kRingBytes)
                               : launch_clustered(row_stats_kernel<kF32, 0>, n_target_rows, S, s, st, kRingBytes);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    if (!p_stats_user) ctx->launches += 1;
    if (timed) cudaEventRecord(ctx->prof_stop[ctx->prof_used++], st);

    }
    if (!sampling) {
        GreedyArgs g;
        g.draft_tokens = draft_tokens; g.p_argmax = ctx->p_argmax; g.cu = cu_rows;
        g.q_seq_stride = q_seq_stride; g.q_pos_stride = q_pos_stride; g.B = B; g.K = K;
        g.n_accepted = n_accepted; g.next_token = next_token;
        e = launch_ex(verify_greedy_kernel, static_cast<unsigned>((B + kWarps - 1) / kWarps), kThreads, 0, 0, st, g);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        ctx->launches += 1;
        return SVIP_OK;
    }

    if (!q_stats) {
        StatsArgs d = s;
        d.logits = q_logits; d.row_stride = q_row_stride; d.draft_rows = 1;
        d.out_stats = ctx->q_stats; d.out_argmax = nullptr; d.thr = q_thr;
        long units = static_cast<long>(B) * K;
        int Sd = pick_cluster(ctx, n_target_rows - B, V, dtype);
        if (truncated)
            e = dtype == SVIP_BF16 ? launch_clustered(row_stats_kernel<kBF16, 1, true>, units, Sd, d, st, kRingBytes)
                                   : launch_clustered(row_stats_kernel<kF32, 1, true>, units, Sd, d, st, kRingBytes);
        else
            e = dtype == SVIP_BF16 ? launch_clustered(row_stats_kernel<kBF16, 1>, units, Sd, d, st, kRingBytes)
                                   : launch_clustered(row_stats_kernel<kF32, 1>, units, Sd, d, st, kRingBytes);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        ctx->launches += 1;
    }

    FinishArgs f;
    f.draft_tokens = draft_tokens; f.q_logits = q_logits; f.q_row_stride = q_row_stride;
    f.q_stats_user = reinterpret_cast<const float2*>(q_stats); f.q_stats_ws = ctx->q_stats;
    f.q_seq_stride = q_seq_stride; f.q_pos_stride = q_pos_stride; f.t_logits = target_logits;
    f.t_row_stride = t_row_stride;
    f.p_stats = p_stats_user ? reinterpret_cast<const float2*>(p_stats_user) : ctx->p_stats;
    f.cu = cu_rows; f.K = K; f.V = V; f.c = c;
    f.uniforms = uniforms; f.n_accepted = n_accepted; f.next_token = next_token; f.status = ctx->status;
    f.p_thr = p_thr; f.q_thr = q_thr;
    f.n_acc_in = nullptr; f.p_stats_out = nullptr;
    // up to two rows per sequence are streamed: long rows are cut finer than the one-wave policy
    // asks for (this kernel runs for many microseconds, so several waves are fine)
    int Sf = pick_cluster(ctx, B, V, dtype);
    if (ctx->cluster_override == 0) {
        const long row_bytes = static_cast<long>(V) * static_cast<long>(esz);
        while (Sf < kMaxCluster && 2 * row_bytes / Sf > (512L << 10)) Sf *= 2;
        if (Sf > kMaxCluster) Sf = kMaxCluster;
    }
    if (truncated)
        e = dtype == SVIP_BF16 ? launch_clustered(verify_finish_kernel<kBF16, true>, B, Sf, f, st, kRingBytes)
                               : launch_clustered(verify_finish_kernel<kF32, true>, B, Sf, f, st, kRingBytes);
    else
        e = dtype == SVIP_BF16 ? launch_clustered(verify_finish_kernel<kBF16>, B, Sf, f, st, kRingBytes)
                               : launch_clustered(verify_finish_kernel<kF32>, B, Sf, f, st, kRingBytes);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return SVIP_OK;
}

int svip_verify(svip_ctx* ctx, const int32_t* draft_tokens, const void* q_logits, long q_row_stride,
                const float* q_stats, long q_seq_stride, long q_pos_stride, const void* target_logits,
                long t_row_stride, svip_dtype dtype, const int32_t* cu_rows, int B, int K,
                int n_target_rows, int V, float T, const float* uniforms, int32_t* n_accepted,
                int32_t* next_token, void* stream) {
    return verify_impl(ctx, draft_tokens, q_logits, q_row_stride, q_stats, q_seq_stride, q_pos_stride,
                       target_logits, t_row_stride, dtype, cu_rows, B, K, n_target_rows, V, T, uniforms,
                       n_accepted, next_token, stream, nullptr, nullptr, nullptr);
}

int svip_verify_early_exit(svip_ctx* ctx, const int32_t* draft_tokens, const void* q_logits, long q_row_stride,
                           const float* q_stats, long q_seq_stride, long q_pos_stride, const void* target_logits,
                           long t_row_stride, svip_dtype dtype, const int32_t* cu_rows, int B, int K,
                           int n_target_rows, int V, float T, const float* uniforms, int32_t* n_accepted,
                           int32_t* next_token, void* stream) {
    return verify_impl(ctx, draft_tokens, q_logits, q_row_stride, q_stats, q_seq_stride, q_pos_stride,
                       target_logits, t_row_stride, dtype, cu_rows, B, K, n_target_rows, V, T, uniforms,
                       n_accepted, next_token, stream, nullptr, nullptr, nullptr, true);
}

int svip_verify_filtered(svip_ctx* ctx, const int32_t* draft_tokens, const void* q_logits, long q_row_stride,
                         const float* q_stats, const float* q_thr, long q_seq_stride, long q_pos_stride,
                         const void* target_logits, long t_row_stride, const float* p_thr, const float* p_stats,
                         svip_dtype dtype, const int32_t* cu_rows, int B, int K, int n_target_rows, int V, float T,
                         const float* uniforms, int32_t* n_accepted, int32_t* next_token, void* stream) {
    if (!q_thr || !p_thr || !(T > 0.f)) return SVIP_ERR_INVALID_ARG;
    if (p_stats && !aligned_to(p_stats, 8)) return SVIP_ERR_INVALID_ARG;
    return verify_impl(ctx, draft_tokens, q_logits, q_row_stride, q_stats, q_seq_stride, q_pos_stride,
                       target_logits, t_row_stride, dtype, cu_rows, B, K, n_target_rows, V, T, uniforms,
                       n_accepted, next_token, stream, q_thr, p_thr, p_stats);
}

int svip_profile_enable(svip_ctx* ctx, int on) {
    if (!ctx) return SVIP_ERR_INVALID_ARG;
    if (ctx->capturing) return SVIP_ERR_STATE;
    if (on && !ctx->prof_start) {
        int prev = 0;
        cudaGetDevice(&prev);
        cudaSetDevice(ctx->device);
        ctx->prof_start = new (std::nothrow) cudaEvent_t[kProfilePairs]();
        ctx->prof_stop = new (std::nothrow) cudaEvent_t[kProfilePairs]();
        cudaError_t e = (ctx->prof_start && ctx->prof_stop) ? cudaSuccess : cudaErrorMemoryAllocation;
        for (int k = 0; k < kProfilePairs && e == cudaSuccess; ++k) {
            e = cudaEventCreate(&ctx->prof_start[k]);
            if (e == cudaSuccess) e = cudaEventCreate(&ctx->prof_stop[k]);
        }
        cudaSetDevice(prev);
        if (e != cudaSuccess) {
            delete[] ctx->prof_start; delete[] ctx->prof_stop;   // events created so far leak with the context
            ctx->prof_start = ctx->prof_stop = nullptr;
            return cuda_fail(ctx, e);
        }
    }
    ctx->profiling = on ? 1 : 0;
    ctx->prof_used = 0;
    return SVIP_OK;
}

int svip_profile_read(svip_ctx* ctx, double* total_ms, long* launches) {
    if (!ctx || !total_ms || !launches) return SVIP_ERR_INVALID_ARG;
    if (ctx->capturing) return SVIP_ERR_STATE;
    double sum = 0.0;
    for (int k = 0; k < ctx->prof_used; ++k) {
        cudaError_t e = cudaEventSynchronize(ctx->prof_stop[k]);
        float ms = 0.f;
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, ctx->prof_start[k], ctx->prof_stop[k]);
        if (e != cudaSuccess) { ctx->prof_used = 0; return cuda_fail(ctx, e); }
        sum += ms;
    }
    *total_ms = sum;
    *launches = ctx->prof_used;
    ctx->prof_used = 0;
    return SVIP_OK;
}

int svip_verify_tree(svip_ctx* ctx, const int32_t* tokens, const int32_t* parent, const void* q_logits,
                     long q_row_stride, const float* q_stats, const void* target_logits, long t_row_stride,
                     svip_dtype dtype, int B, int N, int V, float T, const float* uniforms,
                     int32_t* n_accepted, int32_t* path, int32_t* next_token, void* stream) {
    if (!ctx || !tokens || !parent || !target_logits || !n_accepted || !path || !next_token) return SVIP_ERR_INVALID_ARG;
    if (dtype != SVIP_F32 && dtype != SVIP_BF16) return SVIP_ERR_UNSUPPORTED;
    if (B < 0 || N < 1 || V < 1 || V > 0x7fffffe0 || t_row_stride < 0 || q_row_stride < 0) return SVIP_ERR_INVALID_ARG;
    if (!(T >= 0.f) || std::isinf(T)) return SVIP_ERR_INVALID_ARG;
    const bool sampling = T > 0.f;
    if (sampling && (!q_logits || !uniforms)) return SVIP_ERR_INVALID_ARG;
    const size_t esz = dtype == SVIP_BF16 ? 2 : 4;
    if (!aligned_to(target_logits, esz) || (q_logits && !aligned_to(q_logits, esz))) return SVIP_ERR_INVALID_ARG;
    if (q_stats && !aligned_to(q_stats, 8)) return SVIP_ERR_INVALID_ARG;
    if (static_cast<long>(B) * (static_cast<long>(N) + 1) >= 0x7fffffffL) return SVIP_ERR_INVALID_ARG;
    if (B == 0) return SVIP_OK;
    const long n_rows = static_cast<long>(B) * (N + 1);
    if (n_rows > ctx->max_rows) return SVIP_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const float c = scale_for(T);
    cudaError_t e;
    SVIP_RANGE("svip_verify_tree");
    SVIP_DEBUG_RANGES(ctx, st, target_logits, rows_extent(n_rows, t_row_stride, V, esz), q_logits,
                      rows_extent(n_rows, q_row_stride, V, esz));

    StatsArgs s;
    s.logits = target_logits; s.row_stride = t_row_stride; s.V = V; s.c = c; s.draft_rows = 0; s.K = 1;
    s.cu = nullptr; s.q_seq_stride = 0; s.q_pos_stride = 0;
    s.out_stats = ctx->p_stats; s.out_argmax = sampling ? nullptr : ctx->p_argmax; s.status = ctx->status;
    s.out_partial = nullptr; s.idx_offset = 0; s.thr = nullptr;
    const int S = pick_cluster(ctx, n_rows, V, dtype);
    if (sampling)
        e = dtype == SVIP_BF16 ? launch_clustered(row_stats_kernel<kBF16, 1>, n_rows, S, s, st, kRingBytes)
                               : launch_clustered(row_stats_kernel<kF32, 1>, n_rows, S, s, st, kRingBytes);
    else
        e = dtype == SVIP_BF16 ? launch_clustered(row_stats_kernel<kBF16, 0>, n_rows, S, s, st, kRingBytes)
                               : launch_clustered(row_stats_kernel<kF32, 0>, n_rows, S, s, st, kRingBytes);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;

    if (!sampling) {
        TreeGreedyArgs g;
        g.tokens = tokens; g.parent = parent; g.p_argmax = ctx->p_argmax; g.B = B; g.N = N;
        g.n_accepted = n_accepted; g.path = path; g.next_token = next_token;
        e = launch_ex(verify_tree_greedy_kernel, static_cast<unsigned>((B + kPolicyThreads - 1) / kPolicyThreads),
                      kPolicyThreads, 0, 0, st, g);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        ctx->launches += 1;
        return SVIP_OK;
    }

    if (!q_stats) {
        StatsArgs d = s;
        d.logits = q_logits; d.row_stride = q_row_stride; d.out_stats = ctx->q_stats; d.out_argmax = nullptr;
        e = dtype == SVIP_BF16 ? launch_clustered(row_stats_kernel<kBF16, 1>, n_rows, S, d, st, kRingBytes)
                               : launch_clustered(row_stats_kernel<kF32, 1>, n_rows, S, d, st, kRingBytes);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        ctx->launches += 1;
    }

    TreeArgs t;
    t.tokens = tokens; t.parent = parent; t.q_logits = q_logits; t.q_row_stride = q_row_stride;
    t.q_stats = q_stats ? reinterpret_cast<const float2*>(q_stats) : ctx->q_stats;
    t.t_logits = target_logits; t.t_row_stride = t_row_stride; t.p_stats = ctx->p_stats;
    t.N = N; t.V = V; t.c = c; t.uniforms = uniforms; t.n_accepted = n_accepted; t.path = path;
    t.next_token = next_token; t.status = ctx->status;
    // the walk is a chain of passes over two rows: spread a sequence over as many blocks as the batch leaves room for
    int Sf = pick_cluster(ctx, B, V, dtype);
    if (ctx->cluster_override == 0) {
        const long row_bytes = static_cast<long>(V) * static_cast<long>(esz);
        while (Sf < kMaxCluster && 2 * row_bytes / Sf > (512L << 10)) Sf *= 2;
        if (Sf > kMaxCluster) Sf = kMaxCluster;
    }
    e = dtype == SVIP_BF16 ? launch_clustered(verify_tree_kernel<kBF16>, B, Sf, t, st, 0)
                           : launch_clustered(verify_tree_kernel<kF32>, B, Sf, t, st, 0);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return SVIP_OK;
}

int svip_selftest_wait_timeout(svip_ctx* ctx, long wait_ns, void* stream) {
    if (!ctx || wait_ns < 1 || wait_ns > 100000000L) return SVIP_ERR_INVALID_ARG;
    cudaError_t e = launch_ex(wait_timeout_kernel, 1, 32, 0, 0, static_cast<cudaStream_t>(stream),
                              static_cast<unsigned long long>(wait_ns), ctx->status);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return SVIP_OK;
}

int svip_policy_advance(svip_ctx* ctx, int policy, const uint8_t* stop, const int32_t* gamma,
                        int32_t* draft_len, uint8_t* active, int B, int K_cap, int32_t* n_active,
                        void* stream) {
    if (!ctx || !draft_len || !active || B < 0 || K_cap < 1) return SVIP_ERR_INVALID_ARG;
    if (policy != SVIP_POLICY_ENTROPY && policy != SVIP_POLICY_CONSTANT && policy != SVIP_POLICY_HEURISTIC)
        return SVIP_ERR_INVALID_ARG;
    if (policy == SVIP_POLICY_ENTROPY ? !stop : !gamma) return SVIP_ERR_INVALID_ARG;
    if (B == 0) return SVIP_OK;
    AdvanceArgs a;
    a.policy = policy; a.stop = stop; a.gamma = gamma; a.draft_len = draft_len; a.active = active;
    a.B = B; a.K_cap = K_cap; a.n_active = n_active;
    a.loop.iter = nullptr; a.loop.max_iters = 0; a.loop.handle = 0;
    const bool decides = ctx->loop_open && n_active && n_active == ctx->loop_n_active &&
                         static_cast<cudaStream_t>(stream) == ctx->loop_stream;
    if (decides) a.loop = ctx->loop;
    cudaError_t e = launch_ex(policy_advance_kernel, 1, kPolicyThreads, 0, 0, static_cast<cudaStream_t>(stream), a);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    if (decides) ctx->loop_decided = 1;
    ctx->launches += 1;
    return SVIP_OK;
}

int svip_policy_update(svip_ctx* ctx, int policy, const int32_t* n_accepted, int32_t* draft_len,
                       int32_t* gamma, uint8_t* active, int B, int K_cap, void* stream) {
    if (!ctx || !draft_len || !active || B < 0 || K_cap < 1) return SVIP_ERR_INVALID_ARG;
    if (policy != SVIP_POLICY_ENTROPY && policy != SVIP_POLICY_CONSTANT && policy != SVIP_POLICY_HEURISTIC)
        return SVIP_ERR_INVALID_ARG;
    if (policy == SVIP_POLICY_HEURISTIC && (!gamma || !n_accepted)) return SVIP_ERR_INVALID_ARG;
    if (B == 0) return SVIP_OK;
    UpdateArgs a;
    a.policy = policy; a.n_accepted = n_accepted; a.draft_len = draft_len; a.gamma = gamma; a.active = active;
    a.B = B; a.K_cap = K_cap;
    cudaError_t e = launch_ex(policy_update_kernel, static_cast<unsigned>((B + kPolicyThreads - 1) / kPolicyThreads),
                              kPolicyThreads, 0, 0, static_cast<cudaStream_t>(stream), a);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return SVIP_OK;
}

int svip_vp_partial(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V_shard, long row_stride,
                    float T, int vocab_offset, float* partial, void* stream) {
    if (!ctx || !logits || !partial) return SVIP_ERR_INVALID_ARG;
    if (dtype != SVIP_F32 && dtype != SVIP_BF16) return SVIP_ERR_UNSUPPORTED;
    if (B < 0 || V_shard < 1 || V_shard > 0x7fffffe0 || row_stride < 0 || vocab_offset < 0) return SVIP_ERR_INVALID_ARG;
    if (!(T >= 0.f) || std::isinf(T)) return SVIP_ERR_INVALID_ARG;
    if (!aligned_to(logits, dtype == SVIP_BF16 ? 2 : 4) || !aligned_to(partial, 16)) return SVIP_ERR_INVALID_ARG;
    if (B == 0) return SVIP_OK;
    SVIP_DEBUG_RANGES(ctx, static_cast<cudaStream_t>(stream), logits, rows_extent(B, row_stride, V_shard, dtype == SVIP_BF16 ? 2 : 4));
    StatsArgs s;
    s.logits = logits; s.row_stride = row_stride; s.V = V_shard; s.c = scale_for(T); s.draft_rows = 0; s.K = 1;
    s.cu = nullptr; s.q_seq_stride = 0; s.q_pos_stride = 0; s.out_stats = nullptr; s.out_argmax = nullptr;
    s.status = ctx->status; s.out_partial = reinterpret_cast<float4*>(partial); s.idx_offset = vocab_offset;
    const int S = pick_cluster(ctx, B, V_shard, dtype);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = dtype == SVIP_BF16 ? launch_clustered(row_stats_kernel<kBF16, 2>, B, S, s, st, kRingBytes)
                                       : launch_clustered(row_stats_kernel<kF32, 2>, B, S, s, st, kRingBytes);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return SVIP_OK;
}

int svip_vp_combine(svip_ctx* ctx, const float* partials, int G, int rank, int B, float T, float thresh,
                    const float* uniforms, float* entropy, uint8_t* stop, int32_t* token, int32_t* owner,
                    float* local_target, uint8_t* active, void* stream) {
    if (!ctx || !partials || !entropy || !stop || !token || !owner || !local_target || !active)
        return SVIP_ERR_INVALID_ARG;
    if (G < 1 || rank < 0 || rank >= G || B < 0) return SVIP_ERR_INVALID_ARG;
    if (!(T >= 0.f) || std::isinf(T) || std::isnan(thresh) || (T > 0.f && !uniforms)) return SVIP_ERR_INVALID_ARG;
    if (!aligned_to(partials, 16)) return SVIP_ERR_INVALID_ARG;
    if (B == 0) return SVIP_OK;
    VpCombineArgs a;
    a.partials = reinterpret_cast<const float4*>(partials); a.G = G; a.B = B; a.rank = rank; a.c = scale_for(T);
    a.thresh = thresh; a.greedy = T > 0.f ? 0 : 1; a.uniforms = uniforms; a.entropy = entropy; a.stop = stop;
    a.token = token; a.owner = owner; a.ext_target = local_target; a.active = active; a.status = ctx->status;
    cudaError_t e = launch_ex(vp_combine_kernel, static_cast<unsigned>((B + kPolicyThreads - 1) / kPolicyThreads),
                              kPolicyThreads, 0, 0, static_cast<cudaStream_t>(stream), a);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return SVIP_OK;
}

int svip_vp_locate(svip_ctx* ctx, const void* logits, svip_dtype dtype, int B, int V_shard, long row_stride,
                   float T, const float* local_target, const uint8_t* active, int vocab_offset,
                   int32_t* token, void* stream) {
    if (!ctx || !logits || !local_target || !active || !token) return SVIP_ERR_INVALID_ARG;
    if (dtype != SVIP_F32 && dtype != SVIP_BF16) return SVIP_ERR_UNSUPPORTED;
    if (B < 0 || V_shard < 1 || V_shard > 0x7fffffe0 || row_stride < 0 || vocab_offset < 0) return SVIP_ERR_INVALID_ARG;
    if (!(T > 0.f) || std::isinf(T)) return SVIP_ERR_INVALID_ARG;
    if (!aligned_to(logits, dtype == SVIP_BF16 ? 2 : 4)) return SVIP_ERR_INVALID_ARG;
    if (B == 0) return SVIP_OK;
    SVIP_DEBUG_RANGES(ctx, static_cast<cudaStream_t>(stream), logits, rows_extent(B, row_stride, V_shard, dtype == SVIP_BF16 ? 2 : 4));
    DraftArgs a;
    a.logits = logits; a.row_stride = row_stride; a.V = V_shard; a.c = scale_for(T); a.thresh = 0.f; a.greedy = 0;
    a.uniforms = nullptr; a.token = token; a.entropy = nullptr; a.stop = nullptr; a.row_stats = nullptr;
    a.status = ctx->status; a.active = active; a.ext_target = local_target; a.token_offset = vocab_offset;
    a.pos = nullptr; a.pos_stride = 0; a.slot_stride = 0; a.thr = nullptr;
    const int S = pick_cluster(ctx, B, V_shard, dtype);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = dtype == SVIP_BF16 ? launch_clustered(draft_step_kernel<kBF16, false, 2>, B, S, a, st, kRingBytes)
                                       : launch_clustered(draft_step_kernel<kF32, false, 2>, B, S, a, st, kRingBytes);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return SVIP_OK;
}

int svip_pair_stats(svip_ctx* ctx, const void* q_logits, long q_row_stride, const void* target_logits,
                    long t_row_stride, svip_dtype dtype, int n_pairs, int V, float T, float c_bound,
                    float* out, void* stream) {
    return svip_pair_stats_given(ctx, q_logits, q_row_stride, nullptr, target_logits, t_row_stride, nullptr, dtype,
                                 n_pairs, V, T, c_bound, out, stream);
}

int svip_pair_stats_given(svip_ctx* ctx, const void* q_logits, long q_row_stride, const float* q_stats,
                          const void* target_logits, long t_row_stride, const float* p_stats, svip_dtype dtype,
                          int n_pairs, int V, float T, float c_bound, float* out, void* stream) {
    if (!ctx || !q_logits || !target_logits || !out) return SVIP_ERR_INVALID_ARG;
    if ((q_stats == nullptr) != (p_stats == nullptr)) return SVIP_ERR_INVALID_ARG;
    if (q_stats && (!aligned_to(q_stats, 8) || !aligned_to(p_stats, 8))) return SVIP_ERR_INVALID_ARG;
    const bool given = q_stats != nullptr;
    if (dtype != SVIP_F32 && dtype != SVIP_BF16) return SVIP_ERR_UNSUPPORTED;
    if (n_pairs < 0 || V < 1 || V > 0x7fffffe0 || q_row_stride < 0 || t_row_stride < 0) return SVIP_ERR_INVALID_ARG;
    if (!(T > 0.f) || std::isinf(T) || !(c_bound >= 0.f)) return SVIP_ERR_INVALID_ARG;
    const size_t esz = dtype == SVIP_BF16 ? 2 : 4;
    if (!aligned_to(target_logits, esz) || !aligned_to(q_logits, esz)) return SVIP_ERR_INVALID_ARG;
    if (n_pairs == 0) return SVIP_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    SVIP_RANGE("svip_pair_stats");
    SVIP_DEBUG_RANGES(ctx, st, target_logits, rows_extent(n_pairs, t_row_stride, V, esz), q_logits,
                      rows_extent(n_pairs, q_row_stride, V, esz));
    // (Measured: spreading a pair over more blocks so that the second pass finds the rows in L2 costs more
    // in latency than it saves in traffic: 1024 pairs of 152064 bf16 logits 195 us at one block per pair,
    // 290 us at four.)
    const int S = pick_cluster(ctx, n_pairs, V, dtype);
    PairArgs p;
    p.t_logits = target_logits; p.t_row_stride = t_row_stride; p.q_logits = q_logits; p.q_row_stride = q_row_stride;
    p.V = V; p.c = scale_for(T); p.c_bound = c_bound; p.out = out; p.status = ctx->status;
    p.p_stats = reinterpret_cast<const float2*>(p_stats); p.q_stats = reinterpret_cast<const float2*>(q_stats);
    cudaError_t e;
    if (given)
        e = dtype == SVIP_BF16 ? launch_clustered(pair_stats_kernel<kBF16, true>, n_pairs, S, p, st, kRingBytes)
                               : launch_clustered(pair_stats_kernel<kF32, true>, n_pairs, S, p, st, kRingBytes);
    else
        e = dtype == SVIP_BF16 ? launch_clustered(pair_stats_kernel<kBF16>, n_pairs, S, p, st, kRingBytes)
                               : launch_clustered(pair_stats_kernel<kF32>, n_pairs, S, p, st, kRingBytes);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches += 1;
    return SVIP_OK;
}

int svip_graph_begin(svip_ctx* ctx, void* stream) {
    if (!ctx) return SVIP_ERR_INVALID_ARG;
    if (ctx->capturing) return SVIP_ERR_STATE;
    cudaError_t e = cudaSuccess;
    if (!ctx->loop_stream) {   // made now: no stream is created while a capture is open
        e = cudaStreamCreateWithFlags(&ctx->loop_stream, cudaStreamNonBlocking);
        if (e != cudaSuccess) { ctx->loop_stream = nullptr; return cuda_fail(ctx, e); }
    }
    e = cudaStreamBeginCapture(static_cast<cudaStream_t>(stream), cudaStreamCaptureModeThreadLocal);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->capturing = 1;
    return SVIP_OK;
}

int svip_graph_loop_begin(svip_ctx* ctx, void* stream, const int32_t* n_active, int max_iters, void** body_stream) {
    if (!ctx || !n_active || !body_stream || max_iters < 1) return SVIP_ERR_INVALID_ARG;
    if (!ctx->capturing || ctx->loop_open) return SVIP_ERR_STATE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the iteration counter starts at zero at every replay
    cudaError_t e = cudaMemsetAsync(ctx->loop_iter, 0, sizeof(int), st);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    cudaStreamCaptureStatus status = cudaStreamCaptureStatusNone;
    cudaGraph_t graph = nullptr;
    const cudaGraphNode_t* deps = nullptr;
    size_t n_deps = 0;
    e = cudaStreamGetCaptureInfo(st, &status, nullptr, &graph, &deps, &n_deps);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    if (status != cudaStreamCaptureStatusActive || !graph) return SVIP_ERR_STATE;
    // the body runs once before the first decision (the do-while of Algorithm 1): default value 1
    cudaGraphConditionalHandle handle;
    e = cudaGraphConditionalHandleCreate(&handle, graph, 1, cudaGraphCondAssignDefault);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    cudaGraphNodeParams params = {};
    params.type = cudaGraphNodeTypeConditional;
    params.conditional.handle = handle;
    params.conditional.type = cudaGraphCondTypeWhile;
    params.conditional.size = 1;
    cudaGraphNode_t node = nullptr;
    e = cudaGraphAddNode(&node, graph, deps, n_deps, &params);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    cudaGraph_t body = params.conditional.phGraph_out[0];
    // from here on the graph holds a loop: if its body cannot be recorded, svip_graph_end refuses
    // to hand the graph out (a loop without a deciding kernel would never end)
    // what is recorded on `stream` from here on comes after the loop
    e = cudaStreamUpdateCaptureDependencies(st, &node, 1, cudaStreamSetCaptureDependencies);
    if (e != cudaSuccess) { ctx->loop_failed = 1; return cuda_fail(ctx, e); }
    e = cudaStreamBeginCaptureToGraph(ctx->loop_stream, body, nullptr, nullptr, 0, cudaStreamCaptureModeThreadLocal);
    if (e != cudaSuccess) { ctx->loop_failed = 1; return cuda_fail(ctx, e); }
    ctx->loop.handle = handle;
    ctx->loop.iter = ctx->loop_iter;
    ctx->loop.max_iters = max_iters;
    ctx->loop_n_active = n_active;
    ctx->loop_open = 1;
    ctx->loop_decided = 0;
    t_plain_launches = true;
    *body_stream = ctx->loop_stream;
    return SVIP_OK;
}

int svip_graph_loop_end(svip_ctx* ctx) {
    if (!ctx) return SVIP_ERR_INVALID_ARG;
    if (!ctx->loop_open) return SVIP_ERR_STATE;
    cudaError_t e = cudaSuccess;
    if (!ctx->loop_decided) {   // no svip_policy_advance on the loop's counter in the body: decide here
        e = launch_ex(loop_decide_kernel, 1, 32, 0, 0, ctx->loop_stream, ctx->loop, ctx->loop_n_active);
        if (e == cudaSuccess) ctx->launches += 1;
    }
    cudaGraph_t body = nullptr;
    cudaError_t e2 = cudaStreamEndCapture(ctx->loop_stream, &body);
    ctx->loop_open = 0;
    t_plain_launches = false;
    if (e != cudaSuccess) { ctx->loop_failed = 1; return cuda_fail(ctx, e); }
    if (e2 != cudaSuccess) { ctx->loop_failed = 1; return cuda_fail(ctx, e2); }
    return SVIP_OK;
}

int svip_graph_end(svip_ctx* ctx, void* stream, svip_graph** graph) {
    if (!ctx || !graph) return SVIP_ERR_INVALID_ARG;
    if (!ctx->capturing) return SVIP_ERR_STATE;
    // a loop whose body was left open, or whose decision kernel could not be recorded, would
    // never end at replay: such a graph is not handed out
    bool broken = ctx->loop_failed != 0;
    if (ctx->loop_open) {
        cudaGraph_t body = nullptr;
        cudaStreamEndCapture(ctx->loop_stream, &body);
        ctx->loop_open = 0;
        t_plain_launches = false;
        broken = true;
    }
    ctx->loop_failed = 0;
    ctx->capturing = 0;
    cudaGraph_t g = nullptr;
    cudaError_t e = cudaStreamEndCapture(static_cast<cudaStream_t>(stream), &g);
    if (broken) {
        if (g) cudaGraphDestroy(g);
        cudaGetLastError();
        return SVIP_ERR_STATE;
    }
    if (e != cudaSuccess || !g) return cuda_fail(ctx, e);
    cudaGraphExec_t ex = nullptr;
    e = cudaGraphInstantiate(&ex, g, 0);
    if (e != cudaSuccess) { cudaGraphDestroy(g); return cuda_fail(ctx, e); }
    svip_graph* out = new (std::nothrow) svip_graph();
    if (!out) { cudaGraphExecDestroy(ex); cudaGraphDestroy(g); return SVIP_ERR_CUDA; }
    out->exec = ex; out->graph = g;
    *graph = out;
    return SVIP_OK;
}

int svip_graph_launch(svip_graph* graph, void* stream) {
    if (!graph) return SVIP_ERR_INVALID_ARG;
    return cudaGraphLaunch(graph->exec, static_cast<cudaStream_t>(stream)) == cudaSuccess ? SVIP_OK : SVIP_ERR_CUDA;
}

int svip_graph_destroy(svip_graph* graph) {
    if (!graph) return SVIP_ERR_INVALID_ARG;
    cudaGraphExecDestroy(graph->exec);
    cudaGraphDestroy(graph->graph);
    delete graph;
    return SVIP_OK;
}

// ------------------------------------------------------------------ verify without allocation
//
// Workspace of svip_verify_noalloc: one fixed array in the library's device image instead of
// cudaMalloc'ed memory.  Layout: [p_stats | q_stats | p_argmax | status word].  Every call on a
// device reuses it, so calls that overlap on the GPU race (see include/svip.h).

namespace {

constexpr size_t kNoAllocRows = SVIP_NOALLOC_MAX_ROWS;
constexpr size_t kNoAllocStatsBytes = kNoAllocRows * sizeof(float2);
constexpr size_t kNoAllocBytes = 2 * kNoAllocStatsBytes + kNoAllocRows * sizeof(int32_t) + 256;

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

constexpr int kNoAllocMaxDevices = 64;

struct NoAllocDevice {
    int ready;
    int num_sms;
    unsigned char* base;   // device address of g_noalloc_scratch on this device
};
NoAllocDevice g_noalloc_dev[kNoAllocMaxDevices];
std::mutex g_noalloc_mutex;   // the per-device set-up may be reached from several host threads

// Once per device, with that device current: the host-side name g_noalloc_scratch is not a device
// address, so ask the runtime for the address the kernels must be given.
int noalloc_setup(int device, NoAllocDevice** out) {
    if (device < 0 || device >= kNoAllocMaxDevices) return SVIP_ERR_INVALID_ARG;
    NoAllocDevice* d = &g_noalloc_dev[device];
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!d->ready) {
        int current = -1;
        if (cudaGetDevice(&current) != cudaSuccess) { cudaGetLastError(); return SVIP_ERR_CUDA; }
        if (current != device) return SVIP_ERR_INVALID_ARG;
        int major = 0, sms = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
            cudaGetLastError();
            return SVIP_ERR_CUDA;
        }
        if (major != 10) return SVIP_ERR_UNSUPPORTED;
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return SVIP_ERR_CUDA;
        }
        const void* ringed[] = {
            (const void*)row_stats_kernel<kBF16, 0>, (const void*)row_stats_kernel<kBF16, 1>,
            (const void*)row_stats_kernel<kF32, 0>,  (const void*)row_stats_kernel<kF32, 1>,
            (const void*)verify_finish_kernel<kBF16>, (const void*)verify_finish_kernel<kF32>};
        for (const void* k : ringed)
            if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, kRingBytes) != cudaSuccess) {
                cudaGetLastError();
                return SVIP_ERR_CUDA;
            }
        d->num_sms = sms;
        d->base = static_cast<unsigned char*>(ptr);
        d->ready = 1;
    }
    *out = d;
    return SVIP_OK;
}

}  // namespace

int svip_verify_noalloc(int device, const int32_t* draft_tokens, const void* q_logits, long q_row_stride,
                        const float* q_stats, long q_seq_stride, long q_pos_stride,
                        const void* target_logits, long t_row_stride, svip_dtype dtype,
                        const int32_t* cu_rows, int B, int K, int n_target_rows, int V, float T,
                        const float* uniforms, int32_t* n_accepted, int32_t* next_token,
                        unsigned* status, void* stream) {
    if (n_target_rows > SVIP_NOALLOC_MAX_ROWS) return SVIP_ERR_WORKSPACE;
    NoAllocDevice* d = nullptr;
    int rc = noalloc_setup(device, &d);
    if (rc != SVIP_OK) return rc;
    // A context that lives on this call's stack and points into the fixed array; nothing is allocated.
    svip_ctx view = {};
    view.device = device;
    view.max_rows = SVIP_NOALLOC_MAX_ROWS;
    view.num_sms = d->num_sms;
    view.p_stats = reinterpret_cast<float2*>(d->base);
    view.q_stats = reinterpret_cast<float2*>(d->base + kNoAllocStatsBytes);
    view.p_argmax = reinterpret_cast<int32_t*>(d->base + 2 * kNoAllocStatsBytes);
    unsigned* own_status = reinterpret_cast<unsigned*>(d->base + 2 * kNoAllocStatsBytes +
                                                       kNoAllocRows * sizeof(int32_t));
    view.status = status ? status : own_status;
    // the status word must start at zero; everything else in the array is written before it is read
    if (cudaMemsetAsync(view.status, 0, sizeof(unsigned), static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        cudaGetLastError();
        return SVIP_ERR_CUDA;
    }
    return svip_verify(&view, draft_tokens, q_logits, q_row_stride, q_stats, q_seq_stride, q_pos_stride,
                       target_logits, t_row_stride, dtype, cu_rows, B, K, n_target_rows, V, T, uniforms,
                       n_accepted, next_token, stream);
}

}  // extern "C"

