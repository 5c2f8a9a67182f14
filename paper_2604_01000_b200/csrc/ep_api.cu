// C ABI entry points: argument checks on the host, then the kernels of the other translation units.
#include "ep_common.cuh"

#include <nvtx3/nvToolsExt.h>

#include <algorithm>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>

namespace ep {

int fail(ep_ctx *ctx, int status, const char *fmt, ...) {
    if (ctx) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(ctx->last_error, sizeof(ctx->last_error), fmt, ap);
        va_end(ap);
    }
    return status;
}

int cuda_fail(ep_ctx *ctx, cudaError_t e, const char *what) {
    return fail(ctx, EP_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

// Names of the timed regions as a profiler's timeline shows them (NVTX ranges around the host-side enqueue; they cost
// nothing while no tool is attached).
static const char *const kRangeNames[EP_TIMER_COUNT] = {
    "ep:kmeans assign", "ep:kmeans update", "ep:edge cut", "ep:quality prep", "ep:reorder",
    "ep:kmeans resolve", "ep:graph bandwidth", "ep:relabel", "ep:balance"};

Timed::Timed(ep_ctx *c, cudaStream_t s, int t) : ctx(c), stream(s), timer(c->opt_timer_group * EP_TIMER_COUNT + t) {
    nvtxRangePushA(kRangeNames[t >= 0 && t < EP_TIMER_COUNT ? t : 0]);
    if (!ctx->opt_profile) return;
    if (!ctx->spare_events.empty()) {
        start = ctx->spare_events.back();
        ctx->spare_events.pop_back();
    } else if (cudaEventCreate(&start) != cudaSuccess) {
        start = nullptr;
        return;
    }
    cudaEventRecord(start, stream);
}

void Timed::end(int kernels) {
    ctx->launches += kernels;
    nvtxRangePop();
    if (!start) return;
    cudaEvent_t stop = nullptr;
    if (!ctx->spare_events.empty()) {
        stop = ctx->spare_events.back();
        ctx->spare_events.pop_back();
    } else if (cudaEventCreate(&stop) != cudaSuccess) {
        ctx->spare_events.push_back(start);
        start = nullptr;
        return;
    }
    cudaEventRecord(stop, stream);
    ctx->intervals.push_back({timer, start, stop});
    start = nullptr;
}

}  // namespace ep

using namespace ep;

namespace {

// out[i] = emb[rows[i]]: a warp per row, 16 bytes per lane and step.
__global__ void __launch_bounds__(256) gather_rows(const float *__restrict__ emb, int64_t N, int d4,
                                                   const int64_t *__restrict__ rows, int64_t M,
                                                   float *__restrict__ out, int *status) {
    const int lane = threadIdx.x & 31;
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    for (int64_t i = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); i < M; i += warps) {
        int64_t r = rows[i];
        if (r < 0 || r >= N) {
            if (lane == 0) ep_raise(status, EP_ERR_BAD_INDEX);
            r = 0;
        }
        const float4 *src = reinterpret_cast<const float4 *>(emb) + r * d4;
        float4 *dst = reinterpret_cast<float4 *>(out) + i * d4;
        for (int q = lane; q < d4; q += 32) dst[q] = __ldg(src + q);
    }
}

struct SampledLayout {
    float *sample;
    int32_t *sample_assign;
    void *ws_train, *ws_full;
    size_t train_bytes, full_bytes, used;
};

bool sampled_layout(const ep_ctx *ctx, int64_t N, int d, int K, int64_t M, void *workspace, SampledLayout *out) {
    KMeansPlan train, full;
    if (M < K || M > N || !kmeans_make_plan(ctx, M, d, K, &train) || !kmeans_make_plan(ctx, N, d, K, &full)) return false;
    Arena a(workspace);
    SampledLayout l{};
    l.sample = a.take<float>((size_t)M * d);
    l.sample_assign = a.take<int32_t>(M);
    l.train_bytes = kmeans_workspace_layout(ctx, train, nullptr, nullptr);
    l.full_bytes = kmeans_workspace_layout(ctx, full, nullptr, nullptr);
    l.ws_train = a.take<char>(l.train_bytes);
    l.ws_full = a.take<char>(l.full_bytes);
    l.used = a.used;
    *out = l;
    return true;
}

}  // namespace

namespace {

// mask[v] = 1 when split[v] == which, else 0.
__global__ void __launch_bounds__(256) split_mask(const uint8_t *__restrict__ split, int64_t N, int which,
                                                  uint8_t *__restrict__ mask) {
    const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (v < N) mask[v] = split[v] == which ? 1 : 0;
}

}  // namespace

extern "C" {

const char *ep_status_string(int status) {
    switch (status) {
        case EP_OK: return "ok";
        case EP_ERR_INVALID_ARG: return "invalid argument";
        case EP_ERR_UNSUPPORTED: return "unsupported device or shape";
        case EP_ERR_WORKSPACE: return "workspace too small or misaligned";
        case EP_ERR_BAD_INDEX: return "label, column index or row pointer out of range";
        case EP_ERR_TIMEOUT: return "bounded device wait expired";
        case EP_ERR_CUDA: return "CUDA call failed";
        default: return "unknown status";
    }
}

int ep_create(ep_ctx **out, int device) {
    if (!out) return EP_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || count == 0) return EP_ERR_UNSUPPORTED;   // no CUDA device at all
    if (device < 0 || device >= count) return EP_ERR_INVALID_ARG;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return EP_ERR_CUDA;
    if (prop.major != 10) return EP_ERR_UNSUPPORTED;
    ep_ctx *ctx = new (std::nothrow) ep_ctx();
    if (!ctx) return EP_ERR_CUDA;
    ctx->device = device;
    ctx->sm_count = prop.multiProcessorCount;
    ctx->smem_optin = (int)prop.sharedMemPerBlockOptin;
    ctx->opt_kmeans_path = 0;
    ctx->opt_profile = 0;
    ctx->opt_timer_group = 0;
    ctx->opt_cand_mb = 1024;
    ctx->opt_slice_kb = 56 * 1024;
    ctx->opt_iters_per_launch = 0;
    ctx->launches = 0;
    ctx->last_error[0] = 0;
    DeviceGuard g(device);
    if (cudaMalloc(&ctx->d_status, 256) != cudaSuccess || cudaMemset(ctx->d_status, 0, 256) != cudaSuccess) {
        delete ctx;
        return EP_ERR_CUDA;
    }
    *out = ctx;
    return EP_OK;
}

int ep_destroy(ep_ctx *ctx) {
    if (!ctx) return EP_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    cudaFree(ctx->d_status);
    if (ctx->probe_tex) cudaDestroyTextureObject((cudaTextureObject_t)ctx->probe_tex);
    for (auto &iv : ctx->intervals) {
        cudaEventDestroy(iv.start);
        cudaEventDestroy(iv.stop);
    }
    for (auto e : ctx->spare_events) cudaEventDestroy(e);
    delete ctx;
    return EP_OK;
}

const char *ep_last_error(const ep_ctx *ctx) { return ctx ? ctx->last_error : ""; }

int ep_poll_status(ep_ctx *ctx) {
    if (!ctx) return EP_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    int word = 0;
    EP_CUDA(ctx, cudaDeviceSynchronize());
    EP_CUDA(ctx, cudaMemcpy(&word, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost));
    if (word != 0) EP_CUDA(ctx, cudaMemset(ctx->d_status, 0, sizeof(int)));
    return word;
}

int ep_set_option(ep_ctx *ctx, int option, int value) {
    if (!ctx) return EP_ERR_INVALID_ARG;
    if (option == EP_OPT_KMEANS_PATH && value >= 0 && value <= 2) {
        ctx->opt_kmeans_path = value;
        return EP_OK;
    }
    if (option == EP_OPT_PROFILE && (value == 0 || value == 1)) {
        ctx->opt_profile = value;
        return EP_OK;
    }
    if (option == EP_OPT_TIMER_GROUP && value >= 0 && value < 4) {
        ctx->opt_timer_group = value;
        return EP_OK;
    }
    if (option == EP_OPT_KMEANS_CAND_MB && value >= 1 && value <= 32768) {
        ctx->opt_cand_mb = value;
        return EP_OK;
    }
    if (option == EP_OPT_QUALITY_SLICE_KB && value >= 1 && value <= 4194304) {
        ctx->opt_slice_kb = value;
        return EP_OK;
    }
    if (option == EP_OPT_KMEANS_ITERATIONS_PER_LAUNCH && value >= 0 && value <= 2) {
        ctx->opt_iters_per_launch = value;
        return EP_OK;
    }
    return fail(ctx, EP_ERR_INVALID_ARG, "unknown option %d or value %d", option, value);
}

int ep_get_option(const ep_ctx *ctx, int option, int *value) {
    if (!ctx || !value) return EP_ERR_INVALID_ARG;
    if (option == EP_OPT_KMEANS_PATH) {
        *value = ctx->opt_kmeans_path;
        return EP_OK;
    }
    if (option == EP_OPT_PROFILE) {
        *value = ctx->opt_profile;
        return EP_OK;
    }
    if (option == EP_OPT_TIMER_GROUP) {
        *value = ctx->opt_timer_group;
        return EP_OK;
    }
    if (option == EP_OPT_KMEANS_CAND_MB) {
        *value = ctx->opt_cand_mb;
        return EP_OK;
    }
    if (option == EP_OPT_QUALITY_SLICE_KB) {
        *value = ctx->opt_slice_kb;
        return EP_OK;
    }
    if (option == EP_OPT_KMEANS_ITERATIONS_PER_LAUNCH) {
        *value = ctx->opt_iters_per_launch;
        return EP_OK;
    }
    return EP_ERR_INVALID_ARG;
}

int ep_profile_read(ep_ctx *ctx, int timer, double *total_ms, int64_t *intervals) {
    if (!ctx || timer < 0 || timer >= 4 * EP_TIMER_COUNT) return EP_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    double ms = 0.0;
    int64_t n = 0;
    std::vector<ep_timed_interval> keep;
    for (auto &iv : ctx->intervals) {
        if (iv.timer != timer) {
            keep.push_back(iv);
            continue;
        }
        float t = 0.f;
        EP_CUDA(ctx, cudaEventSynchronize(iv.stop));
        EP_CUDA(ctx, cudaEventElapsedTime(&t, iv.start, iv.stop));
        ms += t;
        n += 1;
        ctx->spare_events.push_back(iv.start);
        ctx->spare_events.push_back(iv.stop);
    }
    ctx->intervals.swap(keep);
    if (total_ms) *total_ms = ms;
    if (intervals) *intervals = n;
    return EP_OK;
}

int64_t ep_launch_count(const ep_ctx *ctx) { return ctx ? ctx->launches : 0; }

int ep_debug_counters(ep_ctx *ctx, int64_t *out) {
    if (!ctx || !out) return EP_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    EP_CUDA(ctx, cudaDeviceSynchronize());
    EP_CUDA(ctx, cudaMemcpy(out, ctx->d_status + EP_COUNTER_WORD0, sizeof(int64_t) * EP_COUNTERS, cudaMemcpyDeviceToHost));
    EP_CUDA(ctx, cudaMemset(ctx->d_status + EP_COUNTER_WORD0, 0, sizeof(int64_t) * EP_COUNTERS));
    return EP_OK;
}

// ---------------------------------------------------------------------------------------------- k-means
size_t ep_kmeans_workspace_bytes(const ep_ctx *ctx, int64_t N, int32_t d, int32_t K) {
    KMeansPlan plan;
    if (!ctx || !kmeans_make_plan(ctx, N, d, K, &plan)) return 0;
    return kmeans_workspace_layout(ctx, plan, nullptr, nullptr);
}

int ep_kmeans(ep_ctx *ctx, const float *emb, int64_t N, int32_t d, int32_t K, int32_t iters,
              const float *init_centroids, int32_t *assign, float *centroids, double *objective, void *workspace,
              size_t workspace_bytes, void *cuda_stream) {
    if (!ctx) return EP_ERR_INVALID_ARG;
    if (!emb || !init_centroids || !assign || !centroids) return fail(ctx, EP_ERR_INVALID_ARG, "null pointer");
    if (!aligned(emb, 16) || !aligned(init_centroids, 16) || !aligned(centroids, 16) || !aligned(assign, 4) ||
        (objective && !aligned(objective, 8)))
        return fail(ctx, EP_ERR_INVALID_ARG, "misaligned pointer");
    if (iters < 0) return fail(ctx, EP_ERR_INVALID_ARG, "iters < 0");
    KMeansPlan plan;
    if (!kmeans_make_plan(ctx, N, d, K, &plan))
        return fail(ctx, EP_ERR_INVALID_ARG, "shape out of range: N=%lld d=%d K=%d", (long long)N, d, K);
    const size_t need = kmeans_workspace_layout(ctx, plan, nullptr, nullptr);
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < need)
        return fail(ctx, EP_ERR_WORKSPACE, "k-means workspace: need %zu bytes, 256-byte aligned", need);
    DeviceGuard g(ctx->device);
    return kmeans_run(ctx, plan, emb, iters, init_centroids, assign, centroids, objective, workspace,
                      static_cast<cudaStream_t>(cuda_stream));
}

// ---------------------------------------------------------------------------------------------- sampled k-means
int ep_gather_rows(ep_ctx *ctx, const float *emb, int64_t N, int32_t d, const int64_t *rows, int64_t M, float *out,
                   void *cuda_stream) {
    if (!ctx) return EP_ERR_INVALID_ARG;
    if (!emb || !rows || !out) return fail(ctx, EP_ERR_INVALID_ARG, "null pointer");
    if (N < 1 || M < 1 || d < 4 || d > 1024 || (d & 3))
        return fail(ctx, EP_ERR_INVALID_ARG, "shape out of range: N=%lld M=%lld d=%d", (long long)N, (long long)M, d);
    if (!aligned(emb, 16) || !aligned(out, 16) || !aligned(rows, 8)) return fail(ctx, EP_ERR_INVALID_ARG, "misaligned pointer");
    DeviceGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int grid = (int)std::max<int64_t>(1, std::min<int64_t>((int64_t)ctx->sm_count * 8, ceil_div(M, 8)));
    gather_rows<<<grid, 256, 0, st>>>(emb, N, d >> 2, rows, M, out, ctx->d_status);
    ctx->launches += 1;
    EP_CUDA(ctx, cudaGetLastError());
    return EP_OK;
}

size_t ep_kmeans_sampled_workspace_bytes(const ep_ctx *ctx, int64_t N, int32_t d, int32_t K, int64_t M) {
    SampledLayout l;
    if (!ctx || !sampled_layout(ctx, N, d, K, M, nullptr, &l)) return 0;
    return l.used;
}

int ep_kmeans_sampled(ep_ctx *ctx, const float *emb, int64_t N, int32_t d, int32_t K, int32_t iters,
                      const int64_t *sample_rows, int64_t M, const float *init_centroids, int32_t *assign,
                      float *centroids, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!ctx) return EP_ERR_INVALID_ARG;
    if (!emb || !sample_rows || !init_centroids || !assign || !centroids) return fail(ctx, EP_ERR_INVALID_ARG, "null pointer");
    if (iters < 1) return fail(ctx, EP_ERR_INVALID_ARG, "the centroids need at least one iteration on the sample");
    SampledLayout l;
    if (!sampled_layout(ctx, N, d, K, M, workspace, &l))
        return fail(ctx, EP_ERR_INVALID_ARG, "shape out of range: N=%lld d=%d K=%d M=%lld (K <= M <= N)", (long long)N, d, K,
                    (long long)M);
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < l.used)
        return fail(ctx, EP_ERR_WORKSPACE, "sampled k-means workspace: need %zu bytes, 256-byte aligned", l.used);
    int rc = ep_gather_rows(ctx, emb, N, d, sample_rows, M, l.sample, cuda_stream);
    if (rc != EP_OK) return rc;
    rc = ep_kmeans(ctx, l.sample, M, d, K, iters, init_centroids, l.sample_assign, centroids, nullptr, l.ws_train,
                   l.train_bytes, cuda_stream);
    if (rc != EP_OK) return rc;
    return ep_kmeans(ctx, emb, N, d, K, 0, centroids, assign, centroids, nullptr, l.ws_full, l.full_bytes, cuda_stream);
}

// ---------------------------------------------------------------------------------------------- quality
static bool quality_shape_ok(int64_t N, int64_t nnz, int32_t K) {
    return N >= 1 && N < (int64_t(1) << 31) && nnz >= 0 && nnz < (int64_t(1) << 62) && K >= 1 && K <= (1 << 24);
}

size_t ep_quality_workspace_bytes(const ep_ctx *ctx, int64_t N, int64_t nnz, int32_t K) {
    if (!ctx || !quality_shape_ok(N, nnz, K)) return 0;
    return quality_workspace_bytes(N, nnz, K);
}

int ep_partition_quality(ep_ctx *ctx, const void *rowptr, int32_t rowptr_is_int64, const int32_t *colidx,
                         int64_t nnz, const int32_t *assign, int64_t N, int32_t K, uint64_t *edge_cut,
                         int64_t *part_vertices, int64_t *part_edges, void *workspace, size_t workspace_bytes,
                         void *cuda_stream) {
    if (!ctx) return EP_ERR_INVALID_ARG;
    if (!quality_shape_ok(N, nnz, K))
        return fail(ctx, EP_ERR_INVALID_ARG, "shape out of range: N=%lld nnz=%lld K=%d", (long long)N, (long long)nnz, K);
    if (!rowptr || (!colidx && nnz > 0) || !assign || !edge_cut || !part_vertices || !part_edges)
        return fail(ctx, EP_ERR_INVALID_ARG, "null pointer");
    if (!rowptr_is_int64 && nnz >= (int64_t(1) << 31))
        return fail(ctx, EP_ERR_INVALID_ARG, "nnz needs a 64-bit row pointer");
    if (!aligned(rowptr, rowptr_is_int64 ? 8 : 4) || !aligned(colidx, 16) || !aligned(assign, 4) ||
        !aligned(edge_cut, 8) || !aligned(part_vertices, 8) || !aligned(part_edges, 8))
        return fail(ctx, EP_ERR_INVALID_ARG, "misaligned pointer");
    const size_t need = quality_workspace_bytes(N, nnz, K);
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < need)
        return fail(ctx, EP_ERR_WORKSPACE, "quality workspace: need %zu bytes, 256-byte aligned", need);
    DeviceGuard g(ctx->device);
    return quality_run(ctx, rowptr, rowptr_is_int64 != 0, colidx, nnz, assign, N, K,
                       reinterpret_cast<unsigned long long *>(edge_cut), reinterpret_cast<long long *>(part_vertices),
                       reinterpret_cast<long long *>(part_edges), workspace, static_cast<cudaStream_t>(cuda_stream));
}

// ---------------------------------------------------------------------------------------------- graph bandwidth
static bool bandwidth_shape_ok(int64_t N, int64_t nnz) {
    return N >= 1 && N < (int64_t(1) << 31) && nnz >= 0 && nnz < (int64_t(1) << 62);
}

size_t ep_graph_bandwidth_workspace_bytes(const ep_ctx *ctx, int64_t N, int64_t nnz) {
    if (!ctx || !bandwidth_shape_ok(N, nnz)) return 0;
    return bandwidth_workspace_bytes(N, nnz);
}

int ep_graph_bandwidth(ep_ctx *ctx, const void *rowptr, int32_t rowptr_is_int64, const int32_t *colidx, int64_t nnz,
                       const int32_t *pi, int64_t N, uint64_t *bandwidth_sum, int32_t *vertex_bandwidth,
                       void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!ctx) return EP_ERR_INVALID_ARG;
    if (!bandwidth_shape_ok(N, nnz))
        return fail(ctx, EP_ERR_INVALID_ARG, "shape out of range: N=%lld nnz=%lld", (long long)N, (long long)nnz);
    if (!rowptr || (!colidx && nnz > 0) || !pi || !bandwidth_sum) return fail(ctx, EP_ERR_INVALID_ARG, "null pointer");
    if (!rowptr_is_int64 && nnz >= (int64_t(1) << 31))
        return fail(ctx, EP_ERR_INVALID_ARG, "nnz needs a 64-bit row pointer");
    if (!aligned(rowptr, rowptr_is_int64 ? 8 : 4) || !aligned(colidx, 16) || !aligned(pi, 4) ||
        !aligned(bandwidth_sum, 8) || (vertex_bandwidth && !aligned(vertex_bandwidth, 4)))
        return fail(ctx, EP_ERR_INVALID_ARG, "misaligned pointer");
    const size_t need = bandwidth_workspace_bytes(N, nnz);
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < need)
        return fail(ctx, EP_ERR_WORKSPACE, "graph bandwidth workspace: need %zu bytes, 256-byte aligned", need);
    DeviceGuard g(ctx->device);
    return bandwidth_run(ctx, rowptr, rowptr_is_int64 != 0, colidx, nnz, pi, N,
                         reinterpret_cast<unsigned long long *>(bandwidth_sum), vertex_bandwidth, workspace,
                         static_cast<cudaStream_t>(cuda_stream));
}

size_t ep_graph_bandwidth_host_arena_bytes(const ep_ctx *ctx, int64_t N, int64_t nnz, int32_t rowptr_is_int64) {
    const size_t ws = ep_graph_bandwidth_workspace_bytes(ctx, N, nnz);
    if (ws == 0) return 0;
    Arena a(nullptr);
    a.take<char>((size_t)(N + 1) * (rowptr_is_int64 ? 8 : 4));
    a.take<int32_t>(nnz);
    a.take<int32_t>(N);
    a.take<int32_t>(N);
    a.take<uint64_t>(1);
    return a.used + ws;
}

int ep_graph_bandwidth_host(ep_ctx *ctx, const void *rowptr, int32_t rowptr_is_int64, const int32_t *colidx,
                            int64_t nnz, const int32_t *pi, int64_t N, uint64_t *bandwidth_sum,
                            int32_t *vertex_bandwidth, void *arena, size_t arena_bytes, void *cuda_stream) {
    if (!ctx) return EP_ERR_INVALID_ARG;
    if (!rowptr || (!colidx && nnz > 0) || !pi || !bandwidth_sum) return fail(ctx, EP_ERR_INVALID_ARG, "null pointer");
    const size_t need = ep_graph_bandwidth_host_arena_bytes(ctx, N, nnz, rowptr_is_int64);
    if (need == 0)
        return fail(ctx, EP_ERR_INVALID_ARG, "shape out of range: N=%lld nnz=%lld", (long long)N, (long long)nnz);
    if (!arena || !aligned(arena, 256) || arena_bytes < need)
        return fail(ctx, EP_ERR_WORKSPACE, "graph bandwidth host arena: need %zu bytes, 256-byte aligned", need);
    DeviceGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    Arena a(arena);
    const size_t rp_bytes = (size_t)(N + 1) * (rowptr_is_int64 ? 8 : 4);
    char *d_rp = a.take<char>(rp_bytes);
    int32_t *d_ci = a.take<int32_t>(nnz);
    int32_t *d_pi = a.take<int32_t>(N);
    int32_t *d_vb = a.take<int32_t>(N);
    uint64_t *d_sum = a.take<uint64_t>(1);
    void *ws = a.base + a.used;
    EP_CUDA(ctx, cudaMemcpyAsync(d_rp, rowptr, rp_bytes, cudaMemcpyHostToDevice, st));
    if (nnz > 0) EP_CUDA(ctx, cudaMemcpyAsync(d_ci, colidx, sizeof(int32_t) * nnz, cudaMemcpyHostToDevice, st));
    EP_CUDA(ctx, cudaMemcpyAsync(d_pi, pi, sizeof(int32_t) * N, cudaMemcpyHostToDevice, st));
    int rc = ep_graph_bandwidth(ctx, d_rp, rowptr_is_int64, d_ci, nnz, d_pi, N, d_sum, vertex_bandwidth ? d_vb : nullptr,
                                ws, arena_bytes - a.used, st);
    if (rc != EP_OK) return rc;
    EP_CUDA(ctx, cudaMemcpyAsync(bandwidth_sum, d_sum, sizeof(uint64_t), cudaMemcpyDeviceToHost, st));
    if (vertex_bandwidth)
        EP_CUDA(ctx, cudaMemcpyAsync(vertex_bandwidth, d_vb, sizeof(int32_t) * N, cudaMemcpyDeviceToHost, st));
    return EP_OK;
}

// ---------------------------------------------------------------------------------------------- relabel
size_t ep_relabel_graph_workspace_bytes(const ep_ctx *ctx, int64_t N, int64_t nnz) {
    if (!ctx || !bandwidth_shape_ok(N, nnz)) return 0;
    return relabel_workspace_bytes(N, nnz);
}

int ep_relabel_graph(ep_ctx *ctx, const void *rowptr, int32_t rowptr_is_int64, const int32_t *colidx, int64_t nnz,
                     const int32_t *perm, const int32_t *inv_perm, int64_t N, void *new_rowptr, int32_t *new_colidx,
                     void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!ctx) return EP_ERR_INVALID_ARG;
    if (!bandwidth_shape_ok(N, nnz))
        return fail(ctx, EP_ERR_INVALID_ARG, "shape out of range: N=%lld nnz=%lld", (long long)N, (long long)nnz);
    if (!rowptr || (!colidx && nnz > 0) || !perm || !inv_perm || !new_rowptr || (!new_colidx && nnz > 0))
        return fail(ctx, EP_ERR_INVALID_ARG, "null pointer");
    if (!rowptr_is_int64 && nnz >= (int64_t(1) << 31))
        return fail(ctx, EP_ERR_INVALID_ARG, "nnz needs a 64-bit row pointer");
    const size_t rw = rowptr_is_int64 ? 8 : 4;
    if (!aligned(rowptr, rw) || !aligned(new_rowptr, rw) || !aligned(colidx, 4) || !aligned(new_colidx, 4) ||
        !aligned(perm, 4) || !aligned(inv_perm, 4))
        return fail(ctx, EP_ERR_INVALID_ARG, "misaligned pointer");
    const size_t need = relabel_workspace_bytes(N, nnz);
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < need)
        return fail(ctx, EP_ERR_WORKSPACE, "relabel workspace: need %zu bytes, 256-byte aligned", need);
    DeviceGuard g(ctx->device);
    return relabel_run(ctx, rowptr, rowptr_is_int64 != 0, colidx, nnz, perm, inv_perm, N, new_rowptr, new_colidx, workspace,
                       static_cast<cudaStream_t>(cuda_stream));
}

int ep_permute_rows(ep_ctx *ctx, const float *emb, int64_t N, int32_t d, const int32_t *perm, float *out,
                    void *cuda_stream) {
    if (!ctx) return EP_ERR_INVALID_ARG;
    if (!emb || !perm || !out || emb == out) return fail(ctx, EP_ERR_INVALID_ARG, "null pointer or out == emb");
    if (N < 1 || N >= (int64_t(1) << 31) || d < 4 || d > 1024 || (d & 3))
        return fail(ctx, EP_ERR_INVALID_ARG, "shape out of range: N=%lld d=%d", (long long)N, d);
    if (!aligned(emb, 16) || !aligned(out, 16) || !aligned(perm, 4)) return fail(ctx, EP_ERR_INVALID_ARG, "misaligned pointer");
    DeviceGuard g(ctx->device);
    return permute_rows_run(ctx, emb, N, d, perm, out, static_cast<cudaStream_t>(cuda_stream));
}

// ---------------------------------------------------------------------------------------------- balance
size_t ep_balance_workspace_bytes(const ep_ctx *ctx, int64_t N, int32_t K, int64_t max_degree) {
    if (!ctx || !balance_shape_ok(N, K, max_degree)) return 0;
    return balance_workspace_bytes(N, K, max_degree);
}

static int balance_check_args(ep_ctx *ctx, const void *rowptr, int32_t rowptr_is_int64, int64_t N, int32_t K,
                              int64_t capacity, int64_t max_degree, const int32_t *assign, void *workspace,
                              size_t workspace_bytes) {
    if (N < 1 || N >= (int64_t(1) << 31) || K < 1 || max_degree < 0 || capacity < 0)
        return fail(ctx, EP_ERR_INVALID_ARG, "shape out of range: N=%lld K=%d max_degree=%lld capacity=%lld", (long long)N, K,
                    (long long)max_degree, (long long)capacity);
    if (!balance_shape_ok(N, K, max_degree))
        return fail(ctx, EP_ERR_UNSUPPORTED, "K=%d with max_degree=%lld: K <= 1024 and K * (max_degree + 1) < 2^30 are required",
                    K, (long long)max_degree);
    if (!rowptr || !assign) return fail(ctx, EP_ERR_INVALID_ARG, "null pointer");
    if (!aligned(rowptr, rowptr_is_int64 ? 8 : 4) || !aligned(assign, 4)) return fail(ctx, EP_ERR_INVALID_ARG, "misaligned pointer");
    const size_t need = balance_workspace_bytes(N, K, max_degree);
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < need)
        return fail(ctx, EP_ERR_WORKSPACE, "balance workspace: need %zu bytes, 256-byte aligned", need);
    return EP_OK;
}

int ep_migrate(ep_ctx *ctx, const void *rowptr, int32_t rowptr_is_int64, int64_t N, int32_t K, const uint8_t *member,
               int64_t capacity, int64_t max_degree, const uint32_t *rand_words, int32_t *assign, int64_t *state,
               void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!ctx) return EP_ERR_INVALID_ARG;
    int rc = balance_check_args(ctx, rowptr, rowptr_is_int64, N, K, capacity, max_degree, assign, workspace, workspace_bytes);
    if (rc != EP_OK) return rc;
    if (!rand_words || !aligned(rand_words, 4) || (state && !aligned(state, 8)))
        return fail(ctx, EP_ERR_INVALID_ARG, "rand_words is null, or a pointer is misaligned");
    DeviceGuard g(ctx->device);
    return migrate_run(ctx, rowptr, rowptr_is_int64 != 0, N, K, member, capacity, max_degree, rand_words, assign,
                       reinterpret_cast<long long *>(state), workspace, static_cast<cudaStream_t>(cuda_stream));
}

int ep_balance(ep_ctx *ctx, const void *rowptr, int32_t rowptr_is_int64, int64_t N, int32_t K, const uint8_t *member,
               int64_t capacity, int64_t max_degree, const uint32_t *rand_words, int32_t max_rounds, int32_t *assign,
               int32_t *rounds_used, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!ctx) return EP_ERR_INVALID_ARG;
    int rc = balance_check_args(ctx, rowptr, rowptr_is_int64, N, K, capacity, max_degree, assign, workspace, workspace_bytes);
    if (rc != EP_OK) return rc;
    if (max_rounds < 0 || (max_rounds > 0 && (!rand_words || !aligned(rand_words, 4))))
        return fail(ctx, EP_ERR_INVALID_ARG, "max_rounds < 0, or rand_words is null or misaligned");
    DeviceGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const long long *d_state = balance_state_ptr(N, K, max_degree, workspace);
    if (rounds_used) *rounds_used = 0;
    for (int r = 0;; ++r) {
        // after the last allowed application only the loads are looked at
        const uint32_t *words = r < max_rounds ? rand_words + (size_t)r * (size_t)N : nullptr;
        rc = migrate_run(ctx, rowptr, rowptr_is_int64 != 0, N, K, member, capacity, max_degree, words, assign, nullptr,
                         workspace, st);
        if (rc != EP_OK) return rc;
        long long state[4];
        EP_CUDA(ctx, cudaMemcpyAsync(state, d_state, sizeof(state), cudaMemcpyDeviceToHost, st));
        EP_CUDA(ctx, cudaStreamSynchronize(st));
        if (state[0] == 0) return EP_OK;                                  // no partition above its capacity
        if (state[2] < 0)
            return fail(ctx, EP_ERR_INVALID_ARG, "capacity %lld x K=%d cannot hold the vertex set", (long long)capacity, K);
        if (!words) return fail(ctx, EP_ERR_UNSUPPORTED, "not balanced after %d applications of the policy", max_rounds);
        if (rounds_used) *rounds_used = r + 1;
    }
}

// ---------------------------------------------------------------------------------------------- phase 2
size_t ep_cluster_and_balance_workspace_bytes(const ep_ctx *ctx, int64_t N, int32_t d, int32_t K, int64_t max_degree) {
    const size_t km = ep_kmeans_workspace_bytes(ctx, N, d, K), bal = ep_balance_workspace_bytes(ctx, N, K, max_degree);
    if (km == 0 || bal == 0) return 0;
    Arena a(nullptr);
    a.take<uint8_t>(N);
    return a.used + std::max(km, bal);
}

int ep_cluster_and_balance(ep_ctx *ctx, const float *emb, int64_t N, int32_t d, int32_t K, int32_t iters,
                           const float *init_centroids, const void *rowptr, int32_t rowptr_is_int64, int64_t max_degree,
                           const uint8_t *split, const int64_t *capacities, const uint32_t *rand_words,
                           int32_t max_rounds, int32_t *assign, float *centroids, int32_t *rounds_used, void *workspace,
                           size_t workspace_bytes, void *cuda_stream) {
    if (!ctx) return EP_ERR_INVALID_ARG;
    if (!split || !capacities) return fail(ctx, EP_ERR_INVALID_ARG, "null pointer");
    const size_t need = ep_cluster_and_balance_workspace_bytes(ctx, N, d, K, max_degree);
    if (need == 0)
        return fail(ctx, EP_ERR_INVALID_ARG, "shape out of range or unsupported: N=%lld d=%d K=%d max_degree=%lld", (long long)N, d,
                    K, (long long)max_degree);
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < need)
        return fail(ctx, EP_ERR_WORKSPACE, "phase 2 workspace: need %zu bytes, 256-byte aligned", need);
    Arena a(workspace);
    uint8_t *mask = a.take<uint8_t>(N);
    void *ws = a.base + a.used;
    const size_t ws_bytes = workspace_bytes - a.used;
    int rc = ep_kmeans(ctx, emb, N, d, K, iters, init_centroids, assign, centroids, nullptr, ws, ws_bytes, cuda_stream);
    if (rc != EP_OK) return rc;
    DeviceGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    for (int s = 0; s < 3; ++s) {
        split_mask<<<(unsigned)ceil_div(N, 256), 256, 0, st>>>(split, N, s, mask);
        ctx->launches += 1;
        EP_CUDA(ctx, cudaGetLastError());
        int32_t used = 0;
        rc = ep_balance(ctx, rowptr, rowptr_is_int64, N, K, mask, capacities[s], max_degree,
                        rand_words ? rand_words + (size_t)s * (size_t)max_rounds * (size_t)N : nullptr, max_rounds, assign, &used,
                        ws, ws_bytes, cuda_stream);
        if (rounds_used) rounds_used[s] = used;
        if (rc != EP_OK) return rc;
    }
    return EP_OK;
}

// ---------------------------------------------------------------------------------------------- reorder
static bool reorder_shape_ok(int64_t N, int32_t K) {
    return N >= 1 && N < (int64_t(1) << 31) && K >= 1 && K <= (1 << 24);
}

size_t ep_reorder_workspace_bytes(const ep_ctx *ctx, int64_t N, int32_t K) {
    if (!ctx || !reorder_shape_ok(N, K)) return 0;
    return reorder_workspace_bytes(N, K);
}

int ep_reorder(ep_ctx *ctx, const int32_t *assign, int64_t N, int32_t K, int32_t *perm, int32_t *inv_perm,
               void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!ctx) return EP_ERR_INVALID_ARG;
    if (!reorder_shape_ok(N, K))
        return fail(ctx, EP_ERR_INVALID_ARG, "shape out of range: N=%lld K=%d", (long long)N, K);
    if (!assign || !perm) return fail(ctx, EP_ERR_INVALID_ARG, "null pointer");
    if (!aligned(assign, 4) || !aligned(perm, 4) || (inv_perm && !aligned(inv_perm, 4)))
        return fail(ctx, EP_ERR_INVALID_ARG, "misaligned pointer");
    const size_t need = reorder_workspace_bytes(N, K);
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < need)
        return fail(ctx, EP_ERR_WORKSPACE, "reorder workspace: need %zu bytes, 256-byte aligned", need);
    DeviceGuard g(ctx->device);
    return reorder_run(ctx, assign, N, K, perm, inv_perm, workspace, static_cast<cudaStream_t>(cuda_stream));
}

// ---------------------------------------------------------------------------------------------- host buffers
size_t ep_kmeans_host_arena_bytes(const ep_ctx *ctx, int64_t N, int32_t d, int32_t K, int32_t iters) {
    const size_t ws = ep_kmeans_workspace_bytes(ctx, N, d, K);
    if (ws == 0 || iters < 0) return 0;
    Arena a(nullptr);
    a.take<float>((size_t)N * d);
    a.take<float>((size_t)K * d);
    a.take<int32_t>(N);
    a.take<double>(iters > 0 ? iters : 1);
    return a.used + ws;
}

int ep_kmeans_host(ep_ctx *ctx, const float *emb, int64_t N, int32_t d, int32_t K, int32_t iters,
                   const float *init_centroids, int32_t *assign, float *centroids, double *objective, void *arena,
                   size_t arena_bytes, void *cuda_stream) {
    if (!ctx) return EP_ERR_INVALID_ARG;
    if (!emb || !init_centroids || !assign || !centroids) return fail(ctx, EP_ERR_INVALID_ARG, "null pointer");
    const size_t need = ep_kmeans_host_arena_bytes(ctx, N, d, K, iters);
    if (need == 0) return fail(ctx, EP_ERR_INVALID_ARG, "shape out of range: N=%lld d=%d K=%d", (long long)N, d, K);
    if (!arena || !aligned(arena, 256) || arena_bytes < need)
        return fail(ctx, EP_ERR_WORKSPACE, "k-means host arena: need %zu bytes, 256-byte aligned", need);
    DeviceGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    Arena a(arena);
    float *d_emb = a.take<float>((size_t)N * d);
    float *d_cent = a.take<float>((size_t)K * d);
    int32_t *d_assign = a.take<int32_t>(N);
    const int T = iters > 0 ? iters : 1;
    double *d_obj = a.take<double>(T);
    void *ws = a.base + a.used;
    EP_CUDA(ctx, cudaMemcpyAsync(d_emb, emb, sizeof(float) * N * d, cudaMemcpyHostToDevice, st));
    EP_CUDA(ctx, cudaMemcpyAsync(d_cent, init_centroids, sizeof(float) * K * d, cudaMemcpyHostToDevice, st));
    int rc = ep_kmeans(ctx, d_emb, N, d, K, iters, d_cent, d_assign, d_cent, objective ? d_obj : nullptr, ws,
                       arena_bytes - a.used, st);
    if (rc != EP_OK) return rc;
    EP_CUDA(ctx, cudaMemcpyAsync(assign, d_assign, sizeof(int32_t) * N, cudaMemcpyDeviceToHost, st));
    EP_CUDA(ctx, cudaMemcpyAsync(centroids, d_cent, sizeof(float) * K * d, cudaMemcpyDeviceToHost, st));
    if (objective) EP_CUDA(ctx, cudaMemcpyAsync(objective, d_obj, sizeof(double) * T, cudaMemcpyDeviceToHost, st));
    return EP_OK;
}

size_t ep_quality_host_arena_bytes(const ep_ctx *ctx, int64_t N, int64_t nnz, int32_t K, int32_t rowptr_is_int64) {
    const size_t ws = ep_quality_workspace_bytes(ctx, N, nnz, K);
    if (ws == 0) return 0;
    Arena a(nullptr);
    a.take<char>((size_t)(N + 1) * (rowptr_is_int64 ? 8 : 4));
    a.take<int32_t>(nnz);
    a.take<int32_t>(N);
    a.take<int64_t>(2 * (size_t)K + 1);
    return a.used + ws;
}

int ep_partition_quality_host(ep_ctx *ctx, const void *rowptr, int32_t rowptr_is_int64, const int32_t *colidx,
                              int64_t nnz, const int32_t *assign, int64_t N, int32_t K, uint64_t *edge_cut,
                              int64_t *part_vertices, int64_t *part_edges, void *arena, size_t arena_bytes,
                              void *cuda_stream) {
    if (!ctx) return EP_ERR_INVALID_ARG;
    if (!rowptr || (!colidx && nnz > 0) || !assign || !edge_cut || !part_vertices || !part_edges)
        return fail(ctx, EP_ERR_INVALID_ARG, "null pointer");
    const size_t need = ep_quality_host_arena_bytes(ctx, N, nnz, K, rowptr_is_int64);
    if (need == 0)
        return fail(ctx, EP_ERR_INVALID_ARG, "shape out of range: N=%lld nnz=%lld K=%d", (long long)N, (long long)nnz, K);
    if (!arena || !aligned(arena, 256) || arena_bytes < need)
        return fail(ctx, EP_ERR_WORKSPACE, "quality host arena: need %zu bytes, 256-byte aligned", need);
    DeviceGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    Arena a(arena);
    const size_t rp_bytes = (size_t)(N + 1) * (rowptr_is_int64 ? 8 : 4);
    char *d_rp = a.take<char>(rp_bytes);
    int32_t *d_ci = a.take<int32_t>(nnz);
    int32_t *d_as = a.take<int32_t>(N);
    int64_t *d_out = a.take<int64_t>(2 * (size_t)K + 1);      // [cut | part_vertices | part_edges]
    void *ws = a.base + a.used;
    EP_CUDA(ctx, cudaMemcpyAsync(d_rp, rowptr, rp_bytes, cudaMemcpyHostToDevice, st));
    if (nnz > 0) EP_CUDA(ctx, cudaMemcpyAsync(d_ci, colidx, sizeof(int32_t) * nnz, cudaMemcpyHostToDevice, st));
    EP_CUDA(ctx, cudaMemcpyAsync(d_as, assign, sizeof(int32_t) * N, cudaMemcpyHostToDevice, st));
    int rc = ep_partition_quality(ctx, d_rp, rowptr_is_int64, d_ci, nnz, d_as, N, K,
                                  reinterpret_cast<uint64_t *>(d_out), d_out + 1, d_out + 1 + K, ws,
                                  arena_bytes - a.used, st);
    if (rc != EP_OK) return rc;
    EP_CUDA(ctx, cudaMemcpyAsync(edge_cut, d_out, sizeof(uint64_t), cudaMemcpyDeviceToHost, st));
    EP_CUDA(ctx, cudaMemcpyAsync(part_vertices, d_out + 1, sizeof(int64_t) * K, cudaMemcpyDeviceToHost, st));
    EP_CUDA(ctx, cudaMemcpyAsync(part_edges, d_out + 1 + K, sizeof(int64_t) * K, cudaMemcpyDeviceToHost, st));
    return EP_OK;
}

size_t ep_reorder_host_arena_bytes(const ep_ctx *ctx, int64_t N, int32_t K) {
    const size_t ws = ep_reorder_workspace_bytes(ctx, N, K);
    if (ws == 0) return 0;
    Arena a(nullptr);
    a.take<int32_t>(N);
    a.take<int32_t>(N);
    a.take<int32_t>(N);
    return a.used + ws;
}

int ep_reorder_host(ep_ctx *ctx, const int32_t *assign, int64_t N, int32_t K, int32_t *perm, int32_t *inv_perm,
                    void *arena, size_t arena_bytes, void *cuda_stream) {
    if (!ctx) return EP_ERR_INVALID_ARG;
    if (!assign || !perm) return fail(ctx, EP_ERR_INVALID_ARG, "null pointer");
    const size_t need = ep_reorder_host_arena_bytes(ctx, N, K);
    if (need == 0) return fail(ctx, EP_ERR_INVALID_ARG, "shape out of range: N=%lld K=%d", (long long)N, K);
    if (!arena || !aligned(arena, 256) || arena_bytes < need)
        return fail(ctx, EP_ERR_WORKSPACE, "reorder host arena: need %zu bytes, 256-byte aligned", need);
    DeviceGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    Arena a(arena);
    int32_t *d_as = a.take<int32_t>(N);
    int32_t *d_perm = a.take<int32_t>(N);
    int32_t *d_inv = a.take<int32_t>(N);
    void *ws = a.base + a.used;
    EP_CUDA(ctx, cudaMemcpyAsync(d_as, assign, sizeof(int32_t) * N, cudaMemcpyHostToDevice, st));
    int rc = ep_reorder(ctx, d_as, N, K, d_perm, inv_perm ? d_inv : nullptr, ws, arena_bytes - a.used, st);
    if (rc != EP_OK) return rc;
    EP_CUDA(ctx, cudaMemcpyAsync(perm, d_perm, sizeof(int32_t) * N, cudaMemcpyDeviceToHost, st));
    if (inv_perm) EP_CUDA(ctx, cudaMemcpyAsync(inv_perm, d_inv, sizeof(int32_t) * N, cudaMemcpyDeviceToHost, st));
    return EP_OK;
}

// ---------------------------------------------------------------------------------------------- whole path, host buffers
struct WholeLayout {
    float *emb, *cent, *cent2;
    int32_t *assign, *assign2, *colidx, *perm, *inv;
    char *rowptr;
    int64_t *out;
    void *ws;
    size_t ws_bytes, used;
};

static bool whole_layout(const ep_ctx *ctx, int64_t N, int32_t d, int32_t K, int32_t K2, int64_t nnz, int32_t is64,
                         void *arena, WholeLayout *out) {
    const int32_t Kf = K2 > 0 ? K2 : K;
    const size_t km = ep_kmeans_workspace_bytes(ctx, N, d, K), km2 = K2 > 0 ? ep_kmeans_workspace_bytes(ctx, N, d, K2) : 1;
    const size_t qw = ep_quality_workspace_bytes(ctx, N, nnz, K), rw = ep_reorder_workspace_bytes(ctx, N, Kf);
    if (km == 0 || km2 == 0 || qw == 0 || rw == 0) return false;
    Arena a(arena);
    WholeLayout l{};
    l.emb = a.take<float>((size_t)N * d);
    l.cent = a.take<float>((size_t)K * d);
    l.cent2 = a.take<float>((size_t)std::max(K2, 1) * d);
    l.assign = a.take<int32_t>(N);
    l.assign2 = a.take<int32_t>(N);
    l.rowptr = a.take<char>((size_t)(N + 1) * (is64 ? 8 : 4));
    l.colidx = a.take<int32_t>(nnz);
    l.out = a.take<int64_t>(2 * (size_t)K + 1);
    l.perm = a.take<int32_t>(N);
    l.inv = a.take<int32_t>(N);
    l.ws_bytes = std::max(std::max(km, km2), std::max(qw, rw));
    l.ws = a.take<char>(l.ws_bytes);
    l.used = a.used;
    *out = l;
    return true;
}

size_t ep_partition_and_reorder_host_arena_bytes(const ep_ctx *ctx, int64_t N, int32_t d, int32_t K, int32_t reorder_K,
                                                 int64_t nnz, int32_t rowptr_is_int64) {
    WholeLayout l;
    if (!ctx || reorder_K < 0 || !whole_layout(ctx, N, d, K, reorder_K, nnz, rowptr_is_int64, nullptr, &l)) return 0;
    return l.used;
}

int ep_partition_and_reorder_host(ep_ctx *ctx, const float *emb, int64_t N, int32_t d, int32_t K, int32_t iters,
                                  const float *init_centroids, int32_t reorder_K, int32_t reorder_iters,
                                  const float *reorder_init, const void *rowptr, int32_t rowptr_is_int64,
                                  const int32_t *colidx, int64_t nnz, int32_t *assign, float *centroids,
                                  uint64_t *edge_cut, int64_t *part_vertices, int64_t *part_edges,
                                  int32_t *reorder_assign, int32_t *perm, int32_t *inv_perm, void *arena,
                                  size_t arena_bytes, void *cuda_stream) {
    if (!ctx) return EP_ERR_INVALID_ARG;
    if (!emb || !init_centroids || !rowptr || (!colidx && nnz > 0) || !assign || !centroids || !edge_cut ||
        !part_vertices || !part_edges || !perm || (reorder_K > 0 && !reorder_init))
        return fail(ctx, EP_ERR_INVALID_ARG, "null pointer");
    if (reorder_K < 0 || iters < 0 || reorder_iters < 0) return fail(ctx, EP_ERR_INVALID_ARG, "negative count");
    WholeLayout l;
    if (!whole_layout(ctx, N, d, K, reorder_K, nnz, rowptr_is_int64, arena, &l))
        return fail(ctx, EP_ERR_INVALID_ARG, "shape out of range: N=%lld d=%d K=%d reorder_K=%d nnz=%lld", (long long)N, d, K,
                    reorder_K, (long long)nnz);
    if (!arena || !aligned(arena, 256) || arena_bytes < l.used)
        return fail(ctx, EP_ERR_WORKSPACE, "host arena: need %zu bytes, 256-byte aligned", l.used);
    DeviceGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const size_t rp_bytes = (size_t)(N + 1) * (rowptr_is_int64 ? 8 : 4);
    // every input once
    EP_CUDA(ctx, cudaMemcpyAsync(l.emb, emb, sizeof(float) * N * d, cudaMemcpyHostToDevice, st));
    EP_CUDA(ctx, cudaMemcpyAsync(l.cent, init_centroids, sizeof(float) * K * d, cudaMemcpyHostToDevice, st));
    if (reorder_K > 0)
        EP_CUDA(ctx, cudaMemcpyAsync(l.cent2, reorder_init, sizeof(float) * reorder_K * d, cudaMemcpyHostToDevice, st));
    EP_CUDA(ctx, cudaMemcpyAsync(l.rowptr, rowptr, rp_bytes, cudaMemcpyHostToDevice, st));
    if (nnz > 0) EP_CUDA(ctx, cudaMemcpyAsync(l.colidx, colidx, sizeof(int32_t) * nnz, cudaMemcpyHostToDevice, st));
    // the partition and its score
    int rc = ep_kmeans(ctx, l.emb, N, d, K, iters, l.cent, l.assign, l.cent, nullptr, l.ws, l.ws_bytes, st);
    if (rc != EP_OK) return rc;
    EP_CUDA(ctx, cudaMemcpyAsync(assign, l.assign, sizeof(int32_t) * N, cudaMemcpyDeviceToHost, st));
    EP_CUDA(ctx, cudaMemcpyAsync(centroids, l.cent, sizeof(float) * K * d, cudaMemcpyDeviceToHost, st));
    rc = ep_partition_quality(ctx, l.rowptr, rowptr_is_int64, l.colidx, nnz, l.assign, N, K, reinterpret_cast<uint64_t *>(l.out),
                              l.out + 1, l.out + 1 + K, l.ws, l.ws_bytes, st);
    if (rc != EP_OK) return rc;
    EP_CUDA(ctx, cudaMemcpyAsync(edge_cut, l.out, sizeof(uint64_t), cudaMemcpyDeviceToHost, st));
    EP_CUDA(ctx, cudaMemcpyAsync(part_vertices, l.out + 1, sizeof(int64_t) * K, cudaMemcpyDeviceToHost, st));
    EP_CUDA(ctx, cudaMemcpyAsync(part_edges, l.out + 1 + K, sizeof(int64_t) * K, cudaMemcpyDeviceToHost, st));
    // the numbering: the clusters of a second, finer run when one is asked for, else the partitions themselves
    const int32_t *fine = l.assign;
    int32_t fineK = K;
    if (reorder_K > 0) {
        rc = ep_kmeans(ctx, l.emb, N, d, reorder_K, reorder_iters, l.cent2, l.assign2, l.cent2, nullptr, l.ws, l.ws_bytes, st);
        if (rc != EP_OK) return rc;
        if (reorder_assign)
            EP_CUDA(ctx, cudaMemcpyAsync(reorder_assign, l.assign2, sizeof(int32_t) * N, cudaMemcpyDeviceToHost, st));
        fine = l.assign2;
        fineK = reorder_K;
    }
    rc = ep_reorder(ctx, fine, N, fineK, l.perm, inv_perm ? l.inv : nullptr, l.ws, l.ws_bytes, st);
    if (rc != EP_OK) return rc;
    EP_CUDA(ctx, cudaMemcpyAsync(perm, l.perm, sizeof(int32_t) * N, cudaMemcpyDeviceToHost, st));
    if (inv_perm) EP_CUDA(ctx, cudaMemcpyAsync(inv_perm, l.inv, sizeof(int32_t) * N, cudaMemcpyDeviceToHost, st));
    return EP_OK;
}

}  // extern "C"
