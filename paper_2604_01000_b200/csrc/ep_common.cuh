// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

#include <vector>

#include "embedpart.h"

struct ep_timed_interval {
    int timer;
    cudaEvent_t start, stop;
};

struct ep_ctx {
    int device;
    int sm_count;
    int smem_optin;        // max dynamic shared memory per block (opt-in), bytes
    int *d_status;         // device status word (max of EP_ERR_* raised by kernels)
    int opt_kmeans_path;   // EP_OPT_KMEANS_PATH
    int opt_profile;       // EP_OPT_PROFILE
    int opt_timer_group;   // EP_OPT_TIMER_GROUP
    int opt_cand_mb;       // EP_OPT_KMEANS_CAND_MB
    int opt_slice_kb;      // EP_OPT_QUALITY_SLICE_KB
    int opt_iters_per_launch;   // EP_OPT_KMEANS_ITERATIONS_PER_LAUNCH
    long long launches;    // kernels launched through this context
    unsigned long long probe_tex = 0;   // texture object of ep_probe_gather's last table (0: none), kept so that the call
    const void *probe_tex_ptr = nullptr;   // stays asynchronous; replaced when another table or size comes
    long long probe_tex_n = 0;
    std::vector<ep_timed_interval> intervals;   // pending event pairs (profile mode)
    std::vector<cudaEvent_t> spare_events;
    char last_error[256];
};

// The 256-byte device block behind ep_ctx::d_status: word 0 is the status, the 64-bit diagnostic
// counters start at this 32-bit word.
constexpr int EP_COUNTER_WORD0 = 16;
constexpr int EP_COUNTERS = 8;

namespace ep {

// ---- host helpers ---------------------------------------------------------------------------
int fail(ep_ctx *ctx, int status, const char *fmt, ...);
int cuda_fail(ep_ctx *ctx, cudaError_t e, const char *what);

#define EP_CUDA(ctx, call)                                                   \
    do {                                                                     \
        cudaError_t _e = (call);                                             \
        if (_e != cudaSuccess) return ep::cuda_fail((ctx), _e, #call);      \
    } while (0)

// Makes the context's device current for the lifetime of the object.
struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) switched = (cudaSetDevice(dev) == cudaSuccess);
    }
    ~DeviceGuard() {
        if (switched) cudaSetDevice(prev);
    }
};

// Bump allocator over the caller's workspace; every block is 256-byte aligned.
struct Arena {
    char *base;
    size_t used;
    explicit Arena(void *p) : base(static_cast<char *>(p)), used(0) {}
    template <typename T>
    T *take(size_t count) {
        size_t bytes = (count * sizeof(T) + 255) & ~size_t(255);
        T *p = base ? reinterpret_cast<T *>(base + used) : nullptr;
        used += bytes;
        return p;
    }
};

// Brackets a region of stream work with CUDA events when profiling is on; counts its kernels always.
struct Timed {
    ep_ctx *ctx;
    cudaStream_t stream;
    int timer;
    cudaEvent_t start = nullptr;
    Timed(ep_ctx *c, cudaStream_t s, int t);
    void end(int kernels);   // records the stop event and adds `kernels` to the launch counter
};

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// ---- k-means (kmeans_simt.cu) ------------------------------------------------------------------
struct KMeansPlan {
    int64_t N;
    int d, K;
    bool fused;        // centroids + per-warp sums live in shared memory, one pass per iteration
    bool tensor;       // labels come from the tcgen05 screening kernel + fp32 resolve kernel
    bool tc_fused;     // few centroids: one tcgen05 kernel assigns and accumulates (implies tensor)
    int warps;         // warps per block of the assign kernel
    int grid;          // blocks of the assign kernel (fused: also the number of partial sums)
    int parts;         // partial-sum slabs the update kernel reduces (fused: grid; otherwise splits per cluster)
    size_t smem;       // dynamic shared memory of the assign kernel
};
bool kmeans_make_plan(const ep_ctx *ctx, int64_t N, int d, int K, KMeansPlan *plan);
size_t kmeans_workspace_layout(const ep_ctx *ctx, const KMeansPlan &plan, void *workspace, struct KMeansBuffers *out);
int kmeans_run(ep_ctx *ctx, const KMeansPlan &plan, const float *emb, int iters, const float *init,
               int32_t *assign, float *centroids, double *objective, void *workspace, cudaStream_t stream);

// ---- k-means on the tensor cores (kmeans_tc.cu) --------------------------------------------------
struct TcState;                                   // tensor maps of one ep_kmeans call
// Tensor map (128-byte swizzle) over a row-major [rows x d] fp32 matrix with boxes of box_rows x 32 floats;
// `map` points at a CUtensorMap.
bool tc_encode_kblock_map(void *map, const float *base, int64_t rows, int d, int box_rows);
bool tc_encode_rowtile_map(void *map, const float *base, int64_t rows, int d, int box_rows);
bool kmeans_tc_shape_ok(const ep_ctx *ctx, int d, int K);
size_t kmeans_tc_state_bytes();
size_t kmeans_tc_cand_bytes(const ep_ctx *ctx, int64_t N, int K);
int kmeans_tc_prepare(ep_ctx *ctx, const float *emb, int64_t N, int d, int K, const float *centroids, TcState *st);
int kmeans_tc_assign(ep_ctx *ctx, const TcState &st, const float *emb, int64_t N, int d, int K, const float *centroids,
                     const float *cn, const float *clo, float *cmaxima, const float2 *rownorm, int32_t *assign,
                     void *cand_ws, cudaStream_t stream);

// ---- fused tensor-core pass for few centroids (kmeans_tc_fused.cu) --------------------------------
struct TcFusedState;
bool kmeans_tcf_shape_ok(const ep_ctx *ctx, int d, int K);
size_t kmeans_tcf_state_bytes();
int kmeans_tcf_grid(const ep_ctx *ctx, int64_t N, int d);
int64_t kmeans_tcf_late_cap(const ep_ctx *ctx, int64_t N, int d);
int kmeans_row_norms(ep_ctx *ctx, const float *emb, int64_t N, int d, float2 *rownorm, cudaStream_t stream);
int kmeans_tcf_prepare(ep_ctx *ctx, const float *emb, int64_t N, int d, int K, const float *ct, TcFusedState *st);
int kmeans_tcf_run(ep_ctx *ctx, const TcFusedState &st, const float *emb, float *centroids, float *cn, float *ct, float *clo,
                   const float2 *rownorm, int64_t N, int d, int K, int32_t *assign, float *psum, int *pcnt, void *late_list,
                   int T, bool update_here, bool use_prev0, bool keep_centroids, double *objterm, double *objective,
                   const double *x2part, int x2n, unsigned *grid_bar, cudaStream_t stream);

// ---- reorder (reorder.cu) -----------------------------------------------------------------------
size_t reorder_workspace_bytes(int64_t N, int K);
// Stable sort of vertex ids by label.  timed = false when a caller brackets the call itself.
int reorder_run(ep_ctx *ctx, const int32_t *assign, int64_t N, int K, int32_t *perm, int32_t *inv_perm,
                void *workspace, cudaStream_t stream, bool timed = true);

// ---- quality (quality.cu) -----------------------------------------------------------------------
size_t quality_workspace_bytes(int64_t N, int64_t nnz, int K);
int quality_run(ep_ctx *ctx, const void *rowptr, bool rowptr64, const int32_t *colidx, int64_t nnz,
                const int32_t *assign, int64_t N, int K, unsigned long long *edge_cut, long long *part_vertices,
                long long *part_edges, void *workspace, cudaStream_t stream);

// ---- graph bandwidth (bandwidth.cu) -------------------------------------------------------------
size_t bandwidth_workspace_bytes(int64_t N, int64_t nnz);
int bandwidth_run(ep_ctx *ctx, const void *rowptr, bool rowptr64, const int32_t *colidx, int64_t nnz,
                  const int32_t *pi, int64_t N, unsigned long long *total, int32_t *vertex_bandwidth, void *workspace,
                  cudaStream_t stream);

// ---- the graph under a new numbering (relabel.cu) -------------------------------------------------
size_t relabel_workspace_bytes(int64_t N, int64_t nnz);
int relabel_run(ep_ctx *ctx, const void *rowptr, bool rowptr64, const int32_t *colidx, int64_t nnz, const int32_t *perm,
                const int32_t *inv_perm, int64_t N, void *new_rowptr, int32_t *new_colidx, void *workspace,
                cudaStream_t stream);
int permute_rows_run(ep_ctx *ctx, const float *emb, int64_t N, int d, const int32_t *perm, float *out,
                     cudaStream_t stream);

// ---- migration policy and balancing loop (balance.cu) ----------------------------------------------
bool balance_shape_ok(int64_t N, int K, int64_t max_degree);
size_t balance_workspace_bytes(int64_t N, int K, int64_t max_degree);
int migrate_run(ep_ctx *ctx, const void *rowptr, bool rowptr64, int64_t N, int K, const uint8_t *member, int64_t capacity,
                int64_t max_degree, const uint32_t *rand_words, int32_t *assign, long long *state_out, void *workspace,
                cudaStream_t stream);
const long long *balance_state_ptr(int64_t N, int K, int64_t max_degree, void *workspace);

}  // namespace ep

// ---- device helpers -------------------------------------------------------------------------------
__device__ __forceinline__ void ep_raise(int *status, int code) { atomicMax(status, code); }

// The bounds-checked build (-DEP_DEBUG: `EP_DEBUG=1 python -m paper_2604_01000_b200.build`, library
// libembedpart_debug.so): an index the kernels compute themselves (a scatter destination, a slot of a list, a row
// taken from a list) is tested before it is used; one that lies outside its array raises EP_ERR_CUDA in the status
// word and the access is skipped, so that a wrong index shows up as a status, never as a fault.  In the ordinary
// build the test is the constant true and costs nothing.
#ifdef EP_DEBUG
__device__ __forceinline__ bool ep_index_ok(long long i, long long n, int *status) {
    if (i >= 0 && i < n) return true;
    ep_raise(status, EP_ERR_CUDA);
    return false;
}
#define EP_INDEX_OK(i, n, status) ep_index_ok((long long)(i), (long long)(n), (status))
#else
#define EP_INDEX_OK(i, n, status) true
#endif
