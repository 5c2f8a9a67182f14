// The graph and the embedding rows stored under a new numbering (Section 4.5.1: the ids of the vertices are
// their positions in memory, and reordering relabels them).
//
// Row i of the new graph is row perm[i] of the old one with every column id u replaced by inv_perm[u]; the
// entries of a row keep their stored order.  Three steps: the new row lengths (a gather of the old ones), their
// prefix sum (tiles of 2048 lengths, a scan of the tile totals in one block, and the add-back), and the copy of
// the rows (a warp per row, rows of 4096 entries or more by a whole block) with the column ids sent through
// inv_perm.  Only integers move, so the output does not depend on the schedule.
#include "ep_common.cuh"

#include <algorithm>

namespace {

constexpr int RL_THREADS = 256;
constexpr int RL_PER_THREAD = 8;
constexpr int RL_TILE = RL_THREADS * RL_PER_THREAD;         // lengths per scan tile
constexpr int RL_LONG_ROW = 4096;                           // rows at least this long are left to whole blocks
constexpr unsigned FULL = 0xffffffffu;

// len[i] = length of old row perm[i] (0 and a status when perm[i] is outside [0, N) or the row pointer steps back).
template <typename RowT>
__global__ void __launch_bounds__(256) relabel_lengths(const RowT *__restrict__ rowptr, const int32_t *__restrict__ perm,
                                                       int64_t N, int64_t nnz, RowT *__restrict__ new_rowptr,
                                                       int *status) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) {
        new_rowptr[0] = 0;
        if ((int64_t)rowptr[0] != 0 || (int64_t)rowptr[N] != nnz) ep_raise(status, EP_ERR_BAD_INDEX);
    }
    if (i >= N) return;
    const int v = perm[i];
    int64_t len = 0;
    if ((unsigned)v < (unsigned)N) {
        len = (int64_t)rowptr[v + 1] - (int64_t)rowptr[v];
        if (len < 0) {
            ep_raise(status, EP_ERR_BAD_INDEX);
            len = 0;
        }
    } else {
        ep_raise(status, EP_ERR_BAD_INDEX);
    }
    new_rowptr[i + 1] = (RowT)len;
}

// In-place inclusive scan of data[0, n) inside tiles of RL_TILE; totals[t] = sum of tile t.
template <typename RowT>
__global__ void __launch_bounds__(RL_THREADS) relabel_scan_tiles(RowT *data, int64_t n, int64_t *totals) {
    __shared__ int64_t warp_sum[RL_THREADS / 32];
    const int64_t base = (int64_t)blockIdx.x * RL_TILE + (int64_t)threadIdx.x * RL_PER_THREAD;
    int64_t v[RL_PER_THREAD];
    int64_t run = 0;
#pragma unroll
    for (int j = 0; j < RL_PER_THREAD; ++j) {
        run += base + j < n ? (int64_t)data[base + j] : 0;
        v[j] = run;
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int64_t inc = run;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int64_t t = __shfl_up_sync(FULL, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) warp_sum[warp] = inc;
    __syncthreads();
    int64_t before = inc - run;                             // sum of the lanes before this one in the warp
    for (int w = 0; w < warp; ++w) before += warp_sum[w];
#pragma unroll
    for (int j = 0; j < RL_PER_THREAD; ++j)
        if (base + j < n) data[base + j] = (RowT)(v[j] + before);
    if (threadIdx.x == RL_THREADS - 1) totals[blockIdx.x] = before + run;
}

// totals[t] <- sum of totals[0, t) (one block, any number of tiles).
__global__ void __launch_bounds__(RL_THREADS) relabel_scan_totals(int64_t *totals, int64_t ntiles) {
    __shared__ int64_t warp_sum[RL_THREADS / 32];
    __shared__ int64_t carry_s;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    for (int64_t t0 = 0; t0 < ntiles; t0 += RL_THREADS) {
        const int64_t t = t0 + threadIdx.x;
        const int64_t mine = t < ntiles ? totals[t] : 0;
        int64_t inc = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int64_t u = __shfl_up_sync(FULL, inc, o);
            if (lane >= o) inc += u;
        }
        if (lane == 31) warp_sum[warp] = inc;
        __syncthreads();
        int64_t before = carry_s + inc - mine;
        for (int w = 0; w < warp; ++w) before += warp_sum[w];
        if (t < ntiles) totals[t] = before;
        __syncthreads();
        if (threadIdx.x == RL_THREADS - 1) carry_s = before + mine;
        __syncthreads();
    }
}

template <typename RowT>
__global__ void __launch_bounds__(RL_THREADS) relabel_scan_add(RowT *data, int64_t n, const int64_t *__restrict__ totals) {
    const int64_t add = totals[blockIdx.x];
    if (add == 0) return;
    const int64_t base = (int64_t)blockIdx.x * RL_TILE;
    for (int j = threadIdx.x; j < RL_TILE; j += RL_THREADS)
        if (base + j < n) data[base + j] = (RowT)((int64_t)data[base + j] + add);
}

// Copies old row perm[i] to new row i, ids mapped through inv_perm.  A warp takes the rows shorter than
// RL_LONG_ROW; the others are listed for relabel_long_rows.
template <typename RowT>
__global__ void __launch_bounds__(256) relabel_rows(const RowT *__restrict__ rowptr, const int32_t *__restrict__ colidx,
                                                    const int32_t *__restrict__ perm, const int32_t *__restrict__ inv_perm,
                                                    int64_t N, const RowT *__restrict__ new_rowptr,
                                                    int32_t *__restrict__ new_colidx, int32_t *long_rows, int *n_long,
                                                    int *status) {
    const int lane = threadIdx.x & 31;
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    unsigned bad = 0;
    for (int64_t i = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); i < N; i += warps) {
        const int v = perm[i];
        if ((unsigned)v >= (unsigned)N) continue;           // reported by relabel_lengths; its new row is empty
        const int64_t src = (int64_t)rowptr[v], len = (int64_t)rowptr[v + 1] - src, dst = (int64_t)new_rowptr[i];
        if (len >= RL_LONG_ROW) {
            if (lane == 0) long_rows[atomicAdd(n_long, 1)] = (int32_t)i;
            continue;
        }
        for (int64_t e = lane; e < len; e += 32) {
            const int u = colidx[src + e];
            const bool in = (unsigned)u < (unsigned)N;
            bad |= in ? 0u : 1u;
            new_colidx[dst + e] = in ? __ldg(inv_perm + u) : 0;   // an id outside [0, N) is reported and stored as 0
        }
    }
    if (bad) ep_raise(status, EP_ERR_BAD_INDEX);
}

template <typename RowT>
__global__ void __launch_bounds__(256) relabel_long_rows(const RowT *__restrict__ rowptr, const int32_t *__restrict__ colidx,
                                                         const int32_t *__restrict__ perm,
                                                         const int32_t *__restrict__ inv_perm, int64_t N,
                                                         const RowT *__restrict__ new_rowptr,
                                                         int32_t *__restrict__ new_colidx,
                                                         const int32_t *__restrict__ long_rows,
                                                         const int *__restrict__ n_long, int *status) {
    const int n = *n_long;
    unsigned bad = 0;
    for (int r = blockIdx.y; r < n; r += gridDim.y) {       // blockIdx.x splits a row, blockIdx.y walks the list
        const int64_t i = long_rows[r];
        const int v = perm[i];
        const int64_t src = (int64_t)rowptr[v], len = (int64_t)rowptr[v + 1] - src, dst = (int64_t)new_rowptr[i];
        for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < len; e += (int64_t)gridDim.x * blockDim.x) {
            const int u = colidx[src + e];
            const bool in = (unsigned)u < (unsigned)N;
            bad |= in ? 0u : 1u;
            new_colidx[dst + e] = in ? __ldg(inv_perm + u) : 0;
        }
    }
    if (bad) ep_raise(status, EP_ERR_BAD_INDEX);
}

// out[i] = emb[perm[i]]: a warp per row, 16 bytes per lane and step.
__global__ void __launch_bounds__(256) permute_rows_kernel(const float *__restrict__ emb, int64_t N, int d4,
                                                           const int32_t *__restrict__ perm, float *__restrict__ out,
                                                           int *status) {
    const int lane = threadIdx.x & 31;
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    for (int64_t i = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); i < N; i += warps) {
        int v = perm[i];
        if ((unsigned)v >= (unsigned)N) {
            if (lane == 0) ep_raise(status, EP_ERR_BAD_INDEX);
            v = 0;
        }
        const float4 *src = reinterpret_cast<const float4 *>(emb) + (int64_t)v * d4;
        float4 *dst = reinterpret_cast<float4 *>(out) + i * d4;
        for (int q = lane; q < d4; q += 32) __stcs(dst + q, __ldcs(src + q));
    }
}

}  // namespace

namespace ep {

struct RelabelBuffers {
    int64_t *totals;
    int32_t *long_rows;
    int *n_long;
};

static size_t relabel_layout(int64_t N, int64_t nnz, void *ws, RelabelBuffers *out) {
    Arena a(ws);
    RelabelBuffers b{};
    b.totals = a.take<int64_t>(ceil_div(N, RL_TILE));
    b.long_rows = a.take<int32_t>(std::min<int64_t>(N, nnz / RL_LONG_ROW + 1));
    b.n_long = a.take<int>(1);
    if (out) *out = b;
    return a.used;
}

size_t relabel_workspace_bytes(int64_t N, int64_t nnz) { return relabel_layout(N, nnz, nullptr, nullptr); }

template <typename RowT>
static int relabel_launch(ep_ctx *ctx, const RowT *rowptr, const int32_t *colidx, int64_t nnz, const int32_t *perm,
                          const int32_t *inv_perm, int64_t N, RowT *new_rowptr, int32_t *new_colidx,
                          const RelabelBuffers &b, cudaStream_t stream) {
    Timed tm(ctx, stream, EP_TIMER_RELABEL);
    EP_CUDA(ctx, cudaMemsetAsync(b.n_long, 0, sizeof(int), stream));
    const unsigned nblk = (unsigned)ceil_div(N, 256);
    const unsigned ntiles = (unsigned)ceil_div(N, RL_TILE);
    relabel_lengths<RowT><<<nblk, 256, 0, stream>>>(rowptr, perm, N, nnz, new_rowptr, ctx->d_status);
    relabel_scan_tiles<RowT><<<ntiles, RL_THREADS, 0, stream>>>(new_rowptr + 1, N, b.totals);
    relabel_scan_totals<<<1, RL_THREADS, 0, stream>>>(b.totals, ntiles);
    relabel_scan_add<RowT><<<ntiles, RL_THREADS, 0, stream>>>(new_rowptr + 1, N, b.totals);
    int kernels = 4;
    if (nnz > 0) {
        const int grid = (int)std::max<int64_t>(1, std::min<int64_t>((int64_t)ctx->sm_count * 8, ceil_div(N, 8)));
        relabel_rows<RowT><<<grid, 256, 0, stream>>>(rowptr, colidx, perm, inv_perm, N, new_rowptr, new_colidx, b.long_rows,
                                                    b.n_long, ctx->d_status);
        relabel_long_rows<RowT><<<dim3(16, (unsigned)ctx->sm_count), 256, 0, stream>>>(
            rowptr, colidx, perm, inv_perm, N, new_rowptr, new_colidx, b.long_rows, b.n_long, ctx->d_status);
        kernels += 2;
    }
    tm.end(kernels);
    EP_CUDA(ctx, cudaGetLastError());
    return EP_OK;
}

int relabel_run(ep_ctx *ctx, const void *rowptr, bool rowptr64, const int32_t *colidx, int64_t nnz, const int32_t *perm,
                const int32_t *inv_perm, int64_t N, void *new_rowptr, int32_t *new_colidx, void *workspace,
                cudaStream_t stream) {
    RelabelBuffers b;
    relabel_layout(N, nnz, workspace, &b);
    if (rowptr64)
        return relabel_launch<int64_t>(ctx, static_cast<const int64_t *>(rowptr), colidx, nnz, perm, inv_perm, N,
                                       static_cast<int64_t *>(new_rowptr), new_colidx, b, stream);
    return relabel_launch<int32_t>(ctx, static_cast<const int32_t *>(rowptr), colidx, nnz, perm, inv_perm, N,
                                   static_cast<int32_t *>(new_rowptr), new_colidx, b, stream);
}

int permute_rows_run(ep_ctx *ctx, const float *emb, int64_t N, int d, const int32_t *perm, float *out,
                     cudaStream_t stream) {
    Timed tm(ctx, stream, EP_TIMER_RELABEL);
    const int grid = (int)std::max<int64_t>(1, std::min<int64_t>((int64_t)ctx->sm_count * 8, ceil_div(N, 8)));
    permute_rows_kernel<<<grid, 256, 0, stream>>>(emb, N, d >> 2, perm, out, ctx->d_status);
    tm.end(1);
    EP_CUDA(ctx, cudaGetLastError());
    return EP_OK;
}

}  // namespace ep
