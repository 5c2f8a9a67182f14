// Vertex bandwidths and their sum for a vertex numbering (Section 4.5.1, Eq. 3, Eq. 4 and Eq. 5) over a CSR graph.
//
// Like the edge-cut pass the work is split by EDGES: a block takes tiles of BW_EDGES consecutive CSR entries,
// streams their column ids with 16-byte loads and recovers the source row of each entry from a bitmap of row
// starts in shared memory.  What differs is the reduction: the gap |pi(v) - pi(u)| of an entry is folded into a
// maximum per ROW.  Inside a tile every row segment has a slot in shared memory (slot 0 for the row that straddles
// the tile start, slot h + 1 for the row whose first entry is at position h); a thread folds its four entries in
// registers, lanes of a warp that hold the same segment combine with match_any + a warp max, and one lane per
// segment issues the shared-memory atomic.  Segments leave the tile with one global atomicMax per row and tile
// (rows longer than a tile meet in global memory), and a last kernel adds the N vertex bandwidths.  Integer
// maxima and sums only: the result does not depend on the schedule.
#include "ep_common.cuh"

#include <algorithm>

namespace {

constexpr int BW_THREADS = 256;
constexpr int BW_VEC = 4;                                   // 16-byte loads per thread per tile
constexpr int BW_EDGES = BW_THREADS * BW_VEC * 4;           // 4096 entries per tile: 33 KB of shared memory, 5 blocks per SM
constexpr int BW_WORDS = BW_EDGES / 32;                     // 128 bitmap words, one per thread of the first four warps
constexpr unsigned FULL = 0xffffffffu;

// tile_row[t] = last row r in [0, N) whose first entry is at or before t * BW_EDGES; tile_row[ntiles] = N-1.
template <typename RowT>
__global__ void bandwidth_tile_rows(const RowT *__restrict__ rowptr, int64_t N, int64_t ntiles, int32_t *tile_row) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t > ntiles) return;
    if (t == ntiles) {
        tile_row[t] = (int32_t)(N - 1);
        return;
    }
    const int64_t e = t * BW_EDGES;
    int64_t lo = 0, hi = N - 1;                             // rowptr[0] = 0 <= e always
    while (lo < hi) {
        const int64_t mid = (lo + hi + 1) >> 1;
        if ((int64_t)rowptr[mid] <= e)
            lo = mid;
        else
            hi = mid - 1;
    }
    tile_row[t] = (int32_t)lo;
}

// Checks the row pointer the way the edge-cut pre-pass does (first and last value, no step backwards).
template <typename RowT>
__global__ void bandwidth_check_rows(const RowT *__restrict__ rowptr, int64_t N, int64_t nnz, int *status) {
    const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (v == 0 && ((int64_t)rowptr[0] != 0 || (int64_t)rowptr[N] != nnz)) ep_raise(status, EP_ERR_BAD_INDEX);
    if (v < N && (int64_t)rowptr[v + 1] < (int64_t)rowptr[v]) ep_raise(status, EP_ERR_BAD_INDEX);
}

template <typename RowT>
__global__ void __launch_bounds__(BW_THREADS, 5)
    vertex_bandwidth_tiles(const RowT *__restrict__ rowptr, const int32_t *__restrict__ colidx, int64_t nnz,
                           const int32_t *__restrict__ pi, int64_t N, const int32_t *__restrict__ tile_row,
                           int64_t ntiles, int32_t *vb, int *status) {
    __shared__ unsigned bitmap[BW_WORDS];
    __shared__ int lasthead[BW_WORDS];
    __shared__ int warp_max[BW_THREADS / 32];
    extern __shared__ __align__(16) int bw_dyn[];
    int32_t *headpi = bw_dyn;                               // [BW_EDGES] pi of the row that starts at this position
    int *segmax = bw_dyn + BW_EDGES;                        // [BW_EDGES + 1] largest gap per row segment of the tile
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const int64_t e0 = tile * BW_EDGES;
        const int ne = (int)min((int64_t)BW_EDGES, nnz - e0);
        const int4 *src = reinterpret_cast<const int4 *>(colidx + e0);
        int4 c[BW_VEC];                                     // this tile's column ids: they depend on nothing below
#pragma unroll
        for (int i = 0; i < BW_VEC; ++i) {
            const int q = (i * BW_THREADS + tid) * 4;
            if (q + 3 < ne) {
                c[i] = __ldcs(src + (q >> 2));
            } else {
                c[i].x = q + 0 < ne ? colidx[e0 + q + 0] : 0;
                c[i].y = q + 1 < ne ? colidx[e0 + q + 1] : 0;
                c[i].z = q + 2 < ne ? colidx[e0 + q + 2] : 0;
                c[i].w = 0;
            }
        }
        __syncthreads();                                    // previous tile fully written back
        if (tid < BW_WORDS) bitmap[tid] = 0u;
        if (tid == 0) segmax[0] = 0;
        __syncthreads();
        const int64_t r_lo = tile_row[tile], r_hi = tile_row[tile + 1];
        const int32_t carry_pi = pi[r_lo];
        for (int64_t r = r_lo + tid; r <= r_hi; r += BW_THREADS) {
            const int64_t s = (int64_t)rowptr[r], e = (int64_t)rowptr[r + 1];
            const int64_t h = s - e0;
            if (e > s && h >= 0 && h < ne) {
                atomicOr(&bitmap[h >> 5], 1u << (h & 31));
                headpi[h] = pi[r];
                segmax[h + 1] = 0;                          // only the slots of row starts are ever used
            }
        }
        __syncthreads();
        {   // lasthead[w] = position of the last set bit in words < w, or -1
            const unsigned wbits = tid < BW_WORDS ? bitmap[tid] : 0u;
            const int mine = wbits ? tid * 32 + 31 - __clz(wbits) : -1;
            int inc = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(FULL, inc, o);
                if (lane >= o) inc = max(inc, t);
            }
            if (lane == 31) warp_max[warp] = inc;
            int excl = __shfl_up_sync(FULL, inc, 1);
            if (lane == 0) excl = -1;
            __syncthreads();
            for (int w = 0; w < warp; ++w) excl = max(excl, warp_max[w]);
            if (tid < BW_WORDS) lasthead[tid] = excl;
        }
        __syncthreads();
        unsigned bad = 0;
        unsigned top = 0u;                                   // largest column id of this thread, as unsigned
#pragma unroll
        for (int i = 0; i < BW_VEC; ++i)
            top = max(max(max(top, (unsigned)c[i].x), max((unsigned)c[i].y, (unsigned)c[i].z)), (unsigned)c[i].w);
        // every lane's ids in range and the tile full: the warp may skip the per-entry range and length tests
        const bool clean = __all_sync(FULL, ne == BW_EDGES && top < (unsigned)N);
        // first every vector's gathers and maxima (nothing between them that would keep the loads apart) ...
        int segs[BW_VEC], maxs[BW_VEC];
#pragma unroll
        for (int i = 0; i < BW_VEC; ++i) {
            const int q = (i * BW_THREADS + tid) * 4;
            const int wd = q >> 5, b = q & 31;
            const unsigned bits = bitmap[wd];
            const unsigned upto = bits & (0xffffffffu >> (31 - b));
            int seg = upto ? (wd << 5) + 31 - __clz(upto) : lasthead[wd];      // -1: the straddling row
            int32_t from = seg >= 0 ? headpi[seg] : carry_pi;
            int m = 0;
            const int cols[4] = {c[i].x, c[i].y, c[i].z, c[i].w};
            if (clean && ((bits >> b) & 0xEu) == 0u) {      // four entries of one row
                m = max(max(abs(from - __ldg(pi + cols[0])), abs(from - __ldg(pi + cols[1]))),
                        max(abs(from - __ldg(pi + cols[2])), abs(from - __ldg(pi + cols[3]))));
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (j > 0 && ((bits >> (b + j)) & 1u)) {    // a row starts inside the vector: close the segment
                        if (m > 0) atomicMax(&segmax[seg + 1], m);
                        seg = q + j;
                        from = headpi[seg];
                        m = 0;
                    }
                    const bool live = q + j < ne;
                    const int col = cols[j];
                    const bool in = (unsigned)col < (unsigned)N;
                    const int32_t to = __ldg(pi + (in ? col : 0));   // an index outside [0, N) is reported, never followed
                    const int gap = abs(from - to);
                    m = (live && in) ? max(m, gap) : m;
                    bad |= (live && !in) ? 1u : 0u;
                }
            }
            segs[i] = q >= ne ? -2 : seg;                    // -2: nothing of this vector is in the tile
            maxs[i] = m;
        }
        // ... then, vector by vector (the whole warp takes each), lanes that end in the same segment combine and
        // one of them issues the shared-memory atomic
#pragma unroll
        for (int i = 0; i < BW_VEC; ++i) {
            const int seg = segs[i], m = maxs[i];
            if (__all_sync(FULL, seg == __shfl_sync(FULL, seg, 0))) {
                const int best = (int)__reduce_max_sync(FULL, (unsigned)m);
                if (lane == 0 && seg >= -1 && best > 0) atomicMax(&segmax[seg + 1], best);
            } else {
                const unsigned peers = __match_any_sync(FULL, seg);
                const int best = (int)__reduce_max_sync(peers, (unsigned)m);
                if (seg >= -1 && best > 0 && lane == __ffs(peers) - 1) atomicMax(&segmax[seg + 1], best);
            }
        }
        if (bad) ep_raise(status, EP_ERR_BAD_INDEX);
        __syncthreads();
        // one atomic per row and tile: rows longer than a tile, or cut by its edge, meet in global memory
        if (tid == 0 && segmax[0] > 0) atomicMax(&vb[r_lo], segmax[0]);
        for (int64_t r = r_lo + tid; r <= r_hi; r += BW_THREADS) {
            const int64_t s = (int64_t)rowptr[r], e = (int64_t)rowptr[r + 1];
            const int64_t h = s - e0;
            if (e > s && h >= 0 && h < ne) {
                const int v = segmax[h + 1];
                if (v > 0) atomicMax(&vb[r], v);
            }
        }
    }
}

__global__ void __launch_bounds__(256) bandwidth_total(const int32_t *__restrict__ vb, int64_t N,
                                                       unsigned long long *total) {
    __shared__ unsigned long long part[8];
    unsigned long long t = 0;
    for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < N; v += (int64_t)gridDim.x * blockDim.x)
        t += (unsigned long long)vb[v];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(FULL, t, o);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = t;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long s = 0;
        for (int w = 0; w < 8; ++w) s += part[w];
        if (s) atomicAdd(total, s);
    }
}

}  // namespace

namespace ep {

struct BandwidthBuffers {
    int32_t *tile_row;
    int32_t *vb;
};

static size_t bandwidth_layout(int64_t N, int64_t nnz, void *ws, BandwidthBuffers *out) {
    Arena a(ws);
    BandwidthBuffers b{};
    b.tile_row = a.take<int32_t>(ceil_div(nnz, BW_EDGES) + 1);
    b.vb = a.take<int32_t>(N);                              // used when the caller does not ask for the per-vertex values
    if (out) *out = b;
    return a.used;
}

size_t bandwidth_workspace_bytes(int64_t N, int64_t nnz) { return bandwidth_layout(N, nnz, nullptr, nullptr); }

template <typename RowT>
static int bandwidth_launch(ep_ctx *ctx, const RowT *rowptr, const int32_t *colidx, int64_t nnz, const int32_t *pi,
                            int64_t N, unsigned long long *total, int32_t *vb, const BandwidthBuffers &b,
                            cudaStream_t stream) {
    const int64_t ntiles = ceil_div(nnz, BW_EDGES);
    Timed tm(ctx, stream, EP_TIMER_GRAPH_BANDWIDTH);
    bandwidth_check_rows<RowT><<<(unsigned)ceil_div(N, 256), 256, 0, stream>>>(rowptr, N, nnz, ctx->d_status);
    int kernels = 2;
    if (ntiles > 0) {
        bandwidth_tile_rows<RowT><<<(unsigned)ceil_div(ntiles + 1, 256), 256, 0, stream>>>(rowptr, N, ntiles, b.tile_row);
        const int grid = (int)std::min<int64_t>(ntiles, (int64_t)ctx->sm_count * 5);
        const size_t dyn = sizeof(int) * (2 * (size_t)BW_EDGES + 1);
        EP_CUDA(ctx, cudaFuncSetAttribute(vertex_bandwidth_tiles<RowT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn));
        vertex_bandwidth_tiles<RowT><<<grid, BW_THREADS, dyn, stream>>>(rowptr, colidx, nnz, pi, N, b.tile_row, ntiles, vb,
                                                                     ctx->d_status);
        kernels += 2;
    }
    const int sgrid = (int)std::max<int64_t>(1, std::min<int64_t>((int64_t)ctx->sm_count * 4, ceil_div(N, 256)));
    bandwidth_total<<<sgrid, 256, 0, stream>>>(vb, N, total);
    tm.end(kernels);
    EP_CUDA(ctx, cudaGetLastError());
    return EP_OK;
}

int bandwidth_run(ep_ctx *ctx, const void *rowptr, bool rowptr64, const int32_t *colidx, int64_t nnz,
                  const int32_t *pi, int64_t N, unsigned long long *total, int32_t *vertex_bandwidth, void *workspace,
                  cudaStream_t stream) {
    BandwidthBuffers b;
    bandwidth_layout(N, nnz, workspace, &b);
    int32_t *vb = vertex_bandwidth ? vertex_bandwidth : b.vb;
    EP_CUDA(ctx, cudaMemsetAsync(total, 0, sizeof(unsigned long long), stream));
    EP_CUDA(ctx, cudaMemsetAsync(vb, 0, sizeof(int32_t) * (size_t)N, stream));
    if (rowptr64)
        return bandwidth_launch<int64_t>(ctx, static_cast<const int64_t *>(rowptr), colidx, nnz, pi, N, total, vb, b, stream);
    return bandwidth_launch<int32_t>(ctx, static_cast<const int32_t *>(rowptr), colidx, nnz, pi, N, total, vb, b, stream);
}

}  // namespace ep
