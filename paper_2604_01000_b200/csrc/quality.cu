// Edge cut and partition loads (Section 2.1.1, Eq. 1 and Eq. 2) over a CSR graph.
//
// The work is split by EDGES, not by rows, so a power-law degree distribution cannot unbalance it:
// every block takes tiles of QT_EDGES consecutive CSR entries, streams their column ids with 16-byte
// loads, and recovers the source vertex of each entry from a bitmap of row starts built in shared
// memory.  Labels are first repacked to the narrowest integer that holds K values so that the
// per-entry label gather touches as few cache lines as possible.
#include "ep_common.cuh"

#include <algorithm>

namespace {

constexpr int QT_THREADS = 256;
constexpr int QT_VEC = 8;                                   // 16-byte loads per thread per tile
constexpr int QT_EDGES = QT_THREADS * QT_VEC * 4;           // 8192 entries per tile
constexpr int QT_WORDS = QT_EDGES / 32;                     // 256 bitmap words, one per thread
constexpr int HIST_SMEM_K = 2048;
constexpr unsigned FULL = 0xffffffffu;

// tile_row[t] = last row r in [0, N) whose first entry is at or before t * QT_EDGES; tile_row[ntiles] = N-1.
template <typename RowT>
__global__ void tile_start_rows(const RowT *__restrict__ rowptr, int64_t N, int64_t ntiles, int32_t *tile_row) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t > ntiles) return;
    if (t == ntiles) {
        tile_row[t] = (int32_t)(N - 1);
        return;
    }
    const int64_t e = t * QT_EDGES;
    int64_t lo = 0, hi = N - 1;                             // rowptr[0] = 0 <= e always
    while (lo < hi) {
        int64_t mid = (lo + hi + 1) >> 1;
        if ((int64_t)rowptr[mid] <= e)
            lo = mid;
        else
            hi = mid - 1;
    }
    tile_row[t] = (int32_t)lo;
}

// Validates and repacks the labels, and accumulates part_vertices / part_edges.
template <typename RowT, typename LabT>
__global__ void __launch_bounds__(256) pack_labels_and_loads(const RowT *__restrict__ rowptr,
                                                             const int32_t *__restrict__ assign, int64_t N,
                                                             int64_t nnz, int K, LabT *__restrict__ lab,
                                                             unsigned long long *part_vertices,
                                                             unsigned long long *part_edges, int *status) {
    // block-local counts: vertices, and the degree sum as two 32-bit words (low word, carries + high parts), because
    // 32-bit additions are native in shared memory and 64-bit ones are not
    __shared__ unsigned int cv[HIST_SMEM_K];
    __shared__ unsigned int ce_lo[HIST_SMEM_K], ce_hi[HIST_SMEM_K];
    const bool local = K <= HIST_SMEM_K;
    if (local) {
        for (int k = threadIdx.x; k < K; k += blockDim.x) {
            cv[k] = 0u;
            ce_lo[k] = 0u;
            ce_hi[k] = 0u;
        }
        __syncthreads();
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        if ((int64_t)rowptr[0] != 0 || (int64_t)rowptr[N] != nnz) ep_raise(status, EP_ERR_BAD_INDEX);
    }
    for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < N; v += (int64_t)gridDim.x * blockDim.x) {
        int a = assign[v];
        if ((unsigned)a >= (unsigned)K) {
            ep_raise(status, EP_ERR_BAD_INDEX);
            a = 0;
        }
        lab[v] = (LabT)a;
        long long deg = (long long)rowptr[v + 1] - (long long)rowptr[v];
        if (deg < 0) {
            ep_raise(status, EP_ERR_BAD_INDEX);
            deg = 0;
        }
        if (local) {
            atomicAdd(&cv[a], 1u);
            const unsigned lo = (unsigned)((unsigned long long)deg & 0xffffffffull);
            const unsigned hi = (unsigned)((unsigned long long)deg >> 32);
            const unsigned old = atomicAdd(&ce_lo[a], lo);
            const unsigned carry = (old + lo < old) ? 1u : 0u;     // the low word wrapped
            if (hi + carry) atomicAdd(&ce_hi[a], hi + carry);
        } else {
            atomicAdd(&part_vertices[a], 1ull);
            atomicAdd(&part_edges[a], (unsigned long long)deg);
        }
    }
    if (local) {
        __syncthreads();
        for (int k = threadIdx.x; k < K; k += blockDim.x) {
            if (cv[k]) atomicAdd(&part_vertices[k], (unsigned long long)cv[k]);
            const unsigned long long e = ((unsigned long long)ce_hi[k] << 32) + ce_lo[k];
            if (e) atomicAdd(&part_edges[k], e);
        }
    }
}

// Counts the cut entries.  For a tile [e0, e0+ne): the rows whose first entry falls inside the tile
// set a bit at that position and park their label there; an entry's source label is the label at the
// nearest set bit at or before it (or, before the first set bit, the label of the row that straddles
// the tile start).
//
// PACK = 0: the label of an entry's target comes from the repacked label array in global memory (L2).
// PACK = 8 / 4: every block first copies all labels into shared memory, one byte / one nibble each (K <= 256 /
// K <= 16, and N small enough to fit), so that the per-entry gather never leaves the SM and the pass becomes a
// plain stream of the column ids.
//
// GROUPS = 1: a block is one group of QT_THREADS threads.  GROUPS = 4: a block of 1024 threads holds four such
// groups, each with its own tile, bitmap and named barrier, sharing one copy of the label table: the form for a
// table so large that only one block fits on an SM, which still needs 32 warps to hide the stream's latency.
//
// SLICED: the launch counts only the entries whose target lies in [col_lo, col_hi) (and reports bad indices only
// when col_lo == 0); the caller launches it once per slice of the vertex range, each slice's labels small enough to
// stay in the L2 while the column ids stream past, and the counts of the launches add up.
template <typename RowT, typename LabT, int PACK, int GROUPS, bool SLICED = false>
__global__ void __launch_bounds__(QT_THREADS * GROUPS, GROUPS == 1 ? 4 : 1)
    edge_cut_tiles(const RowT *__restrict__ rowptr, const int32_t *__restrict__ colidx, int64_t nnz,
                   const LabT *__restrict__ lab, int64_t N, const int32_t *__restrict__ tile_row, int64_t ntiles,
                   unsigned long long *edge_cut, int *status, int32_t col_lo, int32_t col_hi) {
    __shared__ unsigned bitmap_[GROUPS][QT_WORDS];
    __shared__ int lasthead_[GROUPS][QT_WORDS];
    __shared__ LabT headlab_[GROUPS][QT_EDGES];
    __shared__ int warp_max_[GROUPS][QT_THREADS / 32];
    __shared__ unsigned long long block_cut;
    extern __shared__ __align__(16) uint8_t lab_tab[];       // PACK != 0: all labels, packed
    const int grp = GROUPS == 1 ? 0 : (int)(threadIdx.x / QT_THREADS);
    unsigned *bitmap = bitmap_[grp];
    int *lasthead = lasthead_[grp];
    LabT *headlab = headlab_[grp];
    int *warp_max = warp_max_[grp];
    auto group_sync = [&]() {
        if (GROUPS == 1)
            __syncthreads();
        else
            asm volatile("bar.sync %0, %1;" ::"r"(grp + 1), "n"(QT_THREADS) : "memory");
    };
    const int tid = threadIdx.x % QT_THREADS, lane = tid & 31, warp = tid >> 5;
    if (threadIdx.x == 0) block_cut = 0ull;
    unsigned long long my_cut = 0ull;
    if (PACK == 8) {
        for (int64_t v = threadIdx.x * 4; v < N; v += QT_THREADS * GROUPS * 4) {   // N bytes; the array is padded to a multiple of 4
            *reinterpret_cast<uint32_t *>(lab_tab + v) = *reinterpret_cast<const uint32_t *>(reinterpret_cast<const uint8_t *>(lab) + v);
        }
    } else if (PACK == 4) {
        for (int64_t v = threadIdx.x * 4; v < N; v += QT_THREADS * GROUPS * 4) {   // four labels in, two bytes out
            const uint32_t w4 = *reinterpret_cast<const uint32_t *>(reinterpret_cast<const uint8_t *>(lab) + v);
            *reinterpret_cast<uint16_t *>(lab_tab + (v >> 1)) =
                (uint16_t)((w4 & 15u) | ((w4 >> 4) & 0xF0u) | ((w4 >> 8) & 0xF00u) | ((w4 >> 12) & 0xF000u));
        }
    }
    if (PACK != 0) __syncthreads();

    for (int64_t tile = (int64_t)blockIdx.x * GROUPS + grp; tile < ntiles; tile += (int64_t)gridDim.x * GROUPS) {
        const int64_t e0 = tile * QT_EDGES;
        const int ne = (int)min((int64_t)QT_EDGES, nnz - e0);
        const int4 *src = reinterpret_cast<const int4 *>(colidx + e0);
        // issue this tile's column loads first: they do not depend on anything below
        int4 c[QT_VEC];
#pragma unroll
        for (int i = 0; i < QT_VEC; ++i) {
            const int q = (i * QT_THREADS + tid) * 4;
            if (q + 3 < ne) {
                c[i] = __ldcs(src + (q >> 2));
            } else {
                c[i].x = q + 0 < ne ? colidx[e0 + q + 0] : -1;
                c[i].y = q + 1 < ne ? colidx[e0 + q + 1] : -1;
                c[i].z = q + 2 < ne ? colidx[e0 + q + 2] : -1;
                c[i].w = -1;
            }
        }
        group_sync();                                    // previous tile fully consumed
        bitmap[tid] = 0u;
        group_sync();
        const int64_t r_lo = tile_row[tile], r_hi = tile_row[tile + 1];
        const LabT carry = lab[r_lo];
        for (int64_t r = r_lo + tid; r <= r_hi; r += QT_THREADS) {
            const int64_t s = (int64_t)rowptr[r], e = (int64_t)rowptr[r + 1];
            const int64_t h = s - e0;
            if (e > s && h >= 0 && h < ne && EP_INDEX_OK(h, QT_EDGES, status)) {
                atomicOr(&bitmap[h >> 5], 1u << (h & 31));
                headlab[h] = lab[r];
            }
        }
        group_sync();
        {   // lasthead[w] = position of the last set bit in words < w, or -1
            const unsigned wbits = bitmap[tid];
            const int mine = wbits ? tid * 32 + 31 - __clz(wbits) : -1;
            int inc = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int t = __shfl_up_sync(FULL, inc, o);
                if (lane >= o) inc = max(inc, t);
            }
            if (lane == 31) warp_max[warp] = inc;
            int excl = __shfl_up_sync(FULL, inc, 1);
            if (lane == 0) excl = -1;
            group_sync();
            for (int w = 0; w < warp; ++w) excl = max(excl, warp_max[w]);
            lasthead[tid] = excl;
        }
        group_sync();
        unsigned cut = 0, bad = 0;
        // one vector of four entries: their source label from the bitmap, their targets' labels gathered
        auto vec = [&](int q, const int4 &cv, bool full) {
            const int wd = q >> 5, b = q & 31;
            const unsigned bits = bitmap[wd];
            const unsigned upto = bits & (0xffffffffu >> (31 - b));
            const int head = upto ? (wd << 5) + 31 - __clz(upto) : lasthead[wd];
            LabT cur = head >= 0 ? headlab[head] : carry;
            const int cols[4] = {cv.x, cv.y, cv.z, cv.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (j > 0 && ((bits >> (b + j)) & 1u)) cur = headlab[q + j];
                const bool live = full || q + j < ne;
                const int col = cols[j];
                const bool in = (unsigned)col < (unsigned)N;
                const bool mine = !SLICED || (unsigned)(col - col_lo) < (unsigned)(col_hi - col_lo);
                const int cc = (in && mine) ? col : 0;       // an index outside [0, N) is reported, never followed
                unsigned tgt;
                if (PACK == 8)
                    tgt = lab_tab[cc];
                else if (PACK == 4)
                    tgt = (lab_tab[cc >> 1] >> ((cc & 1) << 2)) & 15u;
                else
                    tgt = (in && mine) ? (unsigned)__ldg(lab + cc) : (unsigned)cur;
                cut += (live && in && mine && tgt != (unsigned)cur) ? 1u : 0u;
                bad |= (live && !in && (!SLICED || col_lo == 0)) ? 1u : 0u;
            }
        };
        // The usual vector: a full tile, every index of this thread inside [0, N).  No per-entry range or length
        // test, and one source label for all four entries unless a row starts among the last three.
        auto differs = [&](int col, unsigned cur) -> unsigned {
            if (PACK == 8) return lab_tab[col] != cur ? 1u : 0u;
            if (PACK == 4)   // cur fills both nibbles: compare the nibble of col in place
                return ((lab_tab[col >> 1] ^ cur) & (0xFu << ((col << 2) & 4))) != 0u ? 1u : 0u;
            if (SLICED && (unsigned)(col - col_lo) >= (unsigned)(col_hi - col_lo)) return 0u;   // another launch's entry
            return (unsigned)__ldg(lab + col) != cur ? 1u : 0u;
        };
        auto vec_clean = [&](int q, const int4 &cv) {
            const int wd = q >> 5, b = q & 31;
            const unsigned bits = bitmap[wd];
            const unsigned upto = bits & (0xffffffffu >> (31 - b));
            const int head = upto ? (wd << 5) + 31 - __clz(upto) : lasthead[wd];
            const unsigned cur = head >= 0 ? (unsigned)headlab[head] : (unsigned)carry;
            const unsigned rep = PACK == 4 ? 0x11u : 1u;
            if (((bits >> b) & 0xEu) == 0u) {
                const unsigned cw = cur * rep;
                cut += differs(cv.x, cw) + differs(cv.y, cw) + differs(cv.z, cw) + differs(cv.w, cw);
            } else {
                const unsigned c1 = ((bits >> (b + 1)) & 1u) ? (unsigned)headlab[q + 1] : cur;
                const unsigned c2 = ((bits >> (b + 2)) & 1u) ? (unsigned)headlab[q + 2] : c1;
                const unsigned c3 = ((bits >> (b + 3)) & 1u) ? (unsigned)headlab[q + 3] : c2;
                cut += differs(cv.x, cur * rep) + differs(cv.y, c1 * rep) + differs(cv.z, c2 * rep) + differs(cv.w, c3 * rep);
            }
        };
        unsigned top = 0u;                                   // largest index of this thread, as unsigned
#pragma unroll
        for (int i = 0; i < QT_VEC; ++i)
            top = max(max(max(top, (unsigned)c[i].x), max((unsigned)c[i].y, (unsigned)c[i].z)), (unsigned)c[i].w);
        if (ne == QT_EDGES && top < (unsigned)N) {
#pragma unroll
            for (int i = 0; i < QT_VEC; ++i) vec_clean((i * QT_THREADS + tid) * 4, c[i]);
        } else if (ne == QT_EDGES) {
#pragma unroll
            for (int i = 0; i < QT_VEC; ++i) vec((i * QT_THREADS + tid) * 4, c[i], true);
        } else {
#pragma unroll
            for (int i = 0; i < QT_VEC; ++i) {
                const int q = (i * QT_THREADS + tid) * 4;
                if (q < ne) vec(q, c[i], false);
            }
        }
        if (bad) ep_raise(status, EP_ERR_BAD_INDEX);
        my_cut += cut;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) my_cut += __shfl_xor_sync(FULL, my_cut, o);
    __syncthreads();
    if (lane == 0 && my_cut) atomicAdd(&block_cut, my_cut);
    __syncthreads();
    if (threadIdx.x == 0 && block_cut) atomicAdd(edge_cut, block_cut);
}

template <typename LabT>
size_t lab_bytes(int64_t N) { return (size_t)N * sizeof(LabT); }

}  // namespace

namespace ep {

static inline int label_width(int K) { return K <= 256 ? 1 : K <= 65536 ? 2 : 4; }

struct QualityBuffers {
    void *lab;
    int32_t *tile_row;
};

static size_t quality_layout(int64_t N, int64_t nnz, int K, void *ws, QualityBuffers *out) {
    Arena a(ws);
    QualityBuffers b{};
    b.lab = a.take<char>(((size_t)N + 4) * label_width(K));
    b.tile_row = a.take<int32_t>(ceil_div(nnz, QT_EDGES) + 1);
    if (out) *out = b;
    return a.used;
}

size_t quality_workspace_bytes(int64_t N, int64_t nnz, int K) { return quality_layout(N, nnz, K, nullptr, nullptr); }

template <typename RowT, typename LabT>
static int quality_launch(ep_ctx *ctx, const RowT *rowptr, const int32_t *colidx, int64_t nnz, const int32_t *assign,
                          int64_t N, int K, unsigned long long *edge_cut, unsigned long long *pv,
                          unsigned long long *pe, const QualityBuffers &b, cudaStream_t stream) {
    LabT *lab = static_cast<LabT *>(b.lab);
    const int64_t ntiles = ceil_div(nnz, QT_EDGES);
    const int pgrid = (int)std::max<int64_t>(1, std::min<int64_t>((int64_t)ctx->sm_count * 8, ceil_div(N, 256)));
    {
        Timed tm(ctx, stream, EP_TIMER_QUALITY_PREP);
        pack_labels_and_loads<RowT, LabT><<<pgrid, 256, 0, stream>>>(rowptr, assign, N, nnz, K, lab, pv, pe, ctx->d_status);
        if (ntiles > 0)
            tile_start_rows<RowT><<<(unsigned)ceil_div(ntiles + 1, 256), 256, 0, stream>>>(rowptr, N, ntiles, b.tile_row);
        tm.end(ntiles > 0 ? 2 : 1);
    }
    if (ntiles > 0) {
        Timed tm(ctx, stream, EP_TIMER_EDGE_CUT);
        // labels in shared memory when they fit beside the kernel's static shared memory (about 10.3 KB per group)
        const size_t stat1 = 12 * 1024, stat4 = 44 * 1024;
        const size_t tab4 = ((size_t)N + 7) / 8 * 4 + 16, tab8 = ((size_t)N + 3) / 4 * 4 + 16;
        const size_t room = (size_t)ctx->smem_optin - stat4;
        const int pack = sizeof(LabT) != 1 ? 0 : (K <= 16 && tab4 <= room) ? 4 : (tab8 <= room) ? 8 : 0;
        // worth it only when the copy (N bytes per block) is small beside the block's share of the entries
        const bool use_tab = pack != 0 && (int64_t)N * ctx->sm_count <= nnz * 2;
        bool launched = false;
        if constexpr (sizeof(LabT) == 1) if (use_tab) {
            launched = true;
            const size_t tab = pack == 4 ? tab4 : tab8;
            // four small blocks per SM while four copies of the table fit, else one block of four groups
            const bool small = (tab + stat1) * 4 <= (size_t)ctx->smem_optin;
#define EP_EC(P, G)                                                                                                  \
    do {                                                                                                             \
        auto kern = edge_cut_tiles<RowT, LabT, P, G>;                                                                \
        EP_CUDA(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tab));             \
        const int grid = (int)std::min<int64_t>(ceil_div(ntiles, (int64_t)G), (int64_t)ctx->sm_count * (G == 1 ? 4 : 1)); \
        kern<<<grid, QT_THREADS * G, tab, stream>>>(rowptr, colidx, nnz, lab, N, b.tile_row, ntiles, edge_cut,       \
                                                    ctx->d_status, 0, 0);                                            \
    } while (0)
            if (pack == 4 && small) EP_EC(4, 1);
            else if (pack == 4) EP_EC(4, 4);
            else if (small) EP_EC(8, 1);
            else EP_EC(8, 4);
#undef EP_EC
        }
        int launches = 1;
        if (!launched) {
            const int grid = (int)std::min<int64_t>(ntiles, (int64_t)ctx->sm_count * 4);
            // Labels that cannot stay in the L2 beside the stream cost a DRAM sector per entry.  Then the vertex range
            // is cut into slices whose labels do fit, and the column ids are streamed once per slice: reading them
            // again is cheaper than missing on every gather.
            const size_t lab_total = (size_t)N * sizeof(LabT);
            const int slices = (int)std::min<size_t>(8, ceil_div(lab_total, (size_t)ctx->opt_slice_kb << 10));
            if (slices <= 1) {
                edge_cut_tiles<RowT, LabT, 0, 1><<<grid, QT_THREADS, 0, stream>>>(rowptr, colidx, nnz, lab, N, b.tile_row,
                                                                                ntiles, edge_cut, ctx->d_status, 0, 0);
            } else {
                launches = slices;
                for (int sl = 0; sl < slices; ++sl) {
                    const int32_t lo = (int32_t)(N * sl / slices), hi = (int32_t)(N * (sl + 1) / slices);
                    edge_cut_tiles<RowT, LabT, 0, 1, true><<<grid, QT_THREADS, 0, stream>>>(
                        rowptr, colidx, nnz, lab, N, b.tile_row, ntiles, edge_cut, ctx->d_status, lo, hi);
                }
            }
        }
        tm.end(launches);
    }
    EP_CUDA(ctx, cudaGetLastError());
    return EP_OK;
}

int quality_run(ep_ctx *ctx, const void *rowptr, bool rowptr64, const int32_t *colidx, int64_t nnz,
                const int32_t *assign, int64_t N, int K, unsigned long long *edge_cut, long long *part_vertices,
                long long *part_edges, void *workspace, cudaStream_t stream) {
    QualityBuffers b;
    quality_layout(N, nnz, K, workspace, &b);
    EP_CUDA(ctx, cudaMemsetAsync(edge_cut, 0, sizeof(unsigned long long), stream));
    EP_CUDA(ctx, cudaMemsetAsync(part_vertices, 0, sizeof(long long) * K, stream));
    EP_CUDA(ctx, cudaMemsetAsync(part_edges, 0, sizeof(long long) * K, stream));
    auto *pv = reinterpret_cast<unsigned long long *>(part_vertices);
    auto *pe = reinterpret_cast<unsigned long long *>(part_edges);
    const int w = label_width(K);
#define EP_Q(RowT, LabT) \
    return quality_launch<RowT, LabT>(ctx, static_cast<const RowT *>(rowptr), colidx, nnz, assign, N, K, edge_cut, pv, pe, b, stream)
    if (rowptr64) {
        if (w == 1) EP_Q(int64_t, uint8_t);
        if (w == 2) EP_Q(int64_t, uint16_t);
        EP_Q(int64_t, int32_t);
    } else {
        if (w == 1) EP_Q(int32_t, uint8_t);
        if (w == 2) EP_Q(int32_t, uint16_t);
        EP_Q(int32_t, int32_t);
    }
#undef EP_Q
}

}  // namespace ep
