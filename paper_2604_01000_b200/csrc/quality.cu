// Edge cut and partition loads (Section 2.1.1, Eq. 1 and Eq. 2) over a CSR graph.
//
// The work is split by EDGES, not by rows, so a power-law degree distribution cannot unbalance it:
// every warp takes chunks of QC_EDGES consecutive CSR entries, streams their column ids with 16-byte
// loads, and recovers the source vertex of each entry from a bitmap of row starts built in shared
// memory.  Labels are first repacked to the narrowest integer that holds K values so that the
// per-entry label gather touches as few cache lines as possible.
#include "ep_common.cuh"

#include <algorithm>

namespace {

constexpr int QC_VEC = 8;                                   // 16-byte loads per lane per chunk
constexpr int QC_EDGES = 32 * QC_VEC * 4;                   // 1024 entries per warp chunk
constexpr int QC_WORDS = QC_EDGES / 32;                     // 32 bitmap words, one per lane
constexpr int HIST_SMEM_K = 2048;
constexpr unsigned FULL = 0xffffffffu;

// tile_row[t] = last row r in [0, N) whose first entry is at or before t * QC_EDGES; tile_row[ntiles] = N-1.
template <typename RowT>
__global__ void tile_start_rows(const RowT *__restrict__ rowptr, int64_t N, int64_t ntiles, int32_t *tile_row) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t > ntiles) return;
    if (t == ntiles) {
        tile_row[t] = (int32_t)(N - 1);
        return;
    }
    const int64_t e = t * QC_EDGES;
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

// Counts the cut entries.  Every WARP takes chunks of QC_EDGES consecutive CSR entries and works on them on its own:
// no barrier wider than the warp anywhere, so the warps of a block drift apart and hide one another's latencies.
// For a chunk [e0, e0+ne): the rows whose first entry falls inside it set a bit at that position (a 32-word bitmap of
// the warp's own in shared memory) and park their label there; an entry's source label is the label at the nearest
// set bit at or before it (or, before the first set bit, the label of the row that straddles the chunk start).
//
// PACK = 0: the label of an entry's target comes from the repacked label array in global memory (L2).
// PACK = 8 / 4: every block first copies all labels into shared memory, one byte / one nibble each (K <= 256 /
// K <= 16, and N small enough to fit), so that the per-entry gather never leaves the SM and the pass becomes a
// plain stream of the column ids.  WARPS = 8: four such blocks per SM; WARPS = 32: one block per SM, for a table
// so large that only one copy fits, which still needs 32 warps to hide the stream's latency.
//
// SLICED: the launch counts only the entries whose target lies in [col_lo, col_hi) (and reports bad indices only
// when col_lo == 0); the caller launches it once per slice of the vertex range, each slice's labels small enough to
// stay in the L2 while the column ids stream past, and the counts of the launches add up.
template <typename LabT>
struct WarpScratch {
    unsigned bitmap[QC_WORDS];
    int lasthead[QC_WORDS];                  // 1 + position of the last row start in the words before this one; 0: none
    LabT headlab[QC_EDGES + 4];              // [0]: label of the row that straddles the chunk start; [1 + h]: row starting at h
};

template <typename RowT, typename LabT, int PACK, int WARPS, bool SLICED = false>
__global__ void __launch_bounds__(WARPS * 32, WARPS == 8 ? 4 : 1)
    edge_cut_chunks(const RowT *__restrict__ rowptr, const int32_t *__restrict__ colidx, int64_t nnz,
                    const LabT *__restrict__ lab, int64_t N, const int32_t *__restrict__ chunk_row, int64_t nchunks,
                    unsigned long long *edge_cut, int *status, int32_t col_lo, int32_t col_hi) {
    __shared__ WarpScratch<LabT> scratch[WARPS];
    __shared__ unsigned long long block_cut;
    extern __shared__ __align__(16) uint8_t lab_tab[];       // PACK != 0: all labels, packed
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned *bitmap = scratch[warp].bitmap;
    int *lasthead = scratch[warp].lasthead;
    LabT *headlab = scratch[warp].headlab;
    if (threadIdx.x == 0) block_cut = 0ull;
    unsigned long long my_cut = 0ull;
    if (PACK == 8) {
        for (int64_t v = threadIdx.x * 4; v < N; v += WARPS * 32 * 4) {   // N bytes; the array is padded to a multiple of 4
            *reinterpret_cast<uint32_t *>(lab_tab + v) = *reinterpret_cast<const uint32_t *>(reinterpret_cast<const uint8_t *>(lab) + v);
        }
    } else if (PACK == 4) {
        for (int64_t v = threadIdx.x * 4; v < N; v += WARPS * 32 * 4) {   // four labels in, two bytes out
            const uint32_t w4 = *reinterpret_cast<const uint32_t *>(reinterpret_cast<const uint8_t *>(lab) + v);
            *reinterpret_cast<uint16_t *>(lab_tab + (v >> 1)) =
                (uint16_t)((w4 & 15u) | ((w4 >> 4) & 0xF0u) | ((w4 >> 8) & 0xF00u) | ((w4 >> 12) & 0xF000u));
        }
    }
    __syncthreads();                                         // the table, and block_cut

    // a lane's vectors sit at entries (i * 32 + lane) * 4: always the same bit of their bitmap word
    const int vbit = (lane * 4) & 31;
    const unsigned upto_mask = 0xffffffffu >> (31 - vbit);

    // The rows that start inside a chunk are found through three dependent loads (the chunk's first row, its
    // entries' range, its label).  They are taken out of the chunk's own critical path: a lane's first row of the
    // NEXT chunk and the row range of the chunk after that are loaded while the current chunk is worked on.
    const int64_t stride = (int64_t)gridDim.x * WARPS;
    int64_t chunk = (int64_t)blockIdx.x * WARPS + warp;
    int32_t r_lo = 0, r_hi = -1, n_lo = 0, n_hi = -1;
    int64_t row_s = 0, row_e = 0;                            // entries of row r_lo + lane, and its label
    LabT row_l = 0;
    if (chunk < nchunks) {
        r_lo = chunk_row[chunk];
        r_hi = chunk_row[chunk + 1];
        if (r_lo + lane <= r_hi) {
            row_s = (int64_t)rowptr[r_lo + lane];
            row_e = (int64_t)rowptr[r_lo + lane + 1];
            row_l = lab[r_lo + lane];
        }
    }
    if (chunk + stride < nchunks) {
        n_lo = chunk_row[chunk + stride];
        n_hi = chunk_row[chunk + stride + 1];
    }
    for (; chunk < nchunks; chunk += stride) {
        const int64_t e0 = chunk * QC_EDGES;
        const int ne = (int)min((int64_t)QC_EDGES, nnz - e0);
        const bool full = ne == QC_EDGES;
        const int4 *src = reinterpret_cast<const int4 *>(colidx + e0);
        // issue this chunk's column loads first: they do not depend on anything below
        int4 c[QC_VEC];
        if (full) {
#pragma unroll
            for (int i = 0; i < QC_VEC; ++i) c[i] = __ldcs(src + i * 32 + lane);
        } else {
#pragma unroll
            for (int i = 0; i < QC_VEC; ++i) {
                const int q = (i * 32 + lane) * 4;
                c[i].x = q + 0 < ne ? colidx[e0 + q + 0] : -1;
                c[i].y = q + 1 < ne ? colidx[e0 + q + 1] : -1;
                c[i].z = q + 2 < ne ? colidx[e0 + q + 2] : -1;
                c[i].w = q + 3 < ne ? colidx[e0 + q + 3] : -1;
            }
        }
        int64_t next_s = 0, next_e = 0;
        LabT next_l = 0;
        int32_t nn_lo = 0, nn_hi = -1;
        if (n_lo + lane <= n_hi) {                           // n_hi = -1 when there is no next chunk
            next_s = (int64_t)rowptr[n_lo + lane];
            next_e = (int64_t)rowptr[n_lo + lane + 1];
            next_l = lab[n_lo + lane];
        }
        if (chunk + 2 * stride < nchunks) {
            nn_lo = chunk_row[chunk + 2 * stride];
            nn_hi = chunk_row[chunk + 2 * stride + 1];
        }
        __syncwarp();                                    // previous chunk fully consumed by every lane
        bitmap[lane] = 0u;
        __syncwarp();
        if (lane == 0) headlab[0] = row_l;               // row r_lo: the one that straddles the chunk start
        {
            const int64_t h = row_s - e0;
            if (row_e > row_s && h >= 0 && h < ne && EP_INDEX_OK(h, QC_EDGES, status)) {
                atomicOr(&bitmap[h >> 5], 1u << (h & 31));
                headlab[1 + h] = row_l;
            }
        }
        for (int64_t r = (int64_t)r_lo + 32 + lane; r <= r_hi; r += 32) {
            const int64_t s = (int64_t)rowptr[r], e = (int64_t)rowptr[r + 1];
            const int64_t h = s - e0;
            if (e > s && h >= 0 && h < ne && EP_INDEX_OK(h, QC_EDGES, status)) {
                atomicOr(&bitmap[h >> 5], 1u << (h & 31));
                headlab[1 + h] = lab[r];
            }
        }
        __syncwarp();
        {   // lasthead[w] = 1 + position of the last set bit in the words before w, or 0
            const unsigned wbits = bitmap[lane];
            int inc = wbits ? lane * 32 + 32 - __clz(wbits) : 0;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(FULL, inc, o);
                if (lane >= o) inc = max(inc, t);
            }
            int excl = __shfl_up_sync(FULL, inc, 1);
            if (lane == 0) excl = 0;
            lasthead[lane] = excl;
        }
        __syncwarp();
        unsigned cut = 0, bad = 0;
        // index into headlab of the source label in force at entry q (the first of a vector)
        auto source_of = [&](int wd, unsigned bits) -> int {
            const unsigned upto = bits & upto_mask;
            const int before = lasthead[wd];
            const int inside = (wd << 5) + 32 - __clz(upto);
            return upto ? inside : before;
        };
        // one vector of four entries with every test: a ragged chunk, or an index outside [0, N) somewhere in the warp
        auto vec = [&](int q, const int4 &cv) {
            const int wd = q >> 5;
            const unsigned bits = bitmap[wd];
            LabT cur = headlab[source_of(wd, bits)];
            const int cols[4] = {cv.x, cv.y, cv.z, cv.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (j > 0 && ((bits >> (vbit + j)) & 1u)) cur = headlab[1 + q + j];
                const bool live = q + j < ne;
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
        // The usual vector: a full chunk, every index of the warp inside [0, N).  No per-entry range or length test,
        // and one source label for all four entries unless a row starts among the last three of some lane's vector
        // (decided for the warp as a whole, so that the branch does not diverge).
        auto differs = [&](int col, unsigned cur) -> unsigned {
            if (PACK == 8) return lab_tab[col] != cur ? 1u : 0u;
            if (SLICED && (unsigned)(col - col_lo) >= (unsigned)(col_hi - col_lo)) return 0u;   // another launch's entry
            return (unsigned)__ldg(lab + col) != cur ? 1u : 0u;
        };
        unsigned nib16 = 0u;                                 // PACK == 4: 16 x the differing entries of this chunk
        auto vec_clean = [&](int q, const int4 &cv) {
            const int wd = q >> 5;
            const unsigned bits = bitmap[wd];
            const unsigned c0 = (unsigned)headlab[source_of(wd, bits)];
            const unsigned inner = (bits >> vbit) & 0xEu;
            const bool split = __any_sync(FULL, inner != 0u);
            unsigned c1 = c0, c2 = c0, c3 = c0;
            if (PACK == 4) {
                // Four nibble lookups compared at once.  The four bytes that hold the targets' labels are packed into
                // one word and XORed with the source labels (each in both nibbles of its byte); a byte's mask keeps the
                // nibble its index selects (0x0F or 0xF0 = 0x0F + 0xE1 x the index's lowest bit); a byte differs when
                // the kept nibble is not zero.
                const unsigned t0 = lab_tab[cv.x >> 1], t1 = lab_tab[cv.y >> 1], t2 = lab_tab[cv.z >> 1],
                               t3 = lab_tab[cv.w >> 1];
                const unsigned tw = (t1 * 256u + t0) + (t3 * 256u + t2) * 65536u;
                const unsigned low = __byte_perm(__byte_perm(cv.x, cv.y, 0x0040), __byte_perm(cv.z, cv.w, 0x0040), 0x5410) &
                                     0x01010101u;
                const unsigned mask = low * 0xE1u + 0x0F0F0F0Fu;
                unsigned cw = c0 * 0x11111111u;
                if (split) {
                    const unsigned h1 = headlab[1 + q + 1], h2 = headlab[1 + q + 2], h3 = headlab[1 + q + 3];
                    c1 = (inner & 2u) ? h1 : c0;
                    c2 = (inner & 4u) ? h2 : c1;
                    c3 = (inner & 8u) ? h3 : c2;
                    cw = (c0 | (c1 << 8) | (c2 << 16) | (c3 << 24)) * 0x11u;
                }
                const unsigned v = (tw ^ cw) & mask;
                const unsigned nz = (((v | (v >> 4)) & 0x0F0F0F0Fu) + 0x0F0F0F0Fu) & 0x10101010u;
                nib16 = __dp4a(nz, 0x01010101u, nib16);
            } else {
                if (split) {
                    const unsigned h1 = headlab[1 + q + 1], h2 = headlab[1 + q + 2], h3 = headlab[1 + q + 3];
                    c1 = (inner & 2u) ? h1 : c0;
                    c2 = (inner & 4u) ? h2 : c1;
                    c3 = (inner & 8u) ? h3 : c2;
                }
                cut += differs(cv.x, c0) + differs(cv.y, c1) + differs(cv.z, c2) + differs(cv.w, c3);
            }
        };
        unsigned top = 0u;                                   // largest index of this thread, as unsigned
#pragma unroll
        for (int i = 0; i < QC_VEC; ++i)
            top = max(max(max(top, (unsigned)c[i].x), max((unsigned)c[i].y, (unsigned)c[i].z)), (unsigned)c[i].w);
        if (__all_sync(FULL, full && top < (unsigned)N)) {
#pragma unroll
            for (int i = 0; i < QC_VEC; ++i) vec_clean((i * 32 + lane) * 4, c[i]);
            cut += nib16 >> 4;
        } else {
#pragma unroll
            for (int i = 0; i < QC_VEC; ++i) {
                const int q = (i * 32 + lane) * 4;
                if (q < ne) vec(q, c[i]);
            }
        }
        if (bad) ep_raise(status, EP_ERR_BAD_INDEX);
        my_cut += cut;
        r_lo = n_lo, r_hi = n_hi, n_lo = nn_lo, n_hi = nn_hi;
        row_s = next_s, row_e = next_e, row_l = next_l;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) my_cut += __shfl_xor_sync(FULL, my_cut, o);
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
    b.tile_row = a.take<int32_t>(ceil_div(nnz, QC_EDGES) + 1);
    if (out) *out = b;
    return a.used;
}

size_t quality_workspace_bytes(int64_t N, int64_t nnz, int K) { return quality_layout(N, nnz, K, nullptr, nullptr); }

template <typename RowT, typename LabT>
static int quality_launch(ep_ctx *ctx, const RowT *rowptr, const int32_t *colidx, int64_t nnz, const int32_t *assign,
                          int64_t N, int K, unsigned long long *edge_cut, unsigned long long *pv,
                          unsigned long long *pe, const QualityBuffers &b, cudaStream_t stream) {
    LabT *lab = static_cast<LabT *>(b.lab);
    const int64_t ntiles = ceil_div(nnz, QC_EDGES);
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
        // labels in shared memory when they fit beside the kernel's static shared memory (1.25 KB per warp)
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
            // four blocks of 8 warps per SM while four copies of the table fit, else one block of 32 warps
            const bool small = (tab + stat1) * 4 <= (size_t)ctx->smem_optin;
#define EP_EC(P, G)                                                                                                  \
    do {                                                                                                             \
        auto kern = edge_cut_chunks<RowT, LabT, P, G>;                                                               \
        EP_CUDA(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tab));             \
        const int grid = (int)std::min<int64_t>(ceil_div(ntiles, (int64_t)G), (int64_t)ctx->sm_count * (G == 8 ? 4 : 1)); \
        kern<<<grid, 32 * G, tab, stream>>>(rowptr, colidx, nnz, lab, N, b.tile_row, ntiles, edge_cut,               \
                                            ctx->d_status, 0, 0);                                                    \
    } while (0)
            if (pack == 4 && small) EP_EC(4, 8);
            else if (pack == 4) EP_EC(4, 32);
            else if (small) EP_EC(8, 8);
            else EP_EC(8, 32);
#undef EP_EC
        }
        int launches = 1;
        if (!launched) {
            const int grid = (int)std::min<int64_t>(ceil_div(ntiles, (int64_t)8), (int64_t)ctx->sm_count * 4);
            // Labels that cannot stay in the L2 beside the stream cost a DRAM sector per entry.  Then the vertex range
            // is cut into slices whose labels do fit, and the column ids are streamed once per slice: reading them
            // again is cheaper than missing on every gather.
            const size_t lab_total = (size_t)N * sizeof(LabT);
            const int slices = (int)std::min<size_t>(8, ceil_div(lab_total, (size_t)ctx->opt_slice_kb << 10));
            if (slices <= 1) {
                edge_cut_chunks<RowT, LabT, 0, 8><<<grid, 256, 0, stream>>>(rowptr, colidx, nnz, lab, N, b.tile_row, ntiles,
                                                                            edge_cut, ctx->d_status, 0, 0);
            } else {
                launches = slices;
                for (int sl = 0; sl < slices; ++sl) {
                    const int32_t lo = (int32_t)(N * sl / slices), hi = (int32_t)(N * (sl + 1) / slices);
                    edge_cut_chunks<RowT, LabT, 0, 8, true><<<grid, 256, 0, stream>>>(
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
