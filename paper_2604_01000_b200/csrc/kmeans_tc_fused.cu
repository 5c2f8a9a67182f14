// Fused assign-and-accumulate pass of Lloyd K-Means (Algorithm 3, line 1) for few centroids
// (K <= 64, d <= 128) on the tensor cores: one read of the embedding matrix per iteration.
//
// A persistent block per SM streams 128-row tiles of X through a ring of shared-memory stages (TMA,
// 128-byte swizzle).  All K centroids sit in shared memory for the whole launch, in fp32: the tensor
// core reads their upper 19 bits, the fp32 re-scoring reads all of them.  Three groups of warps work
// on consecutive tiles at the same time:
//   1. one thread issues tcgen05.mma kind::tf32: scores [128 x K] into one of two TMEM accumulators;
//   2. the screen group (4 warps, one row per thread) reads the accumulator back and keeps the two
//      smallest packed (score | column) keys.  If the second is farther from the first than the TF32
//      error bound of that row allows, the first is provably the fp32 argmin.  Otherwise the thread lists
//      the centroids within the bound, and the group re-scores those (row, centroid) pairs in fp32 from
//      the shared-memory tiles, eight pairs per warp step, lowest index winning ties, with the same
//      summation order as the CUDA-core kernels;
//   3. the accumulate group (4 warps) adds every row of the tile into the per-cluster sums it keeps in
//      registers: a warp owns rows, a lane owns columns, the label selects the register by a jump that
//      is uniform across the warp.  No atomics: the order of every addition is fixed by the launch
//      shape, so results repeat bit for bit.
// At the end the accumulate group folds its row groups in order through shared memory into psum[block].
#include "ep_common.cuh"
#include "kmeans_device.cuh"
#include "tc_device.cuh"

#include <math_constants.h>

#include <algorithm>

namespace {

using namespace epk;
using namespace eptc;

constexpr int BM = 128;                 // rows per tile = TMEM lanes
constexpr int KBLK = 32;                // floats in one 128-byte swizzle row
constexpr int MAX_KB = 4;               // d <= 128
constexpr int X_KB_BYTES = BM * 128;    // one k-block of a row tile
constexpr int MAX_STAGES = 8;
constexpr int THREADS = 512;            // warp 0 TMA, 1 MMA, 2 TMEM alloc, 3 idle, 4..7 screen group, 8..15 accumulate group
constexpr int S_WARP0 = 4;
constexpr int A_WARP0 = 8;
constexpr int A_WARPS = 8;
constexpr int MAX_K = 64;
constexpr int ROW_CANDS = 8;            // candidates listed per undecided row before it is scored against all K
constexpr int QUEUE_CAP = BM * ROW_CANDS;

struct FusedShared {
    uint64_t x_full[MAX_STAGES], x_empty[MAX_STAGES];
    uint64_t c_full;
    uint64_t t_full[2], t_empty[2];
    uint64_t lab_full[2], lab_empty[2];
    unsigned long long rowbest[BM];     // undecided rows: min over candidates of (ordered fp32 score << 32 | centroid)
    uint32_t tmem_base;
    int abort;
    int stop;                           // the abort flag as screen thread 0 saw it before the tile's first group barrier
    int qn, fqn;
    int queue[QUEUE_CAP];               // (row in tile << 8) | centroid
    int fullq[BM];                      // rows with more than ROW_CANDS candidates
    int order[2][BM];                   // rows of the tile grouped by label, ascending row inside a label
    int off[2][MAX_K + 1];              // first position of each label in order[]
    int wcnt[2][4][MAX_K + 1];          // rows per (screen warp, label); label MAX_K = rows beyond N
    int cnt[MAX_K];
    float cn[MAX_K];
    float red[2][4];
};

__device__ __forceinline__ void group_sync(int id) { asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory"); }

// Byte offset of 16-byte chunk q of row r in a swizzled tile whose k-blocks are kb_bytes apart.
__device__ __forceinline__ uint32_t chunk_off(int r, int q, int kb_bytes) {
    return (uint32_t)((q >> 3) * kb_bytes + r * 128 + (((q & 7) ^ (r & 7)) << 4));
}

__device__ __forceinline__ unsigned long long pack_score(float sc, int k) {
    uint32_t u = __float_as_uint(sc);
    u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);        // unsigned order = float order
    return ((unsigned long long)u << 32) | (uint32_t)k;
}

// KMAX = 32 or 64: upper bound of K, 8 accumulate warps each owning KMAX / 8 clusters.
// rownorm[i] = (|x_i|, |x_i - trunc_tf32(x_i)|); clo[k] = |c_k - trunc_tf32(c_k)|.
template <int KMAX>
__global__ void __launch_bounds__(THREADS, 1)
kmeans_tc_fused(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_c,
                const float *__restrict__ cn, const float *__restrict__ clo, const float2 *__restrict__ rownorm, int64_t N,
                int d, int K, int npad, int num_kb, int stages, uint32_t idesc, uint32_t tmem_cols, uint32_t key_mask,
                int32_t *__restrict__ assign, float *__restrict__ psum, int *__restrict__ pcnt,
                unsigned long long *counters, int *status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int stage_bytes = num_kb * X_KB_BYTES;
    const int c_kb_bytes = npad * 128;
    uint8_t *x_smem = smem;                                          // [stages][num_kb][128 rows][128 B]
    uint8_t *c_smem = x_smem + (size_t)stages * stage_bytes;         // [num_kb][npad rows][128 B]
    FusedShared *sh = reinterpret_cast<FusedShared *>(c_smem + (size_t)num_kb * c_kb_bytes);
    volatile int *abort_flag = &sh->abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int d4 = d >> 2;
    const int64_t num_tiles = (N + BM - 1) / BM;

    if (threadIdx.x == 0) {
        for (int i = 0; i < MAX_STAGES; ++i) {
            mbar_init(&sh->x_full[i], 1);
            mbar_init(&sh->x_empty[i], A_WARPS);
        }
        mbar_init(&sh->c_full, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sh->t_full[i], 1);
            mbar_init(&sh->t_empty[i], 4);
            mbar_init(&sh->lab_full[i], 4);
            mbar_init(&sh->lab_empty[i], A_WARPS);
        }
        sh->abort = 0;
        sh->stop = 0;
        sh->tmem_base = 0;
        sh->qn = sh->fqn = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int k = threadIdx.x; k < 2 * 4 * (MAX_K + 1); k += blockDim.x) (&sh->wcnt[0][0][0])[k] = 0;
    for (int k = threadIdx.x; k < MAX_K; k += blockDim.x) {
        sh->cnt[k] = 0;
        sh->cn[k] = k < npad ? cn[k] : CUDART_INF_F;     // cn is padded with a huge value beyond K
    }
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)),
                     "r"(tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            mbar_expect_tx(&sh->c_full, (uint32_t)(num_kb * c_kb_bytes));
            for (int kb = 0; kb < num_kb; ++kb)
                tma_load_2d(c_smem + (size_t)kb * c_kb_bytes, &map_c, kb * KBLK, 0, &sh->c_full);
            uint32_t it = 0;
            for (int64_t tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++it) {
                const uint32_t s = it % (uint32_t)stages, ph = (it / (uint32_t)stages) & 1u;
                if (!mbar_wait(&sh->x_empty[s], ph ^ 1u, abort_flag)) break;
                mbar_expect_tx(&sh->x_full[s], (uint32_t)stage_bytes);
                for (int kb = 0; kb < num_kb; ++kb)
                    tma_load_2d(x_smem + (size_t)s * stage_bytes + (size_t)kb * X_KB_BYTES, &map_x, kb * KBLK,
                                (int)(tile * BM), &sh->x_full[s]);
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            bool ok = mbar_wait(&sh->c_full, 0u, abort_flag);
            uint32_t it = 0;
            for (int64_t tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++it) {
                const uint32_t s = it % (uint32_t)stages, ph = (it / (uint32_t)stages) & 1u;
                const uint32_t buf = it & 1u, use = (it >> 1) & 1u;
                if (!(ok = mbar_wait(&sh->t_empty[buf], use ^ 1u, abort_flag))) break;
                if (!(ok = mbar_wait(&sh->x_full[s], ph, abort_flag))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * (uint32_t)npad;
                for (int kb = 0; kb < num_kb; ++kb) {
                    const uint64_t adesc = umma_desc(smem_u32(x_smem + (size_t)s * stage_bytes + (size_t)kb * X_KB_BYTES));
                    const uint64_t bdesc = umma_desc(smem_u32(c_smem + (size_t)kb * c_kb_bytes));
#pragma unroll
                    for (int ks = 0; ks < KBLK / 8; ++ks)
                        umma_tf32(d_tmem, adesc + (uint64_t)(2 * ks), bdesc + (uint64_t)(2 * ks), idesc,
                                  (kb | ks) != 0 ? 1u : 0u);
                }
                umma_commit(&sh->t_full[buf]);
            }
        }
    } else if (warp >= S_WARP0 && warp < A_WARP0) {
        // ---------------------------------------------------------------- screen group: one row per thread
        const int sw = warp - S_WARP0;                     // TMEM lanes 32 sw .. 32 sw + 31
        const int stid = threadIdx.x - S_WARP0 * 32;       // 0..127 = row in tile
        {   // largest centroid norm and truncation residual
            float m2 = 0.f, ml = 0.f;
            for (int k = stid; k < K; k += 128) {
                m2 = fmaxf(m2, cn[k]);
                ml = fmaxf(ml, clo[k]);
            }
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) {
                m2 = fmaxf(m2, __shfl_xor_sync(FULL, m2, o));
                ml = fmaxf(ml, __shfl_xor_sync(FULL, ml, o));
            }
            if (lane == 0) {
                sh->red[0][sw] = m2;
                sh->red[1][sw] = ml;
            }
        }
        group_sync(1);
        const float cmax2 = fmaxf(fmaxf(sh->red[0][0], sh->red[0][1]), fmaxf(sh->red[0][2], sh->red[0][3]));
        const float clomax = fmaxf(fmaxf(sh->red[1][0], sh->red[1][1]), fmaxf(sh->red[1][2], sh->red[1][3]));
        const float cmax = sqrtf(cmax2) * 1.000001f;
        const int slot = lane_chunk_slot(lane);
        unsigned long long n_rows = 0, n_undecided = 0, n_items = 0, n_full = 0;
        mbar_wait(&sh->c_full, 0u, abort_flag);            // the fp32 re-scoring below reads the centroid tile

        float2 nr_next = make_float2(0.f, 0.f);            // this row's norms, fetched one tile ahead
        if ((int64_t)blockIdx.x * BM + stid < N) nr_next = __ldg(rownorm + (int64_t)blockIdx.x * BM + stid);

        uint32_t it = 0;
        for (int64_t tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++it) {
            const uint32_t s = it % (uint32_t)stages, ph = (it / (uint32_t)stages) & 1u;
            const uint32_t buf = it & 1u, use = (it >> 1) & 1u, par = it & 1u;
            const uint8_t *xs = x_smem + (size_t)s * stage_bytes;
            const int64_t row = tile * BM + stid;
            const float2 nr = nr_next;
            {
                const int64_t nrow = (tile + gridDim.x) * BM + stid;
                if (nrow < N) nr_next = __ldg(rownorm + nrow);
            }
            // Waits that give up leave garbage behind but nothing out of bounds; the group leaves the loop
            // together after the next barrier.
            mbar_wait(&sh->lab_empty[par], use ^ 1u, abort_flag);
            mbar_wait(&sh->t_full[buf], use, abort_flag);
            mbar_wait(&sh->x_full[s], ph, abort_flag);
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(sw * 32) << 16) + buf * (uint32_t)npad;
            float a1 = __uint_as_float(KEY_INIT), a2 = a1, b1 = a1, b2 = a1;
            for (int c = 0; c < npad; c += 16) {
                uint32_t v[16];
                tmem_ld16(taddr + c, v);
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float sc = fmaf(-2.f, __uint_as_float(v[j]), sh->cn[c + j]);
                    const float key = __uint_as_float((__float_as_uint(sc) & key_mask) | (uint32_t)(c + j));
                    if (j & 1)
                        keep_two(b1, b2, key);
                    else
                        keep_two(a1, a2, key);
                }
            }
            const float k1 = fminf(a1, b1);
            const float k2 = fminf(fmaxf(a1, b1), fminf(a2, b2));
            const float thr = k1 + 2.f * screen_allowance(nr.x, nr.y, cmax, cmax2, clomax, d);
            const int i1 = (int)(__float_as_uint(k1) & IDX_MASK);
            const bool live = row < N;
            const bool decided = k2 > thr && i1 < K;       // the best screened score cannot be overtaken
            const bool undecided = live && !decided;
            if (__any_sync(FULL, undecided)) {
                // list this row's centroids whose screened score is within the allowance of the best
                int nc = 0;
                if (undecided) sh->rowbest[stid] = ~0ull;
                for (int c = 0; c < npad; c += 16) {
                    uint32_t v[16];
                    tmem_ld16(taddr + c, v);
                    if (undecided) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const float sc = fmaf(-2.f, __uint_as_float(v[j]), sh->cn[c + j]);
                            if (sc <= thr && c + j < K) {
                                if (nc < ROW_CANDS) sh->queue[atomicAdd(&sh->qn, 1)] = (stid << 8) | (c + j);
                                ++nc;
                            }
                        }
                    }
                }
                if (undecided && (nc > ROW_CANDS || nc == 0)) sh->fullq[atomicAdd(&sh->fqn, 1)] = stid;   // nc == 0: NaN scores
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh->t_empty[buf]);
            if (stid == 0) sh->stop = *abort_flag;
            group_sync(1);
            if (sh->stop) break;
            // ---- fp32 re-scoring of the listed (row, centroid) pairs, eight per warp step
            const int qn = min(sh->qn, QUEUE_CAP), fqn = min(sh->fqn, BM);
            for (int base = sw * KC; base < qn; base += 4 * KC) {
                float a[KC];
#pragma unroll
                for (int kk = 0; kk < KC; ++kk) {
                    const int item = sh->queue[min(base + kk, qn - 1)];
                    a[kk] = 0.f;
                    if (lane < d4) {
                        const float4 x = *reinterpret_cast<const float4 *>(xs + chunk_off(item >> 8, lane, X_KB_BYTES));
                        const float4 cc = *reinterpret_cast<const float4 *>(c_smem + chunk_off(item & 255, lane, c_kb_bytes));
                        a[kk] = dot4(x, cc, 0.f);
                    }
                }
                const float dot = reduce8_transposed(a, lane);
                if ((lane & 3) == 0 && base + slot < qn) {
                    const int item = sh->queue[base + slot];
                    float sc = fmaf(-2.f, dot, sh->cn[item & 255]);
                    sc = (sc == sc) ? sc : CUDART_INF_F;
                    atomicMin(&sh->rowbest[item >> 8], pack_score(sc, item & 255));
                }
            }
            // ---- rows with too many candidates: all K centroids
            for (int fi = sw; fi < fqn; fi += 4) {
                const int r = sh->fullq[fi];
                const float4 x = lane < d4 ? *reinterpret_cast<const float4 *>(xs + chunk_off(r, lane, X_KB_BYTES))
                                           : make_float4(0.f, 0.f, 0.f, 0.f);
                unsigned long long best = ~0ull;
                for (int kb = 0; kb < K; kb += KC) {
                    float a[KC];
#pragma unroll
                    for (int kk = 0; kk < KC; ++kk) {
                        a[kk] = 0.f;
                        if (kb + kk < K && lane < d4)
                            a[kk] = dot4(x, *reinterpret_cast<const float4 *>(c_smem + chunk_off(kb + kk, lane, c_kb_bytes)), 0.f);
                    }
                    const float dot = reduce8_transposed(a, lane);
                    const int k = kb + slot;
                    if (k < K) {
                        float sc = fmaf(-2.f, dot, sh->cn[k]);
                        sc = (sc == sc) ? sc : CUDART_INF_F;
                        const unsigned long long p = pack_score(sc, k);
                        best = p < best ? p : best;
                    }
                }
                if ((lane & 3) == 0) atomicMin(&sh->rowbest[r], best);
            }
            group_sync(1);
            // ---- final label of this thread's row
            if (stid == 0) sh->qn = sh->fqn = 0;
            int label = MAX_K;                             // bucket of the rows beyond N
            if (live) {
                label = decided ? i1 : (int)(uint32_t)(sh->rowbest[stid] & 0xffffffffull);
                if (label < 0 || label >= K) label = 0;    // a row of NaNs still gets a valid label
                assign[row] = label;
                ++n_rows;
                n_undecided += undecided ? 1 : 0;
            }
            n_items += (lane == 0 && sw == 0) ? (unsigned long long)qn : 0ull;
            n_full += (lane == 0 && sw == 0) ? (unsigned long long)fqn : 0ull;
            // ---- group the tile's rows by label for the accumulate group (a stable counting sort)
            const unsigned peers = __match_any_sync(FULL, label);
            if (lane == __ffs(peers) - 1) sh->wcnt[par][sw][label] = __popc(peers);
            for (int i = stid; i < 4 * (MAX_K + 1); i += 128) (&sh->wcnt[par ^ 1u][0][0])[i] = 0;
            group_sync(1);
            if (sw == 0) {   // exclusive prefix over the labels: two labels per lane
                const int k0 = 2 * lane, k1 = 2 * lane + 1;
                const int t0 = sh->wcnt[par][0][k0] + sh->wcnt[par][1][k0] + sh->wcnt[par][2][k0] + sh->wcnt[par][3][k0];
                const int t1 = sh->wcnt[par][0][k1] + sh->wcnt[par][1][k1] + sh->wcnt[par][2][k1] + sh->wcnt[par][3][k1];
                int inc = t0 + t1;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int u = __shfl_up_sync(FULL, inc, o);
                    if (lane >= o) inc += u;
                }
                const int ex = inc - t0 - t1;
                sh->off[par][k0] = ex;
                sh->off[par][k1] = ex + t0;
                if (lane == 31) sh->off[par][MAX_K] = inc;
                sh->cnt[k0] += t0;
                sh->cnt[k1] += t1;
            }
            group_sync(1);
            if (live) {
                int pos = sh->off[par][label] + __popc(peers & ((1u << lane) - 1u));
                for (int w2 = 0; w2 < sw; ++w2) pos += sh->wcnt[par][w2][label];
                sh->order[par][pos] = stid;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh->lab_full[par]);
        }
        group_sync(1);
        for (int k = stid; k < K; k += 128) pcnt[(size_t)blockIdx.x * K + k] = sh->cnt[k];
        if (counters) {
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) {
                n_rows += __shfl_xor_sync(FULL, n_rows, o);
                n_undecided += __shfl_xor_sync(FULL, n_undecided, o);
            }
            if (lane == 0) {
                atomicAdd(&counters[0], n_rows);
                atomicAdd(&counters[3], n_undecided);
                atomicAdd(&counters[4], n_items);
                atomicAdd(&counters[5], n_full);
            }
        }
    } else if (warp >= A_WARP0) {
        // ---------------------------------------------------------------- accumulate group
        const int aw = warp - A_WARP0;                     // owns clusters aw, aw + 8, ...
        const int atid = threadIdx.x - A_WARP0 * 32;
        constexpr int OWN = KMAX / A_WARPS;
        const bool has_cols = lane < d4;                   // this lane's 16-byte chunk of a row is chunk `lane`
        float4 acc[OWN];
#pragma unroll
        for (int i = 0; i < OWN; ++i) acc[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        uint32_t it = 0;
        for (int64_t tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++it) {
            const uint32_t s = it % (uint32_t)stages;
            const uint32_t par = it & 1u, use = (it >> 1) & 1u;
            const uint8_t *xs = x_smem + (size_t)s * stage_bytes;
            if (!mbar_wait(&sh->lab_full[par], use, abort_flag)) break;
            if (!mbar_wait(&sh->x_full[s], (it / (uint32_t)stages) & 1u, abort_flag)) break;   // long complete: makes the tile visible here
#pragma unroll
            for (int i = 0; i < OWN; ++i) {
                const int k = aw + A_WARPS * i;
                if (k < K) {
                    const int p1 = sh->off[par][k + 1];
                    for (int p = sh->off[par][k]; p < p1; p += 4) {   // four rows at a time: loads first, adds in row order
                        float4 x[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int r = sh->order[par][min(p + u, p1 - 1)];
                            x[u] = has_cols ? *reinterpret_cast<const float4 *>(xs + chunk_off(r, lane, X_KB_BYTES))
                                            : make_float4(0.f, 0.f, 0.f, 0.f);
                        }
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            if (p + u < p1) {
                                acc[i].x += x[u].x;
                                acc[i].y += x[u].y;
                                acc[i].z += x[u].z;
                                acc[i].w += x[u].w;
                            }
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&sh->x_empty[s]);
                mbar_arrive(&sh->lab_empty[par]);
            }
        }
        // ---- publish this block's sums: every (cluster, chunk) has exactly one owner
        float4 *out = reinterpret_cast<float4 *>(psum) + (size_t)blockIdx.x * K * d4;
#pragma unroll
        for (int i = 0; i < OWN; ++i) {
            const int k = aw + A_WARPS * i;
            if (k < K && has_cols) out[(size_t)k * d4 + lane] = acc[i];
        }
        (void)atid;
    }
    __syncthreads();
    if (sh->abort && threadIdx.x == 0) ep_raise(status, EP_ERR_TIMEOUT);
    if (warp == 2) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

// rownorm[i] = (|x_i|_2, |x_i - trunc_tf32(x_i)|_2), both rounded up a little; one warp per row.
__global__ void __launch_bounds__(256) row_norms(const float *__restrict__ emb, int64_t N, int d, float2 *__restrict__ out) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, d4 = d >> 2;
    for (int64_t row = (int64_t)blockIdx.x * 8 + warp; row < N; row += (int64_t)gridDim.x * 8) {
        float x2 = 0.f, xl2 = 0.f;
        for (int q = lane; q < d4; q += 32) {
            const float4 x = ldg_stream(reinterpret_cast<const float4 *>(emb) + row * d4 + q);
            x2 = dot4(x, x, x2);
            const float4 r = make_float4(x.x - __uint_as_float(__float_as_uint(x.x) & 0xFFFFE000u),
                                         x.y - __uint_as_float(__float_as_uint(x.y) & 0xFFFFE000u),
                                         x.z - __uint_as_float(__float_as_uint(x.z) & 0xFFFFE000u),
                                         x.w - __uint_as_float(__float_as_uint(x.w) & 0xFFFFE000u));
            xl2 = dot4(r, r, xl2);
        }
        x2 = warp_sum(x2);
        xl2 = warp_sum(xl2);
        if (lane == 0) out[row] = make_float2(sqrtf(x2) * 1.000001f, sqrtf(xl2) * 1.000001f);
    }
}

}  // namespace

namespace ep {

struct TcFusedState {
    CUtensorMap map_x, map_c;
    int npad, num_kb, stages, grid;
    size_t smem;
    uint32_t tmem_cols;
};

size_t kmeans_tcf_state_bytes() { return sizeof(TcFusedState); }

static inline int tcf_npad(int K) { return std::max(16, (K + 15) / 16 * 16); }

static size_t tcf_fixed_smem(int d, int K) {
    const int num_kb = (d + KBLK - 1) / KBLK;
    return (size_t)num_kb * tcf_npad(K) * 128 + sizeof(FusedShared) + 1024;
}

bool kmeans_tcf_shape_ok(const ep_ctx *ctx, int d, int K) {
    if (d < KBLK || d > MAX_KB * KBLK || K < 1 || K > MAX_K) return false;
    const int num_kb = (d + KBLK - 1) / KBLK;
    return tcf_fixed_smem(d, K) + 2 * (size_t)num_kb * X_KB_BYTES <= (size_t)ctx->smem_optin;
}

int kmeans_tcf_grid(const ep_ctx *ctx, int64_t N) {
    return (int)std::max<int64_t>(1, std::min<int64_t>(ctx->sm_count, ceil_div(N, BM)));
}

int kmeans_tcf_prepare(ep_ctx *ctx, const float *emb, int64_t N, int d, int K, const float *centroids, float2 *rownorm,
                       TcFusedState *st, cudaStream_t stream) {
    st->npad = tcf_npad(K);
    st->num_kb = (d + KBLK - 1) / KBLK;
    const size_t fixed = tcf_fixed_smem(d, K);
    const size_t stage = (size_t)st->num_kb * X_KB_BYTES;
    st->stages = (int)std::min<size_t>(MAX_STAGES, ((size_t)ctx->smem_optin - fixed) / stage);
    st->smem = fixed + (size_t)st->stages * stage;
    st->grid = kmeans_tcf_grid(ctx, N);
    uint32_t cols = 32;
    while (cols < 2u * (uint32_t)st->npad) cols <<= 1;
    st->tmem_cols = cols;
    if (!tc_encode_kblock_map(&st->map_x, emb, N, d, BM) || !tc_encode_kblock_map(&st->map_c, centroids, K, d, st->npad))
        return fail(ctx, EP_ERR_CUDA, "cuTensorMapEncodeTiled failed for N=%lld d=%d K=%d", (long long)N, d, K);
    Timed tm(ctx, stream, EP_TIMER_KMEANS_UPDATE);
    row_norms<<<(int)std::min<int64_t>((int64_t)ctx->sm_count * 16, ceil_div(N, 8)), 256, 0, stream>>>(emb, N, d, rownorm);
    tm.end(1);
    EP_CUDA(ctx, cudaGetLastError());
    return EP_OK;
}

template <int KMAX>
static int tcf_launch(ep_ctx *ctx, const TcFusedState &st, const float *cn, const float *clo,
                      const float2 *rownorm, int64_t N, int d, int K, int32_t *assign, float *psum, int *pcnt,
                      cudaStream_t stream) {
    auto kern = kmeans_tc_fused<KMAX>;
    EP_CUDA(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)st.smem));
    unsigned long long *counters =
        ctx->opt_profile ? reinterpret_cast<unsigned long long *>(ctx->d_status + EP_COUNTER_WORD0) : nullptr;
    Timed tm(ctx, stream, EP_TIMER_KMEANS_ASSIGN);
    kern<<<st.grid, THREADS, st.smem, stream>>>(st.map_x, st.map_c, cn, clo, rownorm, N, d, K, st.npad, st.num_kb,
                                              st.stages, umma_idesc_tf32_m128(st.npad), st.tmem_cols, ~IDX_MASK, assign,
                                              psum, pcnt, counters, ctx->d_status);
    tm.end(1);
    EP_CUDA(ctx, cudaGetLastError());
    return EP_OK;
}

// One Lloyd assignment + accumulation pass; block b leaves its sums in psum[b][K][d], counts in pcnt[b][K].
int kmeans_tcf_assign(ep_ctx *ctx, const TcFusedState &st, const float *centroids, const float *cn, const float *clo,
                      const float2 *rownorm, int64_t N, int d, int K, int32_t *assign, float *psum, int *pcnt,
                      cudaStream_t stream) {
    (void)centroids;   // the kernel reads them through the tensor map made by kmeans_tcf_prepare
    if (K <= 32) return tcf_launch<32>(ctx, st, cn, clo, rownorm, N, d, K, assign, psum, pcnt, stream);
    return tcf_launch<64>(ctx, st, cn, clo, rownorm, N, d, K, assign, psum, pcnt, stream);
}

}  // namespace ep
