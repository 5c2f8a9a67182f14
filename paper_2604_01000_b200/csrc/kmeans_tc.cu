// Tensor-core assignment step of Lloyd K-Means (Algorithm 3, the clustering step) for many centroids.
//
// The scores |c_k|^2 - 2 x_i.c_k of a tile of 128 rows against all K centroids are a dense
// contraction [128 x d].[d x K].  kmeans_tc_screen runs it on the 5th-generation tensor cores in TF32:
//   - the 128-row tile of X stays in shared memory (TMA, 128-byte swizzle) for all centroid tiles;
//   - centroid tiles of 256 rows stream through a ring of shared-memory stages (TMA, L2-resident);
//   - one thread issues tcgen05.mma kind::tf32 into one of two 256-column TMEM accumulators;
//   - eight epilogue warps read the other accumulator back (tcgen05.ld) and keep, per row and per group
//     of 128 centroids, the two smallest scores with the column index packed into the low mantissa bits,
//     and the two smallest of the whole row.
// TF32 keeps 10 mantissa bits of each operand, so these scores only screen.  A row whose second smallest
// score lies outside the TF32 error bound of its smallest has its label at once: the screen kernel writes
// it.  The other rows go on a list, and kmeans_tc_resolve re-evaluates in fp32 every centroid that the
// bound cannot exclude: the best of each group whose best is within the bound of the row's overall best,
// and a whole group when its second best is within the bound as well (its hidden third might be).  The
// label is the candidate nearest in fp32 squared distance (direct form), the lowest index winning ties.
#include "ep_common.cuh"
#include "kmeans_device.cuh"
#include "tc_device.cuh"

#include <cuda.h>
#include <math_constants.h>

#include <algorithm>
#include <mutex>

namespace {

using namespace epk;
using namespace eptc;

constexpr int BM = 128;                    // rows per tile = TMEM lanes
constexpr int BN = 256;                    // centroids per accumulator
constexpr int GROUP = 128;                 // centroids per candidate group: one epilogue warp's columns
constexpr int KBLK = 32;                   // floats in one 128-byte swizzle row
constexpr int MAX_KB = 8;                  // d <= 256
constexpr int MAX_STAGES = 4;
constexpr int X_KB_BYTES = BM * 128;       // one k-block of the X tile
constexpr int C_STAGE_BYTES = BN * 128;    // one k-block of a centroid tile
constexpr int TC_THREADS = 384;            // warp 0 TMA, warp 1 MMA, warp 2 TMEM, warp 3 idle, warps 4..11 epilogue
constexpr int EPI_WARP0 = 4;
constexpr int EPI_WARPS = 8;
constexpr uint32_t TMEM_COLS = 512;

constexpr uint32_t IDESC = umma_idesc_tf32_m128(BN);

struct TcShared {
    uint64_t x_full[MAX_KB], x_empty[MAX_KB];
    uint64_t c_full[MAX_STAGES], c_empty[MAX_STAGES];
    uint64_t t_full[2], t_empty[2];
    uint64_t drain;                        // after an abort: the MMAs still in flight have completed
    uint32_t tmem_base;
    int abort;
    uint64_t h_full[4][4];                 // [tile & 3][32-row quarter]: the warp of columns 128..255 has left its result
    float4 other_half[4][BM];              // (smallest key, second smallest, group of the smallest) per row; four tiles
                                           // deep, which is further than the two accumulators let one warp run ahead
};

// Screening pass over the rows [row_begin, row_end): for row r and group g (centroids [128 g, 128 g + 128))
// cand[(r - row_begin) * G + g] = the two smallest TF32 scores of the group as packed keys.
// cn holds |c_k|^2 for k < K and a huge finite value up to the next multiple of 256.  key_mask is
// ~(GROUP - 1); it arrives as an argument so that clearing the index bits and inserting the (compile-
// time) index stay one three-input logic operation instead of two with an immediate each.
// A row with a single centroid inside the allowance (see screen_allowance) gets assign[r] here; every
// other row is appended to slow_list (row number and the centroid with the smallest key, any order) and counted
// in *slow_count, which the caller has zeroed.  counters, when given, receives the number of rows screened in word 0.
// CN_SMEM: all of cn is first copied behind the barriers in shared memory (the host checks that it fits).
template <bool CN_SMEM>
__global__ void __launch_bounds__(TC_THREADS, 1)
kmeans_tc_screen(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_c,
                 const float *__restrict__ cn, int64_t row_begin, int64_t row_end, int num_kb, int num_nt, int stages,
                 int G, uint32_t key_mask, int d, int K, const float *__restrict__ cmaxima,
                 const float2 *__restrict__ rownorm, uint2 *__restrict__ cand, int32_t *__restrict__ assign,
                 int2 *__restrict__ slow_list, int *__restrict__ slow_count, unsigned long long *counters,
                 int *status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *x_smem = smem;                                         // [num_kb][128 rows][128 B]
    uint8_t *c_smem = x_smem + (size_t)num_kb * X_KB_BYTES;         // [stages][256 rows][128 B]
    TcShared *sh = reinterpret_cast<TcShared *>(c_smem + (size_t)stages * C_STAGE_BYTES);
    float *cn_s = reinterpret_cast<float *>(sh + 1);                // [num_nt * BN] when CN_SMEM
    volatile int *abort_flag = &sh->abort;
    if (CN_SMEM)
        for (int i = threadIdx.x; i < num_nt * BN; i += TC_THREADS) cn_s[i] = cn[i];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t num_tiles = (row_end - row_begin + BM - 1) / BM;

    if (threadIdx.x == 0) {
        for (int i = 0; i < MAX_KB; ++i) {
            mbar_init(&sh->x_full[i], 1);
            mbar_init(&sh->x_empty[i], 1);
        }
        for (int i = 0; i < MAX_STAGES; ++i) {
            mbar_init(&sh->c_full[i], 1);
            mbar_init(&sh->c_empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sh->t_full[i], 1);
            mbar_init(&sh->t_empty[i], EPI_WARPS);
        }
        for (int i = 0; i < 16; ++i) mbar_init(&sh->h_full[i >> 2][i & 3], 1);
        mbar_init(&sh->drain, 1);
        sh->abort = 0;
        sh->tmem_base = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)),
                     "r"(TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer: the whole warp runs the loop
        // (uniform control flow and operands), one elected lane issues (see the elected forms in tc_device.cuh)
        {
            uint32_t it = 0, s = 0, ph = 0;                        // centroid tiles issued; ring stage and phase of the next one
            bool ok = true;
            int64_t x_tile = -1;                                   // local index of the last tile any k-block was loaded for
            const uint32_t x_base = smem_u32(x_smem), c_base = smem_u32(c_smem);
            for (int64_t lt = 0, tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++lt) {
                const int row0 = (int)(row_begin + tile * BM);
                for (int nt = 0; ok && nt < num_nt; ++nt) {
                    for (int kb = 0; kb < num_kb; ++kb, ++it) {
                        if (nt == 0) {   // this tile's rows, one k-block at a time, as the previous tile lets go of them
                            if (!(ok = __all_sync(FULL, mbar_wait(&sh->x_empty[kb], (uint32_t)(lt & 1) ^ 1u, abort_flag)))) break;
                            mbar_expect_tx_elected(&sh->x_full[kb], X_KB_BYTES);
                            tma_load_2d_elected(x_base + (uint32_t)kb * X_KB_BYTES, &map_x, kb * KBLK, row0, &sh->x_full[kb]);
                            x_tile = lt;
                        }
                        if (!(ok = __all_sync(FULL, mbar_wait(&sh->c_empty[s], ph ^ 1u, abort_flag)))) break;
                        mbar_expect_tx_elected(&sh->c_full[s], C_STAGE_BYTES);
                        tma_load_2d_elected(c_base + s * (uint32_t)C_STAGE_BYTES, &map_c, kb * KBLK, nt * BN, &sh->c_full[s]);
                        if (++s == (uint32_t)stages) {             // (no division in the issue loops)
                            s = 0;
                            ph ^= 1u;
                        }
                    }
                }
            }
            if (lane == 0 && (!ok || *abort_flag)) {
                // On the way out after an abort: the loads already issued get time to land, so that nothing of this
                // block's own still writes into its shared memory when it leaves.  (A k-block of x whose barrier is
                // still in an earlier phase was not loaded for the last tile: the wait then runs to its limit.)
#pragma unroll 1
                for (uint32_t j = it > (uint32_t)stages ? it - (uint32_t)stages : 0u; j < it; ++j)
                    mbar_wait_quiet(&sh->c_full[j % (uint32_t)stages], (j / (uint32_t)stages) & 1u, DRAIN_LIMIT_CLOCKS);
                if (x_tile >= 0)
#pragma unroll 1
                    for (int kb = 0; kb < num_kb; ++kb) mbar_wait_quiet(&sh->x_full[kb], (uint32_t)(x_tile & 1), DRAIN_LIMIT_CLOCKS);
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer: the whole warp runs the loop,
        // one elected lane issues
        {
            uint32_t it = 0, acc = 0, s = 0, ph = 0;
            bool ok = true;
            const uint32_t x_base = smem_u32(x_smem), c_base = smem_u32(c_smem);
            static_assert(KBLK == 32, "umma_tf32_kblock_elected issues the four K-steps of a 32-float k-block");
            for (int64_t lt = 0, tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++lt) {
                for (int nt = 0; ok && nt < num_nt; ++nt, ++acc) {
                    const uint32_t buf = acc & 1u, use = (acc >> 1) & 1u;
                    if (!(ok = __all_sync(FULL, mbar_wait(&sh->t_empty[buf], use ^ 1u, abort_flag)))) break;
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + buf * BN;
                    for (int kb = 0; kb < num_kb; ++kb, ++it) {
                        if (nt == 0 && !(ok = __all_sync(FULL, mbar_wait(&sh->x_full[kb], (uint32_t)(lt & 1), abort_flag)))) break;
                        if (!(ok = __all_sync(FULL, mbar_wait(&sh->c_full[s], ph, abort_flag)))) break;
                        tc_fence_after();
                        umma_tf32_kblock_elected(d_tmem, umma_desc(x_base + (uint32_t)kb * X_KB_BYTES),
                                                 umma_desc(c_base + s * (uint32_t)C_STAGE_BYTES), IDESC, (uint32_t)kb);
                        umma_commit_elected(&sh->c_empty[s]);
                        if (nt == num_nt - 1) umma_commit_elected(&sh->x_empty[kb]);
                        if (++s == (uint32_t)stages) {
                            s = 0;
                            ph ^= 1u;
                        }
                    }
                    if (ok) umma_commit_elected(&sh->t_full[buf]);
                }
            }
            if (__any_sync(FULL, !ok || *abort_flag)) {
                // after an abort the accumulators are given back at the end of the kernel: first every MMA issued
                // here must have completed (the commit comes from the lane that issued them: the same election)
                umma_commit_elected(&sh->drain);
                if (lane == 0) mbar_wait_quiet(&sh->drain, 0u, DRAIN_LIMIT_CLOCKS);
            }
        }
    } else if (warp >= EPI_WARP0) {
        // ---------------------------------------------------------------- epilogue
        const int quad = warp & 3;                         // TMEM lanes 32 quad .. 32 quad + 31 belong to this warp
        const int half = (warp - EPI_WARP0) >> 2;          // which 128 of the accumulator's 256 columns
        const float cmax2 = cmaxima[0], clomax = cmaxima[1];   // largest |c_k|^2 and largest rounding residual
        const float cmax = sqrtf(cmax2) * 1.000001f;
        uint32_t acc = 0, n_live = 0;
        bool ok = true;
        for (int64_t lt = 0, tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++lt) {
            const int64_t row = row_begin + tile * BM + quad * 32 + lane;
            float2 nr = make_float2(0.f, 0.f);
            if (row < row_end) nr = __ldg(rownorm + row);
            const float allow2 = 2.f * screen_allowance(nr.x, nr.y, cmax, cmax2, clomax, d);
            float run1 = __uint_as_float(KEY_INIT), run2 = run1;   // the row's two smallest keys over this half's groups
            int rung = 0;                                          // group of run1
            float cut = run1;                                      // scores above it are out of the race
            for (int nt = 0; ok && nt < num_nt; ++nt, ++acc) {
                const uint32_t buf = acc & 1u, use = (acc >> 1) & 1u;
                if (!(ok = mbar_wait(&sh->t_full[buf], use, abort_flag))) break;
                tc_fence_after();
                const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + buf * BN + half * GROUP;
                const float *cn_grp = cn + (size_t)nt * BN + half * GROUP;
                float a1 = __uint_as_float(KEY_INIT), a2 = a1, b1 = a1, b2 = a1;
                // 32 columns at a time; the next 32 are on their way from TMEM while these are ranked
                // A score above cut = (smallest key this warp has seen for the row) + twice the allowance can
                // never be the row's fp32 argmin nor tie with it, and the final threshold is no larger than any
                // earlier cut: such scores are dropped eight at a time, before they are packed and ranked.
                auto rank32 = [&](const uint32_t (&v)[32], int c) {
#pragma unroll
                    for (int h = 0; h < 4; ++h) {
                        float s[8];
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            float4 n4;
                            if (CN_SMEM)
                                n4 = *(reinterpret_cast<const float4 *>(cn_s + nt * BN + half * GROUP + c * 32 + h * 8) + q);
                            else
                                n4 = __ldg(reinterpret_cast<const float4 *>(cn_grp + c * 32 + h * 8) + q);
                            s[q * 4 + 0] = fmaf(-2.f, __uint_as_float(v[h * 8 + q * 4 + 0]), n4.x);
                            s[q * 4 + 1] = fmaf(-2.f, __uint_as_float(v[h * 8 + q * 4 + 1]), n4.y);
                            s[q * 4 + 2] = fmaf(-2.f, __uint_as_float(v[h * 8 + q * 4 + 2]), n4.z);
                            s[q * 4 + 3] = fmaf(-2.f, __uint_as_float(v[h * 8 + q * 4 + 3]), n4.w);
                        }
                        const float m = fmin3(fmin3(s[0], s[1], s[2]), fmin3(s[3], s[4], s[5]), fminf(s[6], s[7]));
                        if (__any_sync(FULL, m <= cut)) {   // one lane is enough: the whole warp ranks the block
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const float key =
                                    __uint_as_float((__float_as_uint(s[j]) & key_mask) | (uint32_t)(c * 32 + h * 8 + j));
                                if (j & 1)
                                    keep_two(b1, b2, key);
                                else
                                    keep_two(a1, a2, key);
                            }
                            cut = fminf(cut, fminf(a1, b1) + allow2);
                        }
                    }
                };
                uint32_t va[32], vb[32];
                tmem_ld32_issue(taddr, va);
                tmem_ld_wait(va);
                tmem_ld32_issue(taddr + 32, vb);
                rank32(va, 0);
                tmem_ld_wait(vb);
                tmem_ld32_issue(taddr + 64, va);
                rank32(vb, 1);
                tmem_ld_wait(va);
                tmem_ld32_issue(taddr + 96, vb);
                rank32(va, 2);
                tmem_ld_wait(vb);
                tc_fence_before();                          // every column is in registers: the accumulator is free
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh->t_empty[buf]);
                rank32(vb, 3);
                const float k1 = fminf(a1, b1);
                const float k2 = fminf(fmaxf(a1, b1), fminf(a2, b2));
                const int g = nt * 2 + half;
                if (row < row_end)
                    cand[(size_t)(row - row_begin) * G + g] = make_uint2(__float_as_uint(k1), __float_as_uint(k2));
                rung = k1 < run1 ? g : rung;
                run2 = fminf(fmaxf(run1, k1), fminf(run2, k2));
                run1 = fminf(run1, k1);
            }
            if (!ok) break;
            // the two warps that own these 32 rows meet
            float4 *slot = &sh->other_half[lt & 3][quad * 32 + lane];
            if (half == 1) {
                *slot = make_float4(run1, run2, __int_as_float(rung), 0.f);
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh->h_full[lt & 3][quad]);
            } else {
                if (!(ok = mbar_wait(&sh->h_full[lt & 3][quad], (uint32_t)((lt >> 2) & 1), abort_flag))) break;
                const float4 o = *slot;
                const float lo = fminf(run1, o.x);
                const float second = fminf(fmaxf(run1, o.x), fminf(run2, o.y));
                const int glo = o.x < run1 ? __float_as_int(o.z) : rung;
                const int kone = glo * GROUP + (int)(__float_as_uint(lo) & IDX_MASK);
                const float thr = lo + allow2;
                const bool live = row < row_end;
                // one centroid inside the allowance, every other one outside: it is the fp32 argmin
                const bool fast = live && second > thr && kone < K;
                if (fast) assign[row] = kone;
                n_live += live ? 1u : 0u;
                const unsigned slow = __ballot_sync(FULL, live && !fast);
                if (slow) {
                    int base = 0;
                    if (lane == 0) base = atomicAdd(slow_count, __popc(slow));
                    base = __shfl_sync(FULL, base, 0);
                    if (live && !fast && EP_INDEX_OK(base + __popc(slow & ((1u << lane) - 1u)), row_end - row_begin, status))
                        slow_list[base + __popc(slow & ((1u << lane) - 1u))] = make_int2((int)(row - row_begin), kone);
                }
            }
        }
        if (counters && half == 0) {
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) n_live += __shfl_xor_sync(FULL, n_live, o);
            if (lane == 0 && n_live) atomicAdd(&counters[0], (unsigned long long)n_live);
        }
    }
    __syncthreads();
    if (sh->abort && threadIdx.x == 0) ep_raise(status, EP_ERR_TIMEOUT);
    if (warp == 2) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// out[0] = max_k cn[k], out[1] = max_k clo[k] (one block).
__global__ void __launch_bounds__(1024) centroid_maxima(const float *__restrict__ cn, const float *__restrict__ clo, int K,
                                                        float *__restrict__ out) {
    __shared__ float red[2][32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float m2 = 0.f, ml = 0.f;
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
        m2 = fmaxf(m2, cn[k]);
        ml = fmaxf(ml, clo[k]);
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
        m2 = fmaxf(m2, __shfl_xor_sync(FULL, m2, o));
        ml = fmaxf(ml, __shfl_xor_sync(FULL, ml, o));
    }
    if (lane == 0) {
        red[0][warp] = m2;
        red[1][warp] = ml;
    }
    __syncthreads();
    if (warp == 0) {
        m2 = red[0][lane];
        ml = red[1][lane];
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) {
            m2 = fmaxf(m2, __shfl_xor_sync(FULL, m2, o));
            ml = fmaxf(ml, __shfl_xor_sync(FULL, ml, o));
        }
        if (lane == 0) {
            out[0] = m2;
            out[1] = ml;
        }
    }
}

// Exact fp32 decision for the rows the screening pass listed (slow_list holds the row number relative to
// row_begin and the centroid with the row's smallest key, *slow_count entries).  One warp per row; lane l holds
// the 16-byte slices l, l+32, ... of the row, as in the CUDA-core kernels.  rownorm[i] = (|x_i|,
// |x_i - trunc_tf32(x_i)|), computed once per call.
//
// The listed centroid is evaluated first (its row of C comes with the prefetch of the row), both as the score
// f = |c|^2 - 2 x.c and as the squared distance.  With E the allowance, a centroid h can only be as near as the
// listed one if its key is at most f + E (key(h) <= score(h) + E <= f + E): that threshold, never larger than the
// screening pass's own (smallest key + 2E), decides which other centroids are evaluated and which groups are
// scanned.  The label is the candidate with the smallest squared distance in the direct form sum_j (x_j - c_j)^2,
// lowest index on ties: the rows that arrive here are the near ties, and only the direct form separates two
// distances whose gap is small beside |x|^2 and |c|^2.
template <int VPL>
__global__ void __launch_bounds__(256) kmeans_tc_resolve(const float *__restrict__ emb, int64_t row_begin, int rows, int d, int K,
                                                         int G, const float *__restrict__ C,
                                                         const float *__restrict__ cn,
                                                         const float *__restrict__ cmaxima,
                                                         const float2 *__restrict__ rownorm,
                                                         const uint2 *__restrict__ cand,
                                                         const int2 *__restrict__ slow_list,
                                                         const int *__restrict__ slow_count,
                                                         int32_t *__restrict__ assign, unsigned long long *counters) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, d4 = d >> 2;
    const float cmax2 = cmaxima[0], clomax = cmaxima[1];   // largest |c_k|^2 and largest rounding residual
    const float cmax = sqrtf(cmax2) * 1.000001f;
    unsigned long long n_single = 0, n_scan = 0, n_rows = 0;
    const float4 *C4 = reinterpret_cast<const float4 *>(C);
    const int slot = lane_chunk_slot(lane);
    const int n_slow = min(*slow_count, rows);            // the list never holds more than the chunk's rows
    auto entry = [&](int64_t i) {
        int2 e = make_int2(-1, -1);
        if (i < n_slow) {
            e = slow_list[i];
            e.x = min(max(e.x, 0), rows - 1);
        }
        return e;
    };

    // Each warp fetches its next row (keys, norms, the row itself, the first centroid) while it works on the
    // current one, and the list entry after that.
    const int stride = (int)gridDim.x * 8;
    uint2 key_n = make_uint2(KEY_INIT, KEY_INIT);
    float2 nr_n = make_float2(0.f, 0.f);
    float4 x_n[VPL], c_n[VPL];
    float cn_n = 0.f;
    auto fetch = [&](int2 e) {
        if (e.x >= 0) {
            const int64_t r = row_begin + e.x;
            if (lane < G) key_n = cand[(size_t)e.x * G + lane];
            nr_n = __ldg(rownorm + r);
            const int kf = (unsigned)e.y < (unsigned)K ? e.y : 0;
            cn_n = __ldg(cn + kf);
#pragma unroll
            for (int v = 0; v < VPL; ++v) {
                const int q = lane + 32 * v;
                x_n[v] = q < d4 ? ldg_stream(reinterpret_cast<const float4 *>(emb) + r * d4 + q) : make_float4(0.f, 0.f, 0.f, 0.f);
                c_n[v] = q < d4 ? __ldg(C4 + (size_t)kf * d4 + q) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
    };
    const int first = (int)blockIdx.x * 8 + warp;
    int2 ent = entry(first);
    int2 ent_n = entry((int64_t)first + stride);
    fetch(ent);
    for (int i = first; i < n_slow; i += stride) {
        ++n_rows;
        const int rel = ent.x;
        const int kfirst = (unsigned)ent.y < (unsigned)K ? ent.y : -1;   // -1: nothing usable was listed (a row of NaNs)
        const int64_t row = row_begin + rel;
        const uint2 *cr = cand + (size_t)rel * G;
        const float2 nr = nr_n;
        const uint2 key0 = lane < G ? key_n : make_uint2(KEY_INIT, KEY_INIT);   // this lane's group of the first 32
        float4 x[VPL];
        float acc_f = 0.f, dist_f = 0.f;
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            x[v] = x_n[v];
            acc_f = dot4(x[v], c_n[v], acc_f);
            dist_f = dist4(x[v], c_n[v], dist_f);
        }
        const float cn_f = cn_n;
        ent = ent_n;
        ent_n = entry((int64_t)i + 2 * (int64_t)stride);
        fetch(ent);
        // Candidates are compared by their squared distance in the direct form sum_j (x_j - c_j)^2 (accurate
        // relative to the distance itself: these are the near ties).  The score |c|^2 - 2 x.c of the listed
        // centroid only places the threshold below.
        float best = CUDART_INF_F;
        int bidx = 0x7fffffff;
        float score_first = CUDART_INF_F;
        if (kfirst >= 0) {
            const float sf = fmaf(-2.f, warp_sum(acc_f), cn_f), df = warp_sum(dist_f);
            score_first = (sf == sf) ? sf : CUDART_INF_F;
            best = (df == df) ? df : CUDART_INF_F;
            bidx = kfirst;
            ++n_single;
        }
        // no centroid whose key lies above this can be as near as the listed one
        const float thr = score_first + screen_allowance(nr.x, nr.y, cmax, cmax2, clomax, d);

        bool lanes_differ = false;                 // set once a lane holds a score the others do not
        for (int g0 = 0; g0 < G; g0 += 32) {
            const int g = g0 + lane;
            uint2 key = key0;
            if (g0 > 0) key = g < G ? cr[g] : make_uint2(KEY_INIT, KEY_INIT);
            // the centroid scored above is the first key of its group: it is not scored again on its own
            const bool is_first = kfirst >= 0 && g == (kfirst >> 7) && (int)(key.x & IDX_MASK) == (kfirst & (int)IDX_MASK);
            const unsigned m1 = __ballot_sync(FULL, __uint_as_float(key.x) <= thr);
            const unsigned mboth = __ballot_sync(FULL, __uint_as_float(key.y) <= thr);
            const unsigned mfirst = __ballot_sync(FULL, is_first);
            // groups with one centroid inside the allowance: score those centroids (one or two of them is the
            // usual case: a plain warp sum each; more go eight per reduction)
            unsigned ms = m1 & ~mboth & ~mfirst;
            if (__popc(ms) <= 4) {
                while (ms) {   // two at a time: their loads and their reductions overlap
                    const int src0 = __ffs(ms) - 1;
                    ms &= ms - 1;
                    const bool two = ms != 0u;
                    const int src1 = two ? __ffs(ms) - 1 : src0;
                    ms &= ms - 1;
                    const int k0 = (g0 + src0) * GROUP + (int)(__shfl_sync(FULL, key.x, src0) & IDX_MASK);
                    const int k1 = (g0 + src1) * GROUP + (int)(__shfl_sync(FULL, key.x, src1) & IDX_MASK);
                    const bool use0 = k0 < K, use1 = two && k1 < K;
                    const int kk0 = use0 ? k0 : 0, kk1 = use1 ? k1 : 0;
                    float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
                    for (int v = 0; v < VPL; ++v) {
                        const int q = lane + 32 * v;
                        if (q < d4) {
                            const float4 c0 = __ldg(C4 + (size_t)kk0 * d4 + q), c1 = __ldg(C4 + (size_t)kk1 * d4 + q);
                            acc0 = dist4(x[v], c0, acc0);
                            acc1 = dist4(x[v], c1, acc1);
                        }
                    }
#pragma unroll
                    for (int m = 16; m >= 1; m >>= 1) {   // two warp_sum trees side by side
                        acc0 += __shfl_xor_sync(FULL, acc0, m);
                        acc1 += __shfl_xor_sync(FULL, acc1, m);
                    }
                    float s0 = acc0, s1 = acc1;
                    s0 = (s0 == s0) ? s0 : CUDART_INF_F;
                    s1 = (s1 == s1) ? s1 : CUDART_INF_F;
                    n_single += (use0 ? 1 : 0) + (use1 ? 1 : 0);
                    if (use0 && (s0 < best || (s0 == best && k0 < bidx))) {
                        best = s0;
                        bidx = k0;
                    }
                    if (use1 && (s1 < best || (s1 == best && k1 < bidx))) {
                        best = s1;
                        bidx = k1;
                    }
                }
            }
            lanes_differ |= (ms | (m1 & mboth)) != 0u;
            while (ms) {
                float acc[KC];
                int myk = -1;
#pragma unroll
                for (int kk = 0; kk < KC; ++kk) {
                    acc[kk] = 0.f;
                    if (ms) {
                        const int src = __ffs(ms) - 1;
                        ms &= ms - 1;
                        const int kone = (g0 + src) * GROUP + (int)(__shfl_sync(FULL, key.x, src) & IDX_MASK);
                        if (kone < K) {
                            ++n_single;
                            if (kk == slot) myk = kone;
#pragma unroll
                            for (int v = 0; v < VPL; ++v) {
                                const int q = lane + 32 * v;
                                if (q < d4) acc[kk] = dist4(x[v], __ldg(C4 + (size_t)kone * d4 + q), acc[kk]);
                            }
                        }
                    }
                }
                float s = reduce8_transposed(acc, lane);
                if (myk >= 0) {
                    s = (s == s) ? s : CUDART_INF_F;
                    if (s < best || (s == best && myk < bidx)) {
                        best = s;
                        bidx = myk;
                    }
                }
            }
            // groups with two inside: a third may hide behind them, so the whole group is scored
            unsigned mscan = m1 & mboth;
            while (mscan) {
                const int src = __ffs(mscan) - 1;
                mscan &= mscan - 1;
                ++n_scan;
                const int kbase = (g0 + src) * GROUP;
                const int kend = min(K, kbase + GROUP);
                for (int kb = kbase; kb < kend; kb += KC) {
                    float acc[KC];
#pragma unroll
                    for (int kk = 0; kk < KC; ++kk) {
                        acc[kk] = 0.f;
                        if (kb + kk < kend) {
#pragma unroll
                            for (int v = 0; v < VPL; ++v) {
                                const int q = lane + 32 * v;
                                if (q < d4) acc[kk] = dist4(x[v], __ldg(C4 + (size_t)(kb + kk) * d4 + q), acc[kk]);
                            }
                        }
                    }
                    const float dist = reduce8_transposed(acc, lane);
                    const int k = kb + slot;
                    float s = k < kend ? dist : CUDART_INF_F;
                    s = (s == s) ? s : CUDART_INF_F;
                    if (s < best || (s == best && k < bidx)) {
                        best = s;
                        bidx = k;
                    }
                }
            }
        }
        if (lanes_differ) {
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) {
                const float ov = __shfl_xor_sync(FULL, best, o);
                const int oi = __shfl_xor_sync(FULL, bidx, o);
                if (ov < best || (ov == best && oi < bidx)) {
                    best = ov;
                    bidx = oi;
                }
            }
        }
        if (lane == 0) assign[row] = (bidx >= 0 && bidx < K) ? bidx : 0;   // a row of NaNs still gets a valid label
    }
    if (counters && lane == 0) {
        atomicAdd(&counters[4], n_rows);
        atomicAdd(&counters[1], n_single);
        atomicAdd(&counters[2], n_scan);
    }
}

}  // namespace

namespace ep {

// ---- host ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

// Map over a row-major [rows x d] fp32 matrix whose boxes are `box_rows` rows of one 128-byte k-block.
bool tc_encode_kblock_map(void *map_out, const float *base, int64_t rows, int d, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    CUtensorMap *map = static_cast<CUtensorMap *>(map_out);
    const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)d * sizeof(float)};
    const cuuint32_t box[2] = {(cuuint32_t)32, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


// The same matrix (d a multiple of 32) seen as [d / 32 k-blocks][rows][32 floats], so that ONE box brings a tile of
// `box_rows` rows with all its k-blocks, laid out in shared memory k-block after k-block exactly as the boxes of the map
// above leave them one by one.  Coordinates: (0, first row, 0).
bool tc_encode_rowtile_map(void *map_out, const float *base, int64_t rows, int d, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn || d % 32 != 0 || d / 32 > 256 || box_rows > 256) return false;
    CUtensorMap *map = static_cast<CUtensorMap *>(map_out);
    const cuuint64_t dims[3] = {(cuuint64_t)32, (cuuint64_t)rows, (cuuint64_t)(d / 32)};
    const cuuint64_t strides[2] = {(cuuint64_t)d * sizeof(float), (cuuint64_t)32 * sizeof(float)};
    const cuuint32_t box[3] = {(cuuint32_t)32, (cuuint32_t)box_rows, (cuuint32_t)(d / 32)};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct TcState {
    CUtensorMap map_x, map_c;
};

size_t kmeans_tc_state_bytes() { return sizeof(TcState); }

bool kmeans_tc_shape_ok(const ep_ctx *ctx, int d, int K) {
    (void)K;
    if (d < KBLK || d > MAX_KB * KBLK) return false;
    const int num_kb = (d + KBLK - 1) / KBLK;
    return (size_t)num_kb * X_KB_BYTES + 2 * (size_t)C_STAGE_BYTES + sizeof(TcShared) + 1024 <= (size_t)ctx->smem_optin;
}

int kmeans_tc_groups(int K) { return (K + BN - 1) / BN * 2; }

int64_t kmeans_tc_chunk_rows(const ep_ctx *ctx, int64_t N, int K) {
    const int64_t wave = (int64_t)BM * ctx->sm_count;                       // rows one pass of the grid covers
    const int64_t budget = ((int64_t)ctx->opt_cand_mb << 20) / ((int64_t)kmeans_tc_groups(K) * (int64_t)sizeof(uint2));
    const int64_t rows = std::max<int64_t>(1, budget / wave) * wave;
    return std::min<int64_t>(rows, ceil_div(N, BM) * BM);
}

// Candidate keys of one chunk of rows, the chunk's list of undecided rows, and one list length per chunk.
size_t kmeans_tc_cand_bytes(const ep_ctx *ctx, int64_t N, int K) {
    const int64_t chunk = kmeans_tc_chunk_rows(ctx, N, K);
    return (size_t)chunk * kmeans_tc_groups(K) * sizeof(uint2) + (size_t)chunk * sizeof(int2) +
           (size_t)ceil_div(N, chunk) * sizeof(int);
}

int kmeans_tc_prepare(ep_ctx *ctx, const float *emb, int64_t N, int d, int K, const float *centroids, TcState *st) {
    if (!tc_encode_kblock_map(&st->map_x, emb, N, d, BM) || !tc_encode_kblock_map(&st->map_c, centroids, K, d, BN))
        return fail(ctx, EP_ERR_CUDA, "cuTensorMapEncodeTiled failed for N=%lld d=%d K=%d", (long long)N, d, K);
    return EP_OK;
}

// One assignment step on the tensor-core path: labels of all N rows against `centroids` / `cn`.
int kmeans_tc_assign(ep_ctx *ctx, const TcState &st, const float *emb, int64_t N, int d, int K,
                     const float *centroids, const float *cn, const float *clo, float *cmaxima, const float2 *rownorm,
                     int32_t *assign, void *cand_ws, cudaStream_t stream) {
    const int num_kb = (d + KBLK - 1) / KBLK;
    const int num_nt = (K + BN - 1) / BN;
    const int G = num_nt * 2;
    size_t fixed = (size_t)num_kb * X_KB_BYTES + sizeof(TcShared) + 1024;
    int stages = (int)std::min<size_t>(MAX_STAGES, ((size_t)ctx->smem_optin - fixed) / C_STAGE_BYTES);
    // |c|^2 of every centroid in shared memory too, unless that would cost the ring more than one stage
    const size_t cn_bytes = (size_t)num_nt * BN * sizeof(float);
    bool cn_smem = false;
    if (fixed + cn_bytes + 2 * (size_t)C_STAGE_BYTES <= (size_t)ctx->smem_optin) {
        const int with = (int)std::min<size_t>(MAX_STAGES, ((size_t)ctx->smem_optin - fixed - cn_bytes) / C_STAGE_BYTES);
        if (with >= std::min(stages, 3)) {
            cn_smem = true;
            stages = with;
            fixed += cn_bytes;
        }
    }
    const size_t smem = fixed + (size_t)stages * C_STAGE_BYTES;
    auto screen = cn_smem ? kmeans_tc_screen<true> : kmeans_tc_screen<false>;
    EP_CUDA(ctx, cudaFuncSetAttribute(screen, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int64_t chunk = kmeans_tc_chunk_rows(ctx, N, K);
    const int64_t nchunks = ceil_div(N, chunk);
    uint2 *cand = static_cast<uint2 *>(cand_ws);
    int2 *slow_list = reinterpret_cast<int2 *>(cand + (size_t)chunk * G);
    int *slow_count = reinterpret_cast<int *>(slow_list + chunk);       // one counter per chunk
    unsigned long long *counters =
        ctx->opt_profile ? reinterpret_cast<unsigned long long *>(ctx->d_status + EP_COUNTER_WORD0) : nullptr;
    {
        Timed tm(ctx, stream, EP_TIMER_KMEANS_RESOLVE);
        EP_CUDA(ctx, cudaMemsetAsync(slow_count, 0, sizeof(int) * (size_t)nchunks, stream));
        centroid_maxima<<<1, 1024, 0, stream>>>(cn, clo, K, cmaxima);
        tm.end(1);
    }
    int launches = 0;
    for (int64_t r0 = 0, c = 0; r0 < N; r0 += chunk, ++c) {
        const int64_t r1 = std::min(N, r0 + chunk);
        const int grid = (int)std::min<int64_t>(ctx->sm_count, ceil_div(r1 - r0, BM));
        {
            Timed tm(ctx, stream, EP_TIMER_KMEANS_ASSIGN);
            screen<<<grid, TC_THREADS, smem, stream>>>(st.map_x, st.map_c, cn, r0, r1, num_kb, num_nt, stages, G,
                                                               ~IDX_MASK, d, K, cmaxima, rownorm, cand, assign, slow_list,
                                                               slow_count + c, counters, ctx->d_status);
            tm.end(1);
        }
        Timed tm(ctx, stream, EP_TIMER_KMEANS_RESOLVE);
        const int rgrid = (int)std::min<int64_t>((int64_t)ctx->sm_count * 8, ceil_div(r1 - r0, 8));
        if (d <= 128)
            kmeans_tc_resolve<1><<<rgrid, 256, 0, stream>>>(emb, r0, (int)(r1 - r0), d, K, G, centroids, cn, cmaxima, rownorm, cand, slow_list,
                                                           slow_count + c, assign, counters);
        else
            kmeans_tc_resolve<2><<<rgrid, 256, 0, stream>>>(emb, r0, (int)(r1 - r0), d, K, G, centroids, cn, cmaxima, rownorm, cand, slow_list,
                                                           slow_count + c, assign, counters);
        tm.end(1);
        launches += 2;
    }
    (void)launches;
    EP_CUDA(ctx, cudaGetLastError());
    return EP_OK;
}

}  // namespace ep
