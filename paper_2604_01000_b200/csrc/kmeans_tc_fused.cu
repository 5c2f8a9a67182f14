// Fused assign-and-accumulate pass of Lloyd K-Means (Algorithm 3, line 1) for few centroids
// (K <= 128, d <= 128) on the tensor cores: one read of the embedding matrix per iteration.
//
// A persistent block per SM streams 128-row tiles of X through a ring of shared-memory stages (TMA,
// 128-byte swizzle).  All K centroids (their TF32-rounded copy) sit in shared memory for the whole
// launch.  Per tile:
//   1. one thread issues tcgen05.mma kind::tf32: scores [128 x K] into one of two TMEM accumulators;
//   2. four warps read the accumulator back, one row per thread, and keep the two smallest packed
//      (score | column) keys.  If the second key is farther from the first than the TF32 error bound
//      of that row allows, the first is provably the fp32 argmin and becomes the label.  Otherwise the
//      row is queued;
//   3. queued rows are scored against all K centroids in fp32 (a warp per row, the row read from the
//      shared-memory tile) with the lowest index winning ties, exactly as the CUDA-core kernels do;
//   4. every (cluster, 16-byte column chunk) pair has one owning thread that adds up, in row order,
//      the tile's rows carrying that label, straight from the shared-memory tile into registers.
// The block's sums and counts go to psum[block] / pcnt[block] at the end; the order of every addition
// is fixed by the launch shape, so results repeat bit for bit.
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
constexpr int THREADS = 384;            // warp 0 TMA, warp 1 MMA, warp 2 TMEM alloc, warp 3 idle, warps 4..11 consumers
constexpr int CONS_WARP0 = 4;
constexpr int CONS_WARPS = 8;

struct FusedShared {
    uint64_t x_full[MAX_STAGES], x_empty[MAX_STAGES];
    uint64_t c_full;
    uint64_t t_full[2], t_empty[2];
    uint32_t tmem_base;
    int abort;
    int stop[2];       // the abort flag as consumer thread 0 saw it before a tile's first consumer barrier
    int qn[2];
    int queue[2][BM];
    int lab[2][BM];
    float red[2][8];
};

__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// 16-byte chunk q of row r of a swizzled row tile (k-blocks of 128 rows x 128 bytes).
__device__ __forceinline__ float4 tile_chunk(const uint8_t *xs, int r, int q) {
    return *reinterpret_cast<const float4 *>(xs + (size_t)(q >> 3) * X_KB_BYTES + r * 128 + (((q & 7) ^ (r & 7)) << 4));
}

// KPW = clusters per consumer warp (K <= 8 KPW).  rownorm[i] = (|x_i|, |x_i - trunc_tf32(x_i)|).
template <int KPW>
__global__ void __launch_bounds__(THREADS, 1)
kmeans_tc_fused(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_c,
                const float *__restrict__ C, const float *__restrict__ cn, const float *__restrict__ clo,
                const float2 *__restrict__ rownorm, int64_t N, int d, int K, int npad, int num_kb, int stages,
                uint32_t idesc, uint32_t tmem_cols, uint32_t key_mask, int32_t *__restrict__ assign,
                float *__restrict__ psum, int *__restrict__ pcnt, unsigned long long *counters, int *status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int stage_bytes = num_kb * X_KB_BYTES;
    uint8_t *x_smem = smem;                                          // [stages][num_kb][128 rows][128 B]
    uint8_t *c_smem = x_smem + (size_t)stages * stage_bytes;         // [num_kb][npad rows][128 B]
    FusedShared *sh = reinterpret_cast<FusedShared *>(c_smem + (size_t)num_kb * npad * 128);
    volatile int *abort_flag = &sh->abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t num_tiles = (N + BM - 1) / BM;

    if (threadIdx.x == 0) {
        for (int i = 0; i < MAX_STAGES; ++i) {
            mbar_init(&sh->x_full[i], 1);
            mbar_init(&sh->x_empty[i], CONS_WARPS);
        }
        mbar_init(&sh->c_full, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sh->t_full[i], 1);
            mbar_init(&sh->t_empty[i], 4);
        }
        sh->abort = 0;
        sh->tmem_base = 0;
        sh->qn[0] = sh->qn[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
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
            mbar_expect_tx(&sh->c_full, (uint32_t)(num_kb * npad * 128));
            for (int kb = 0; kb < num_kb; ++kb)
                tma_load_2d(c_smem + (size_t)kb * npad * 128, &map_c, kb * KBLK, 0, &sh->c_full);
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
                    const uint64_t bdesc = umma_desc(smem_u32(c_smem + (size_t)kb * npad * 128));
#pragma unroll
                    for (int ks = 0; ks < KBLK / 8; ++ks)
                        umma_tf32(d_tmem, adesc + (uint64_t)(2 * ks), bdesc + (uint64_t)(2 * ks), idesc,
                                  (kb | ks) != 0 ? 1u : 0u);
                }
                umma_commit(&sh->t_full[buf]);
            }
        }
    } else if (warp >= CONS_WARP0) {
        // ---------------------------------------------------------------- consumers
        const int cw = warp - CONS_WARP0;                  // 0..7
        const int ctid = threadIdx.x - CONS_WARP0 * 32;    // 0..255
        const int d4 = d >> 2;
        // largest centroid norm and rounding residual
        {
            float m2 = 0.f, ml = 0.f;
            for (int k = ctid; k < K; k += 256) {
                m2 = fmaxf(m2, cn[k]);
                ml = fmaxf(ml, clo[k]);
            }
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) {
                m2 = fmaxf(m2, __shfl_xor_sync(FULL, m2, o));
                ml = fmaxf(ml, __shfl_xor_sync(FULL, ml, o));
            }
            if (lane == 0) {
                sh->red[0][cw] = m2;
                sh->red[1][cw] = ml;
            }
        }
        consumer_sync();
        float cmax2 = sh->red[0][0], clomax = sh->red[1][0];
#pragma unroll
        for (int w = 1; w < 8; ++w) {
            cmax2 = fmaxf(cmax2, sh->red[0][w]);
            clomax = fmaxf(clomax, sh->red[1][w]);
        }
        const float cmax = sqrtf(cmax2) * 1.000001f;
        const float4 *C4 = reinterpret_cast<const float4 *>(C);
        const int slot = lane_chunk_slot(lane);

        float4 acc[KPW];
        int cnt[KPW];
#pragma unroll
        for (int i = 0; i < KPW; ++i) {
            acc[i] = make_float4(0.f, 0.f, 0.f, 0.f);
            cnt[i] = 0;
        }
        unsigned long long n_rows = 0, n_queued = 0;

        uint32_t it = 0;
        for (int64_t tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++it) {
            const uint32_t s = it % (uint32_t)stages;
            const uint32_t buf = it & 1u, use = (it >> 1) & 1u, par = it & 1u;
            const uint8_t *xs = x_smem + (size_t)s * stage_bytes;
            const int64_t row0 = tile * BM;
            if (cw < 4) {
                // ---- one row per thread: the two best screened scores, then label or queue
                const int r = cw * 32 + lane;
                const int64_t row = row0 + r;
                if (mbar_wait(&sh->t_full[buf], use, abort_flag)) {
                    tc_fence_after();
                    const uint32_t taddr = tmem_base + ((uint32_t)(cw * 32) << 16) + buf * (uint32_t)npad;
                    float a1 = __uint_as_float(KEY_INIT), a2 = a1, b1 = a1, b2 = a1;
                    for (int c = 0; c < npad; c += 16) {
                        uint32_t v[16];
                        tmem_ld16(taddr + c, v);
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const float4 n4 = __ldg(reinterpret_cast<const float4 *>(cn + c) + q);
                            const float nn[4] = {n4.x, n4.y, n4.z, n4.w};
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const float sc = fmaf(-2.f, __uint_as_float(v[q * 4 + j]), nn[j]);
                                const float key = __uint_as_float((__float_as_uint(sc) & key_mask) | (uint32_t)(c + q * 4 + j));
                                if (j & 1)
                                    keep_two(b1, b2, key);
                                else
                                    keep_two(a1, a2, key);
                            }
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sh->t_empty[buf]);
                    const float k1 = fminf(a1, b1);
                    const float k2 = fminf(fmaxf(a1, b1), fminf(a2, b2));
                    int label = -1;
                    if (row < N) {
                        const float2 nr = __ldg(rownorm + row);
                        const float thr = k1 + 2.f * screen_allowance(nr.x, nr.y, cmax, cmax2, clomax, d);
                        const int i1 = (int)(__float_as_uint(k1) & IDX_MASK);
                        if (k2 > thr && i1 < K) {
                            label = i1;
                            assign[row] = i1;
                        } else {
                            sh->queue[par][atomicAdd(&sh->qn[par], 1)] = r;   // includes rows whose keys are NaN
                        }
                        ++n_rows;
                    }
                    sh->lab[par][r] = label;
                }
                if (ctid == 0) sh->stop[par] = *abort_flag;
            }
            consumer_sync();
            if (sh->stop[par]) break;   // one thread's reading, so all eight warps leave together
            // ---- queued rows: exact fp32 scores against all K centroids, a warp per row
            const int qn = sh->qn[par];
            for (int qi = cw; qi < qn; qi += CONS_WARPS) {
                const int r = sh->queue[par][qi];
                const float4 x = lane < d4 ? tile_chunk(xs, r, lane) : make_float4(0.f, 0.f, 0.f, 0.f);
                float best = CUDART_INF_F;
                int bidx = 0x7fffffff;
                for (int kb = 0; kb < K; kb += KC) {
                    float a[KC];
#pragma unroll
                    for (int kk = 0; kk < KC; ++kk) {
                        a[kk] = 0.f;
                        if (kb + kk < K && lane < d4) a[kk] = dot4(x, __ldg(C4 + (size_t)(kb + kk) * d4 + lane), 0.f);
                    }
                    const float dot = reduce8_transposed(a, lane);
                    const int k = kb + slot;
                    float sc = k < K ? fmaf(-2.f, dot, cn[k]) : CUDART_INF_F;
                    sc = (sc == sc) ? sc : CUDART_INF_F;
                    if (sc < best || (sc == best && k < bidx)) {
                        best = sc;
                        bidx = k;
                    }
                }
#pragma unroll
                for (int o = 16; o >= 1; o >>= 1) {
                    const float ov = __shfl_xor_sync(FULL, best, o);
                    const int oi = __shfl_xor_sync(FULL, bidx, o);
                    if (ov < best || (ov == best && oi < bidx)) {
                        best = ov;
                        bidx = oi;
                    }
                }
                if (bidx < 0 || bidx >= K) bidx = 0;   // a row of NaNs still gets a valid label
                if (lane == 0) {
                    sh->lab[par][r] = bidx;
                    assign[row0 + r] = bidx;
                }
                ++n_queued;
            }
            consumer_sync();
            if (ctid == 0) sh->qn[par] = 0;
            // ---- accumulate: warp cw owns clusters cw, cw + 8, ...; lane owns 16-byte chunk `lane`
            int l[BM / 32];
#pragma unroll
            for (int j = 0; j < BM / 32; ++j) l[j] = sh->lab[par][j * 32 + lane];
#pragma unroll
            for (int i = 0; i < KPW; ++i) {
                const int k = cw + CONS_WARPS * i;
                if (k < K) {
#pragma unroll
                    for (int j = 0; j < BM / 32; ++j) {
                        unsigned m = __ballot_sync(FULL, l[j] == k);
                        cnt[i] += __popc(m);
                        while (m) {
                            const int r = j * 32 + __ffs(m) - 1;
                            m &= m - 1;
                            if (lane < d4) {
                                const float4 x = tile_chunk(xs, r, lane);
                                acc[i].x += x.x;
                                acc[i].y += x.y;
                                acc[i].z += x.z;
                                acc[i].w += x.w;
                            }
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh->x_empty[s]);
        }
        // ---- publish this block's partial sums and counts
        float4 *out = reinterpret_cast<float4 *>(psum) + (size_t)blockIdx.x * K * d4;
#pragma unroll
        for (int i = 0; i < KPW; ++i) {
            const int k = cw + CONS_WARPS * i;
            if (k < K) {
                if (lane < d4) out[(size_t)k * d4 + lane] = acc[i];
                if (lane == 0) pcnt[(size_t)blockIdx.x * K + k] = cnt[i];
            }
        }
        if (counters && lane == 0) {
            atomicAdd(&counters[0], n_rows);
            atomicAdd(&counters[3], n_queued);
        }
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
    if (d < KBLK || d > MAX_KB * KBLK || K < 1 || K > 128) return false;
    const int num_kb = (d + KBLK - 1) / KBLK;
    return tcf_fixed_smem(d, K) + 2 * (size_t)num_kb * X_KB_BYTES <= (size_t)ctx->smem_optin;
}

int kmeans_tcf_grid(const ep_ctx *ctx, int64_t N) {
    return (int)std::max<int64_t>(1, std::min<int64_t>(ctx->sm_count, ceil_div(N, BM)));
}

int kmeans_tcf_prepare(ep_ctx *ctx, const float *emb, int64_t N, int d, int K, const float *ct, float2 *rownorm,
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
    if (!tc_encode_kblock_map(&st->map_x, emb, N, d, BM) || !tc_encode_kblock_map(&st->map_c, ct, K, d, st->npad))
        return fail(ctx, EP_ERR_CUDA, "cuTensorMapEncodeTiled failed for N=%lld d=%d K=%d", (long long)N, d, K);
    Timed tm(ctx, stream, EP_TIMER_KMEANS_UPDATE);
    row_norms<<<(int)std::min<int64_t>((int64_t)ctx->sm_count * 16, ceil_div(N, 8)), 256, 0, stream>>>(emb, N, d, rownorm);
    tm.end(1);
    EP_CUDA(ctx, cudaGetLastError());
    return EP_OK;
}

template <int KPW>
static int tcf_launch(ep_ctx *ctx, const TcFusedState &st, const float *centroids, const float *cn, const float *clo,
                      const float2 *rownorm, int64_t N, int d, int K, int32_t *assign, float *psum, int *pcnt,
                      cudaStream_t stream) {
    auto kern = kmeans_tc_fused<KPW>;
    EP_CUDA(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)st.smem));
    unsigned long long *counters =
        ctx->opt_profile ? reinterpret_cast<unsigned long long *>(ctx->d_status + EP_COUNTER_WORD0) : nullptr;
    Timed tm(ctx, stream, EP_TIMER_KMEANS_ASSIGN);
    kern<<<st.grid, THREADS, st.smem, stream>>>(st.map_x, st.map_c, centroids, cn, clo, rownorm, N, d, K, st.npad, st.num_kb,
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
    if (K <= 32) return tcf_launch<4>(ctx, st, centroids, cn, clo, rownorm, N, d, K, assign, psum, pcnt, stream);
    if (K <= 64) return tcf_launch<8>(ctx, st, centroids, cn, clo, rownorm, N, d, K, assign, psum, pcnt, stream);
    return tcf_launch<16>(ctx, st, centroids, cn, clo, rownorm, N, d, K, assign, psum, pcnt, stream);
}

}  // namespace ep
