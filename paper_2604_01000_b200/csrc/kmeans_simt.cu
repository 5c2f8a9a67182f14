// Lloyd K-Means on CUDA cores (Algorithm 3, the clustering step): the assign-and-accumulate pass, the centroid
// update and the per-call driver.  A warp owns whole rows; lane l holds the 16-byte slices
// l, l+32, ... of a row in registers, so a row is read from HBM exactly once, coalesced.
#include "ep_common.cuh"
#include "kmeans_device.cuh"

#include <math_constants.h>

#include <algorithm>
#include <type_traits>

namespace {

using namespace epk;

constexpr int UPD_THREADS = 128;

template <int VPL, int R>
struct Rows {
    float4 x[R][VPL];
};

template <int VPL, int R>
__device__ __forceinline__ void load_rows(Rows<VPL, R> &r, const float *emb, int64_t row, int64_t row_end, int d4,
                                          int lane) {
#pragma unroll
    for (int i = 0; i < R; ++i) {
#pragma unroll
        for (int v = 0; v < VPL; ++v) {
            int q = lane + 32 * v;
            if (row + i < row_end && q < d4)
                r.x[i][v] = ldg_stream(reinterpret_cast<const float4 *>(emb) + (row + i) * (int64_t)d4 + q);
            else
                r.x[i][v] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
    }
}

// Scores R rows against the kcount (multiple of KC) centroids staged at cs (row pitch DP4 float4,
// zero padded) with |c|^2 at cn (+inf for padding), and folds them into the per-lane running best.
// Score of (row, k) = |c_k|^2 - 2 x.c_k; the row's |x|^2 does not change the argmin.
// second[i] follows the smallest score this lane has seen for row i other than best[i] (a later tie counts).
template <int VPL, int R>
__device__ __forceinline__ void score_chunk(const Rows<VPL, R> &rows, const float4 *cs, const float *cn, int kbase,
                                            int kcount, int lane, float (&best)[R], int (&bidx)[R], float (&second)[R]) {
    constexpr int DP4 = VPL * 32;
    const int slot = lane_chunk_slot(lane);
    for (int kb = 0; kb < kcount; kb += KC) {
        float acc[R][KC];
#pragma unroll
        for (int i = 0; i < R; ++i)
#pragma unroll
            for (int kk = 0; kk < KC; ++kk) acc[i][kk] = 0.f;
#pragma unroll
        for (int kk = 0; kk < KC; ++kk) {
#pragma unroll
            for (int v = 0; v < VPL; ++v) {
                float4 c = cs[(kb + kk) * DP4 + lane + 32 * v];
#pragma unroll
                for (int i = 0; i < R; ++i) acc[i][kk] = dot4(rows.x[i][v], c, acc[i][kk]);
            }
        }
        float cnk = cn[kb + slot];
#pragma unroll
        for (int i = 0; i < R; ++i) {
            float dot = reduce8_transposed(acc[i], lane);
            float s = fmaf(-2.f, dot, cnk);
            s = (s == s) ? s : CUDART_INF_F;          // a NaN score never wins
            if (s < best[i]) {                         // strict: the earlier (lower) index keeps a tie
                second[i] = best[i];
                best[i] = s;
                bidx[i] = kbase + kb + slot;
            } else {
                second[i] = fminf(second[i], s);
            }
        }
    }
}

// Warp-wide argmin of (best, bidx) with the lowest index winning ties; every lane gets the result.
// The eight lane groups that differ in lane bits 4, 3, 2 hold eight different centroid slots.
__device__ __forceinline__ int warp_argmin(float &best, int bidx) {
#pragma unroll
    for (int m = 16; m >= 4; m >>= 1) {
        float ov = __shfl_xor_sync(FULL, best, m);
        int oi = __shfl_xor_sync(FULL, bidx, m);
        if (ov < best || (ov == best && oi < bidx)) {
            best = ov;
            bidx = oi;
        }
    }
    return bidx;
}

// Smallest score of the row apart from the winner's: a lane's own best when the winner lives in another
// slot, its runner-up otherwise.
__device__ __forceinline__ float warp_runner_up(float lane_best, int lane_bidx, float lane_second, int winner) {
    float v = lane_bidx == winner ? lane_second : lane_best;
#pragma unroll
    for (int m = 16; m >= 4; m >>= 1) v = fminf(v, __shfl_xor_sync(FULL, v, m));
    return v;
}

// How far two scores |c|^2 - 2 x.c may lie apart in fp32 and still be in the wrong order: twice the rounding
// error of one score.  The dot product is 4 VPL sequential fused multiply-adds per lane and five pairwise
// additions across the warp, each exact to 2^-24 of the running magnitude (at most |x||c|); |c|^2 and the
// final fused multiply-add add one rounding each.
template <int VPL>
__device__ __forceinline__ float score_resolution(float xnorm, float cmax, float cmax2) {
    constexpr float U = 5.9604645e-8f;                       // 2^-24
    return 2.2f * U * ((float)(2 * (4 * VPL + 5) + 3) * xnorm * cmax + 2.f * cmax2);
}

// The row's label by squared distance in the direct form sum_j (x_j - c_j)^2 over all K centroids, lowest
// index on ties.  For rows whose two best scores are closer than score_resolution: the direct form is
// accurate relative to the distance itself, so it separates what the expansion cannot.
template <int VPL>
__device__ __noinline__ int argmin_direct(const float4 (&x)[VPL], const float *__restrict__ C, int K, int d4, int lane) {
    const float4 *C4 = reinterpret_cast<const float4 *>(C);
    const int slot = lane_chunk_slot(lane);
    float best = CUDART_INF_F;
    int bidx = 0x7fffffff;
    for (int kb = 0; kb < K; kb += KC) {
        float acc[KC];
#pragma unroll
        for (int kk = 0; kk < KC; ++kk) {
            acc[kk] = 0.f;
            if (kb + kk < K) {
#pragma unroll
                for (int v = 0; v < VPL; ++v) {
                    const int q = lane + 32 * v;
                    if (q < d4) acc[kk] = dist4(x[v], __ldg(C4 + (size_t)(kb + kk) * d4 + q), acc[kk]);
                }
            }
        }
        float s = reduce8_transposed(acc, lane);
        const int k = kb + slot;
        s = (k < K && s == s) ? s : CUDART_INF_F;
        if (s < best) {
            best = s;
            bidx = k;
        }
    }
    bidx = warp_argmin(best, bidx);
    return (bidx >= 0 && bidx < K) ? bidx : 0;
}

// max_k cnorm[k] over the K real centroids, for every thread of the block (red: 32 floats of shared memory).
__device__ __forceinline__ float block_max_norm2(const float *__restrict__ cnorm, int K, float *red) {
    float m = 0.f;
    for (int k = threadIdx.x; k < K; k += blockDim.x) m = fmaxf(m, cnorm[k]);
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) m = fmaxf(m, __shfl_xor_sync(FULL, m, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
    __syncthreads();
    m = 0.f;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) m = fmaxf(m, red[w]);
    __syncthreads();
    return m;
}

// |x_i|_2 of the R rows a warp holds (every lane gets them).
template <int VPL, int R>
__device__ __forceinline__ void row_norms_of(const Rows<VPL, R> &rows, float (&xn)[R]) {
#pragma unroll
    for (int i = 0; i < R; ++i) {
        float t = 0.f;
#pragma unroll
        for (int v = 0; v < VPL; ++v) t = dot4(rows.x[i][v], rows.x[i][v], t);
        xn[i] = sqrtf(warp_sum(t));
    }
}

// Copies centroids [k0, k0+kcount) into shared memory with row pitch DP4 float4, zero-filling the
// padding columns and the rows at or beyond K, and their squared norms (+inf beyond K).
__device__ __forceinline__ void stage_centroids(float4 *cs, float *cn, const float *C, const float *cnorm, int k0,
                                                int kcount, int K, int d4, int DP4) {
    for (int i = threadIdx.x; i < kcount * DP4; i += blockDim.x) {
        int k = i / DP4, q = i - k * DP4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (k0 + k < K && q < d4) v = __ldg(reinterpret_cast<const float4 *>(C) + (int64_t)(k0 + k) * d4 + q);
        cs[i] = v;
    }
    for (int k = threadIdx.x; k < kcount; k += blockDim.x) cn[k] = (k0 + k < K) ? cnorm[k0 + k] : CUDART_INF_F;
}

// Fused pass for small K: centroids and one private sum table per warp live in shared memory.
// Each warp walks a contiguous run of rows, so the order of every addition is fixed by the launch
// shape alone.  Block b leaves its partial sums in psum[b] and its label counts in pcnt[b].
template <int VPL, int R>
__global__ void __launch_bounds__(256) kmeans_assign_fused(const float *__restrict__ emb, int64_t N, int d, int K,
                                                           int Kpad, const float *__restrict__ C,
                                                           const float *__restrict__ cnorm,
                                                           int32_t *__restrict__ assign, float *__restrict__ psum,
                                                           int *__restrict__ pcnt, int64_t rows_per_block,
                                                           int64_t rows_per_warp) {
    constexpr int DP4 = VPL * 32;
    extern __shared__ float4 smem4[];
    const int W = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int d4 = d >> 2;
    float4 *cs = smem4;                                   // [Kpad][DP4]
    float4 *sw = cs + (size_t)Kpad * DP4;                 // [W][K][DP4]
    float *cn = reinterpret_cast<float *>(sw + (size_t)W * K * DP4);   // [Kpad]
    int *cw = reinterpret_cast<int *>(cn + Kpad);         // [W][K]

    __shared__ float red[32];
    const float cmax2 = block_max_norm2(cnorm, K, red);
    const float cmax = sqrtf(cmax2);
    stage_centroids(cs, cn, C, cnorm, 0, Kpad, K, d4, DP4);
    for (int i = threadIdx.x; i < W * K * DP4; i += blockDim.x) sw[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int i = threadIdx.x; i < W * K; i += blockDim.x) cw[i] = 0;
    __syncthreads();

    const int64_t blk0 = (int64_t)blockIdx.x * rows_per_block;
    const int64_t blk1 = min(N, blk0 + rows_per_block);
    const int64_t w0 = min(blk1, blk0 + (int64_t)warp * rows_per_warp);
    const int64_t w1 = min(blk1, w0 + rows_per_warp);
    float4 *mysum = sw + (size_t)warp * K * DP4;
    int *mycnt = cw + warp * K;

    Rows<VPL, R> cur, nxt;
    load_rows(cur, emb, w0, w1, d4, lane);
    for (int64_t row = w0; row < w1; row += R) {
        load_rows(nxt, emb, row + R, w1, d4, lane);
        float best[R], second[R], xn[R];
        int bidx[R];
#pragma unroll
        for (int i = 0; i < R; ++i) {
            best[i] = second[i] = CUDART_INF_F;
            bidx[i] = 0;
        }
        score_chunk<VPL, R>(cur, cs, cn, 0, Kpad, lane, best, bidx, second);
        row_norms_of<VPL, R>(cur, xn);
#pragma unroll
        for (int i = 0; i < R; ++i) {
            if (row + i < w1) {
                float wbest = best[i];
                int a = warp_argmin(wbest, bidx[i]);
                const float runner = warp_runner_up(best[i], bidx[i], second[i], a);
                // too close to call from the scores: decide by the distances themselves
                if (__any_sync(FULL, runner - wbest <= score_resolution<VPL>(xn[i], cmax, cmax2)))
                    a = argmin_direct<VPL>(cur.x[i], C, K, d4, lane);
#pragma unroll
                for (int v = 0; v < VPL; ++v) {
                    float4 s = mysum[a * DP4 + lane + 32 * v];
                    s.x += cur.x[i][v].x;
                    s.y += cur.x[i][v].y;
                    s.z += cur.x[i][v].z;
                    s.w += cur.x[i][v].w;
                    mysum[a * DP4 + lane + 32 * v] = s;
                }
                if (lane == 0) {
                    mycnt[a] += 1;
                    assign[row + i] = a;
                }
            }
        }
        cur = nxt;
    }
    __syncthreads();
    // fold the warps' tables in warp order and publish this block's partials
    float4 *out = reinterpret_cast<float4 *>(psum) + (size_t)blockIdx.x * K * d4;
    for (int i = threadIdx.x; i < K * d4; i += blockDim.x) {
        int k = i / d4, q = i - k * d4;
        float4 s = sw[k * DP4 + q];
        for (int w = 1; w < W; ++w) {
            float4 t = sw[((size_t)w * K + k) * DP4 + q];
            s.x += t.x;
            s.y += t.y;
            s.z += t.z;
            s.w += t.w;
        }
        out[i] = s;
    }
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
        int c = 0;
        for (int w = 0; w < W; ++w) c += cw[w * K + k];
        pcnt[(size_t)blockIdx.x * K + k] = c;
    }
}

// Label-only pass for K too large for the fused kernel: a block keeps W*R rows in registers and
// streams the centroid table through shared memory in chunks.
template <int VPL, int R>
__global__ void __launch_bounds__(256) kmeans_assign_chunked(const float *__restrict__ emb, int64_t N, int d, int K,
                                                             int Kpad, int kchunk, const float *__restrict__ C,
                                                             const float *__restrict__ cnorm,
                                                             int32_t *__restrict__ assign) {
    constexpr int DP4 = VPL * 32;
    extern __shared__ float4 smem4[];
    const int W = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int d4 = d >> 2;
    float4 *cs = smem4;                                            // [kchunk][DP4]
    float *cn = reinterpret_cast<float *>(cs + (size_t)kchunk * DP4);   // [kchunk]
    __shared__ float red[32];
    const float cmax2 = block_max_norm2(cnorm, K, red);
    const float cmax = sqrtf(cmax2);
    const int64_t batch = (int64_t)W * R;
    for (int64_t b0 = (int64_t)blockIdx.x * batch; b0 < N; b0 += (int64_t)gridDim.x * batch) {
        const int64_t row = b0 + (int64_t)warp * R;
        Rows<VPL, R> cur;
        load_rows(cur, emb, row, N, d4, lane);
        float best[R], second[R], xn[R];
        int bidx[R];
#pragma unroll
        for (int i = 0; i < R; ++i) {
            best[i] = second[i] = CUDART_INF_F;
            bidx[i] = 0;
        }
        for (int k0 = 0; k0 < Kpad; k0 += kchunk) {
            const int kc = min(kchunk, Kpad - k0);
            __syncthreads();
            stage_centroids(cs, cn, C, cnorm, k0, kc, K, d4, DP4);
            __syncthreads();
            score_chunk<VPL, R>(cur, cs, cn, k0, kc, lane, best, bidx, second);
        }
        row_norms_of<VPL, R>(cur, xn);
#pragma unroll
        for (int i = 0; i < R; ++i) {
            float wbest = best[i];
            int a = warp_argmin(wbest, bidx[i]);
            const float runner = warp_runner_up(best[i], bidx[i], second[i], a);
            // too close to call from the scores: decide by the distances themselves
            if (row + i < N && __any_sync(FULL, runner - wbest <= score_resolution<VPL>(xn[i], cmax, cmax2)))
                a = argmin_direct<VPL>(cur.x[i], C, K, d4, lane);
            if (lane == 0 && row + i < N) assign[row + i] = a;
        }
    }
}

// Sums the rows of each cluster for the label-only path.  order lists the row ids grouped by label
// (ascending ids inside a group), off[k] is the first position of cluster k.  Block (k, s) adds up
// slice s of cluster k in a fixed order and leaves the result in psum[s][k], the count in pcnt[s][k].
template <int VPL>
__global__ void __launch_bounds__(256) kmeans_segment_sums(const float *__restrict__ emb, int d, int K,
                                                           const int32_t *__restrict__ order,
                                                           const int64_t *__restrict__ off,
                                                           float *__restrict__ psum, int *__restrict__ pcnt) {
    __shared__ float4 red[8][VPL * 32];
    const int k = blockIdx.x, s = blockIdx.y, S = gridDim.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, d4 = d >> 2;
    const int64_t n = off[k + 1] - off[k];
    const int64_t p0 = off[k] + n * s / S, p1 = off[k] + n * (s + 1) / S;
    float4 acc[VPL];
#pragma unroll
    for (int v = 0; v < VPL; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    // several rows of this warp in flight at a time; they are added in the order of the list all the same
    constexpr int AHEAD = VPL <= 2 ? 4 : VPL == 4 ? 2 : 1;
    for (int64_t p = p0 + warp; p < p1; p += 8 * AHEAD) {
        int64_t row[AHEAD];
#pragma unroll
        for (int u = 0; u < AHEAD; ++u) row[u] = p + 8 * u < p1 ? (int64_t)order[p + 8 * u] : -1;
        float4 x[AHEAD][VPL];
#pragma unroll
        for (int u = 0; u < AHEAD; ++u)
#pragma unroll
            for (int v = 0; v < VPL; ++v) {
                const int q = lane + 32 * v;
                x[u][v] = (row[u] >= 0 && q < d4) ? ldg_stream(reinterpret_cast<const float4 *>(emb) + row[u] * d4 + q)
                                                  : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
        for (int u = 0; u < AHEAD; ++u)
            if (row[u] >= 0) {
#pragma unroll
                for (int v = 0; v < VPL; ++v) {
                    acc[v].x += x[u][v].x;
                    acc[v].y += x[u][v].y;
                    acc[v].z += x[u][v].z;
                    acc[v].w += x[u][v].w;
                }
            }
    }
#pragma unroll
    for (int v = 0; v < VPL; ++v) red[warp][lane + 32 * v] = acc[v];
    __syncthreads();
    float4 *out = reinterpret_cast<float4 *>(psum) + ((size_t)s * K + k) * d4;
    for (int q = threadIdx.x; q < d4; q += blockDim.x) {
        float4 t = red[0][q];
        for (int w = 1; w < 8; ++w) {
            t.x += red[w][q].x;
            t.y += red[w][q].y;
            t.z += red[w][q].z;
            t.w += red[w][q].w;
        }
        out[q] = t;
    }
    if (threadIdx.x == 0) pcnt[(size_t)s * K + k] = (int)(p1 - p0);
}

// hist[k] = number of rows labelled k (integer atomics: exact whatever the order).
// Up to LH_SMEM_K clusters are first counted in the block's shared memory.
constexpr int LH_SMEM_K = 8192;

__global__ void __launch_bounds__(256) label_histogram(const int32_t *__restrict__ assign, int64_t N, int K,
                                                       unsigned long long *hist) {
    __shared__ unsigned int local[LH_SMEM_K];
    const bool in_block = K <= LH_SMEM_K;
    if (in_block) {
        for (int k = threadIdx.x; k < K; k += blockDim.x) local[k] = 0u;
        __syncthreads();
    }
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < N; i += (int64_t)gridDim.x * blockDim.x) {
        const int a = assign[i];
        if (in_block)
            atomicAdd(&local[a], 1u);
        else
            atomicAdd(&hist[a], 1ull);
    }
    if (in_block) {
        __syncthreads();
        for (int k = threadIdx.x; k < K; k += blockDim.x)
            if (local[k]) atomicAdd(&hist[k], (unsigned long long)local[k]);
    }
}

// off[0..K] = exclusive prefix sum of hist (one block; K <= 65536).
__global__ void label_offsets(const unsigned long long *__restrict__ hist, int K, int64_t *off) {
    __shared__ long long part[256];
    const int per = (K + 255) / 256;
    const int k0 = min(K, (int)threadIdx.x * per), k1 = min(K, k0 + per);
    long long s = 0;
    for (int k = k0; k < k1; ++k) s += (long long)hist[k];
    part[threadIdx.x] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        long long run = 0;
        for (int t = 0; t < 256; ++t) {
            long long v = part[t];
            part[t] = run;
            run += v;
        }
    }
    __syncthreads();
    long long run = part[threadIdx.x];
    for (int k = k0; k < k1; ++k) {
        off[k] = run;
        run += (long long)hist[k];
    }
    if (k1 == K && k0 <= K) off[K] = run;
}

template <int T>
__device__ __forceinline__ double block_sum_fixed(double v, double *buf) {
    buf[threadIdx.x] = v;
    __syncthreads();
#pragma unroll
    for (int s = T / 2; s > 0; s >>= 1) {
        if ((int)threadIdx.x < s) buf[threadIdx.x] += buf[threadIdx.x + s];
        __syncthreads();
    }
    double r = buf[0];
    __syncthreads();
    return r;
}

// Nearest TF32 value (10 explicit mantissa bits) of an fp32 number, kept in an fp32 container.
__device__ __forceinline__ float round_to_tf32(float x) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return __uint_as_float(r);
}

// What the tensor cores see of a centroid coordinate, and what they miss.  With a TF32 copy (ct given) the
// copy holds the nearest TF32 value; without one the tensor core itself drops the low 13 mantissa bits.
__device__ __forceinline__ float tf32_image(float c, bool rounded) {
    return rounded ? round_to_tf32(c) : __uint_as_float(__float_as_uint(c) & 0xFFFFE000u);
}

// |c_k|^2 of the initial centroids (fp64 sum, rounded once).  Tensor-core paths also get clo[k], an upper
// bound of |c_k - image(c_k)|_2, and, when ct is given, the TF32-rounded copy itself.
__global__ void __launch_bounds__(UPD_THREADS) centroid_norms(const float *__restrict__ C, int d, float *cnorm,
                                                              float *__restrict__ ct, float *__restrict__ clo) {
    __shared__ double buf[UPD_THREADS];
    const int k = blockIdx.x;
    double t = 0.0, tl = 0.0;
    for (int j = threadIdx.x; j < d; j += UPD_THREADS) {
        const float cf = C[(size_t)k * d + j];
        const double c = cf;
        t += c * c;
        if (clo) {
            const float r = tf32_image(cf, ct != nullptr);
            if (ct) ct[(size_t)k * d + j] = r;
            const double lo = (double)cf - (double)r;
            tl += lo * lo;
        }
    }
    t = block_sum_fixed<UPD_THREADS>(t, buf);
    if (clo) tl = block_sum_fixed<UPD_THREADS>(tl, buf);
    if (threadIdx.x == 0) {
        cnorm[k] = (float)t;
        if (clo) clo[k] = (float)(sqrt(tl) * 1.000001);
    }
}

// Centroid update, one block per cluster: S_k = sum over the partial slabs (fp64, slab order),
// c_k <- S_k / n_k when n_k > 0, else unchanged; also |c_k|^2 of the new centroid and this
// cluster's share of the objective, n_k |c|^2 - 2 c.S_k with c the centroid the rows were assigned
// against (the rows' own sum of |x|^2 is added once by objective_finalize).
__global__ void __launch_bounds__(UPD_THREADS) centroid_update_few(const float *__restrict__ psum,
                                                               const int *__restrict__ pcnt, int parts, int K, int d,
                                                               float *C, float *cnorm, double *objterm,
                                                               int keep_centroids, float *__restrict__ ct,
                                                               float *__restrict__ clo) {
    __shared__ double buf[UPD_THREADS];
    const int k = blockIdx.x;
    long long n = 0;
    for (int p = 0; p < parts; ++p) n += pcnt[(size_t)p * K + k];
    double t_cs = 0.0, t_cc = 0.0, t_nn = 0.0, t_lo = 0.0;
    for (int j = threadIdx.x; j < d; j += UPD_THREADS) {
        double S = 0.0;
        for (int p = 0; p < parts; ++p) S += (double)psum[((size_t)p * K + k) * d + j];
        const float cold = C[(size_t)k * d + j];
        float cnew = cold;
        if (n > 0 && !keep_centroids) cnew = (float)(S / (double)n);
        t_cs += (double)cold * S;
        t_cc += (double)cold * (double)cold;
        t_nn += (double)cnew * (double)cnew;
        C[(size_t)k * d + j] = cnew;
        if (clo) {   // tensor-core paths: what the next screening pass will not see of this centroid
            const float r = tf32_image(cnew, ct != nullptr);
            if (ct) ct[(size_t)k * d + j] = r;
            const double lo = (double)cnew - (double)r;
            t_lo += lo * lo;
        }
    }
    if (clo) t_lo = block_sum_fixed<UPD_THREADS>(t_lo, buf);
    t_cs = block_sum_fixed<UPD_THREADS>(t_cs, buf);
    t_cc = block_sum_fixed<UPD_THREADS>(t_cc, buf);
    t_nn = block_sum_fixed<UPD_THREADS>(t_nn, buf);
    if (threadIdx.x == 0) {
        cnorm[k] = (float)t_nn;
        objterm[k] = (double)n * t_cc - 2.0 * t_cs;
        if (clo) clo[k] = (float)(sqrt(t_lo) * 1.000001);
    }
}

// The same update for many slabs (the fused kernels leave one or two per SM), one block of 1024 per cluster.  S_k = sum over the partial slabs in fp64: with
// G = UPD2_THREADS / dpad thread groups, group g adds its contiguous share of the slabs in slab order and the
// group sums are then added in group order (a fixed tree: results repeat).  c_k <- S_k / n_k when n_k > 0,
// else unchanged; also |c_k|^2 of the new centroid and this cluster's share of the objective,
// n_k |c|^2 - 2 c.S_k with c the centroid the rows were assigned against (the rows' own sum of |x|^2 is
// added once by objective_finalize).
constexpr int UPD2_THREADS = 1024;

__global__ void __launch_bounds__(UPD2_THREADS) centroid_update_many(const float *__restrict__ psum,
                                                                const int *__restrict__ pcnt, int parts, int K, int d,
                                                                float *C, float *cnorm, double *objterm,
                                                                int keep_centroids, float *__restrict__ ct,
                                                                float *__restrict__ clo) {
    __shared__ double buf[UPD2_THREADS];
    __shared__ long long n_s;
    const int k = blockIdx.x;
    const int dpad = (d + 31) / 32 * 32;
    const int G = max(1, UPD2_THREADS / dpad);            // dpad <= 1024
    const int g = threadIdx.x / dpad, j = threadIdx.x - g * dpad;
    const bool mine = g < G && j < d;
    {   // n_k: integer, any order
        long long n = 0;
        for (int p = threadIdx.x; p < parts; p += UPD2_THREADS) n += pcnt[(size_t)p * K + k];
        buf[threadIdx.x] = (double)n;                     // counts are far below 2^53: exact
        __syncthreads();
        for (int s2 = UPD2_THREADS / 2; s2 > 0; s2 >>= 1) {
            if ((int)threadIdx.x < s2) buf[threadIdx.x] += buf[threadIdx.x + s2];
            __syncthreads();
        }
        if (threadIdx.x == 0) n_s = (long long)buf[0];
        __syncthreads();
    }
    const long long n = n_s;
    double part = 0.0;
    if (mine) {
        const int p0 = (int)((long long)parts * g / G), p1 = (int)((long long)parts * (g + 1) / G);
        for (int p = p0; p < p1; ++p) part += (double)psum[((size_t)p * K + k) * d + j];
    }
    buf[threadIdx.x] = part;
    __syncthreads();
    double t_cs = 0.0, t_cc = 0.0, t_nn = 0.0, t_lo = 0.0;
    if (g == 0 && j < d) {
        double S = buf[j];
        for (int gg = 1; gg < G; ++gg) S += buf[gg * dpad + j];
        const float cold = C[(size_t)k * d + j];
        float cnew = cold;
        if (n > 0 && !keep_centroids) cnew = (float)(S / (double)n);
        t_cs = (double)cold * S;
        t_cc = (double)cold * (double)cold;
        t_nn = (double)cnew * (double)cnew;
        C[(size_t)k * d + j] = cnew;
        if (clo) {   // tensor-core paths: what the next screening pass will not see of this centroid
            const float r = tf32_image(cnew, ct != nullptr);
            if (ct) ct[(size_t)k * d + j] = r;
            const double lo = (double)cnew - (double)r;
            t_lo = lo * lo;
        }
    }
    __syncthreads();
    if (clo) t_lo = block_sum_fixed<UPD2_THREADS>(t_lo, buf);
    t_cs = block_sum_fixed<UPD2_THREADS>(t_cs, buf);
    t_cc = block_sum_fixed<UPD2_THREADS>(t_cc, buf);
    t_nn = block_sum_fixed<UPD2_THREADS>(t_nn, buf);
    if (threadIdx.x == 0) {
        cnorm[k] = (float)t_nn;
        objterm[k] = (double)n * t_cc - 2.0 * t_cs;
        if (clo) clo[k] = (float)(sqrt(t_lo) * 1.000001);
    }
}

// x2part[b] = sum of squares of block b's share of the embedding matrix (fp64).
__global__ void __launch_bounds__(256) sum_of_squares(const float *__restrict__ emb, int64_t n4, double *x2part) {
    __shared__ double buf[256];
    const int64_t per = (n4 + gridDim.x - 1) / gridDim.x;
    const int64_t i0 = blockIdx.x * per, i1 = min(n4, i0 + per);
    double t = 0.0;
    for (int64_t i = i0 + threadIdx.x; i < i1; i += 256) {
        float4 x = ldg_stream(reinterpret_cast<const float4 *>(emb) + i);
        t += (double)x.x * x.x + (double)x.y * x.y + (double)x.z * x.z + (double)x.w * x.w;
    }
    t = block_sum_fixed<256>(t, buf);
    if (threadIdx.x == 0) x2part[blockIdx.x] = t;
}

// objective[t] = sum_i |x_i|^2 + sum_k objterm[k], both summed in index order.
__global__ void __launch_bounds__(256) objective_finalize(const double *__restrict__ x2part, int nparts,
                                                          const double *__restrict__ objterm, int K, double *out) {
    __shared__ double buf[256];
    double t = 0.0;
    for (int i = threadIdx.x; i < nparts; i += 256) t += x2part[i];
    for (int k = threadIdx.x; k < K; k += 256) t += objterm[k];
    t = block_sum_fixed<256>(t, buf);
    if (threadIdx.x == 0) *out = t;
}

constexpr int X2_BLOCKS = 1184;
constexpr int FUSED_TC_MIN_K = 2;     // auto: the fused tensor-core kernel from here on, when the shape allows it
constexpr int LARGE_TC_MIN_K = 65;    // auto: screening + resolve from here on (below, d > 128 stays on the CUDA cores)
constexpr int CN_PAD = 256;           // |c|^2 is padded to the tensor path's centroid tile

template <typename F>
int dispatch_vpl(int d, F &&f) {
    if (d <= 128) return f(std::integral_constant<int, 1>{});
    if (d <= 256) return f(std::integral_constant<int, 2>{});
    if (d <= 512) return f(std::integral_constant<int, 4>{});
    return f(std::integral_constant<int, 8>{});
}

}  // namespace

namespace ep {

struct KMeansBuffers {
    float *cnorm;
    float *psum;
    int *pcnt;
    double *objterm;
    double *x2part;
    unsigned long long *hist;
    int64_t *off;
    int32_t *order;
    void *sort_ws;
    void *cand;        // tensor path: screening keys of one row chunk
    float *ct;         // tensor path: centroids rounded to TF32
    float *clo;        // tensor path: |c_k - ct_k|
    float2 *rownorm;   // tensor paths: (|x_i|, |x_i - trunc(x_i)|)
    float *cmaxima;    // large-K tensor path: max |c|^2 and max rounding residual of this iteration
    void *late_list;   // fused tensor path: per screen warp, the rows the screening left undecided (16 bytes each)
    unsigned *grid_bar;   // fused tensor path: the word its blocks meet on
};

static inline int vpl_of(int d) { return d <= 128 ? 1 : d <= 256 ? 2 : d <= 512 ? 4 : 8; }
static inline int rows_per_step(int vpl) { return vpl == 1 ? 4 : vpl == 2 ? 2 : 1; }

bool kmeans_make_plan(const ep_ctx *ctx, int64_t N, int d, int K, KMeansPlan *plan) {
    if (N < 1 || N >= (int64_t(1) << 31) || d < 4 || d > 1024 || (d & 3) || K < 1 || K > 65536 || K > N) return false;
    KMeansPlan p{};
    p.N = N;
    p.d = d;
    p.K = K;
    const int vpl = vpl_of(d);
    const size_t row_bytes = (size_t)vpl * 512;                   // padded centroid row in shared memory
    const int Kpad = (K + KC - 1) / KC * KC;
    const size_t budget = (size_t)ctx->smem_optin - 1024;
    // fused: Kpad centroid rows + W*K sum rows + norms + counts
    int W = 0;
    for (int w = 8; w >= 2; --w) {
        size_t need = Kpad * row_bytes + (size_t)w * K * row_bytes + Kpad * 4 + (size_t)w * K * 4;
        if (need <= budget) {
            W = w;
            break;
        }
    }
    const bool tc_ok = kmeans_tc_shape_ok(ctx, d, K), tcf_ok = kmeans_tcf_shape_ok(ctx, d, K);
    const bool forced = ctx->opt_kmeans_path == 2, autop = ctx->opt_kmeans_path == 0;
    p.tc_fused = tcf_ok && (forced || (autop && K >= FUSED_TC_MIN_K));
    p.tensor = p.tc_fused || (tc_ok && (forced || (autop && K >= LARGE_TC_MIN_K)));
    p.fused = !p.tensor && W >= 4 && K <= 256;
    if (p.tc_fused) {
        p.warps = 12;
        p.smem = 0;
        p.grid = kmeans_tcf_grid(ctx, N, d);
        p.parts = p.grid;
    } else if (p.fused) {
        p.warps = W;
        p.smem = Kpad * row_bytes + (size_t)W * K * row_bytes + Kpad * 4 + (size_t)W * K * 4;
        const int64_t step = (int64_t)W * rows_per_step(vpl);
        const int per_sm = (2 * (p.smem + 1024) <= (size_t)ctx->smem_optin) ? 2 : 1;   // registers allow two blocks
        p.grid = (int)std::max<int64_t>(1, std::min<int64_t>((int64_t)ctx->sm_count * per_sm, ceil_div(N, step)));
        p.parts = p.grid;
    } else {
        p.warps = 8;
        int kchunk = (int)std::min<size_t>(Kpad, (96 * 1024) / row_bytes / KC * KC);
        p.smem = (size_t)kchunk * row_bytes + (size_t)kchunk * 4;
        const int64_t batch = 8 * rows_per_step(vpl);
        p.grid = (int)std::max<int64_t>(1, std::min<int64_t>((int64_t)ctx->sm_count * 2, ceil_div(N, batch)));
        p.parts = (int)std::max<int64_t>(1, std::min<int64_t>(64, ceil_div(2048, K)));
    }
    *plan = p;
    return true;
}

size_t kmeans_workspace_layout(const ep_ctx *ctx, const KMeansPlan &p, void *workspace, KMeansBuffers *out) {
    (void)ctx;
    Arena a(workspace);
    KMeansBuffers b{};
    b.cnorm = a.take<float>((size_t)ceil_div(p.K, CN_PAD) * CN_PAD);
    b.psum = a.take<float>((size_t)p.parts * p.K * p.d);
    b.pcnt = a.take<int>((size_t)p.parts * p.K);
    b.objterm = a.take<double>(p.K);
    b.x2part = a.take<double>(X2_BLOCKS);
    if (!p.fused && !p.tc_fused) {
        b.hist = a.take<unsigned long long>(p.K);
        b.off = a.take<int64_t>(p.K + 1);
        b.order = a.take<int32_t>(p.N);
        b.sort_ws = a.take<char>(reorder_workspace_bytes(p.N, p.K));
    }
    if (p.tensor) {
        b.rownorm = a.take<float2>(p.N);
        if (p.tc_fused) {
            b.late_list = a.take<int4>((size_t)kmeans_tcf_late_cap(ctx, p.N, p.d) * 4 * p.grid);
            b.grid_bar = a.take<unsigned>(64 + 64 * 16 * 4 * 2);   // the barrier word, then 32 KB for the update's shares
        } else {
            b.cand = a.take<char>(kmeans_tc_cand_bytes(ctx, p.N, p.K));
            b.cmaxima = a.take<float>(2);
        }
        b.ct = a.take<float>((size_t)p.K * p.d);
        b.clo = a.take<float>(p.K);
    }
    if (out) *out = b;
    return a.used;
}

int kmeans_run(ep_ctx *ctx, const KMeansPlan &p, const float *emb, int iters, const float *init, int32_t *assign,
               float *centroids, double *objective, void *workspace, cudaStream_t stream) {
    KMeansBuffers b;
    kmeans_workspace_layout(ctx, p, workspace, &b);
    const int K = p.K, d = p.d;
    const int Kpad = (K + KC - 1) / KC * KC;
    const int64_t N = p.N;

    if (centroids != init)
        EP_CUDA(ctx, cudaMemcpyAsync(centroids, init, sizeof(float) * K * d, cudaMemcpyDeviceToDevice, stream));
    alignas(64) unsigned char tc_state_mem[512];
    TcState *tc_state = reinterpret_cast<TcState *>(tc_state_mem);
    TcFusedState *tcf_state = reinterpret_cast<TcFusedState *>(tc_state_mem);
    if (p.tensor) {
        if (std::max(kmeans_tc_state_bytes(), kmeans_tcf_state_bytes()) > sizeof(tc_state_mem))
            return fail(ctx, EP_ERR_CUDA, "tensor map state too large");
        int rc = p.tc_fused ? kmeans_tcf_prepare(ctx, emb, N, d, K, b.ct, tcf_state)
                            : kmeans_tc_prepare(ctx, emb, N, d, K, b.ct, tc_state);
        if (rc != EP_OK) return rc;
        rc = kmeans_row_norms(ctx, emb, N, d, b.rownorm, stream);
        if (rc != EP_OK) return rc;
        // the padding of |c|^2 must never win: every byte 0x7F makes each float 3.39e38
        EP_CUDA(ctx, cudaMemsetAsync(b.cnorm, 0x7F, sizeof(float) * (size_t)ceil_div(K, CN_PAD) * CN_PAD, stream));
    }
    {
        Timed tm(ctx, stream, EP_TIMER_KMEANS_UPDATE);
        centroid_norms<<<K, UPD_THREADS, 0, stream>>>(centroids, d, b.cnorm, b.ct, b.clo);
        if (objective) sum_of_squares<<<X2_BLOCKS, 256, 0, stream>>>(emb, N * (d / 4), b.x2part);
        tm.end(objective ? 2 : 1);
    }

    const int T = iters > 0 ? iters : 1;
    // Few centroids on the tensor cores: all iterations of the call, centroid updates included, run inside one launch
    // (no gaps, prologues or second kernels between iterations; measured faster at every size from 10 K to 111 M rows).
    // One launch per iteration plus the update kernel of the other paths remains as an option.
    const bool one_launch = p.tc_fused && ctx->opt_iters_per_launch != 1;
    if (one_launch) {
        int rc = kmeans_tcf_run(ctx, *tcf_state, emb, centroids, b.cnorm, b.ct, b.clo, b.rownorm, N, d, K, assign, b.psum, b.pcnt,
                                b.late_list, T, /*update_here=*/true, false, iters == 0, b.objterm, objective, b.x2part,
                                X2_BLOCKS, b.grid_bar, stream);
        if (rc != EP_OK) return rc;
        EP_CUDA(ctx, cudaGetLastError());
        return EP_OK;
    }
    for (int t = 0; t < T; ++t) {
        int rc = dispatch_vpl(d, [&](auto vpl_c) -> int {
            constexpr int VPL = decltype(vpl_c)::value;
            constexpr int R = VPL == 1 ? 4 : VPL == 2 ? 2 : 1;
            if (p.tc_fused) {
                return kmeans_tcf_run(ctx, *tcf_state, emb, centroids, b.cnorm, b.ct, b.clo, b.rownorm, N, d, K, assign, b.psum,
                                      b.pcnt, b.late_list, 1, /*update_here=*/false, /*use_prev0=*/t > 0, false, b.objterm, nullptr,
                                      b.x2part, X2_BLOCKS, b.grid_bar, stream);
            } else if (p.fused) {
                auto kern = kmeans_assign_fused<VPL, R>;
                EP_CUDA(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem));
                int64_t rpw = ceil_div(ceil_div(N, p.grid), p.warps);
                rpw = ceil_div(rpw, R) * R;
                int64_t rpb = rpw * p.warps;
                Timed tm(ctx, stream, EP_TIMER_KMEANS_ASSIGN);
                kern<<<p.grid, p.warps * 32, p.smem, stream>>>(emb, N, d, K, Kpad, centroids, b.cnorm, assign, b.psum,
                                                             b.pcnt, rpb, rpw);
                tm.end(1);
            } else {
                if (p.tensor) {
                    int r1 = kmeans_tc_assign(ctx, *tc_state, emb, N, d, K, centroids, b.cnorm, b.clo, b.cmaxima, b.rownorm, assign, b.cand, stream);
                    if (r1 != EP_OK) return r1;
                } else {
                    auto kern = kmeans_assign_chunked<VPL, R>;
                    EP_CUDA(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem));
                    const int row_bytes = VPL * 512;
                    int kchunk = (int)std::min<size_t>(Kpad, (96 * 1024) / row_bytes / KC * KC);
                    Timed tm(ctx, stream, EP_TIMER_KMEANS_ASSIGN);
                    kern<<<p.grid, 256, p.smem, stream>>>(emb, N, d, K, Kpad, kchunk, centroids, b.cnorm, assign);
                    tm.end(1);
                }
                // group the rows by label, then sum each group in a fixed order
                Timed tm(ctx, stream, EP_TIMER_KMEANS_UPDATE);
                EP_CUDA(ctx, cudaMemsetAsync(b.hist, 0, sizeof(unsigned long long) * K, stream));
                label_histogram<<<ctx->sm_count * 4, 256, 0, stream>>>(assign, N, K, b.hist);
                label_offsets<<<1, 256, 0, stream>>>(b.hist, K, b.off);
                int r2 = reorder_run(ctx, assign, N, K, b.order, nullptr, b.sort_ws, stream, /*timed=*/false);
                if (r2 != EP_OK) return r2;
                kmeans_segment_sums<VPL><<<dim3(K, p.parts), 256, 0, stream>>>(emb, d, K, b.order, b.off, b.psum, b.pcnt);
                tm.end(3);
            }
            return EP_OK;
        });
        if (rc != EP_OK) return rc;
        Timed tm(ctx, stream, EP_TIMER_KMEANS_UPDATE);
        if (p.parts >= 32 && d <= 512)
            centroid_update_many<<<K, UPD2_THREADS, 0, stream>>>(b.psum, b.pcnt, p.parts, K, d, centroids, b.cnorm, b.objterm,
                                                         iters == 0 ? 1 : 0, b.ct, b.clo);
        else
            centroid_update_few<<<K, UPD_THREADS, 0, stream>>>(b.psum, b.pcnt, p.parts, K, d, centroids, b.cnorm, b.objterm,
                                                       iters == 0 ? 1 : 0, b.ct, b.clo);
        if (objective) objective_finalize<<<1, 256, 0, stream>>>(b.x2part, X2_BLOCKS, b.objterm, K, objective + t);
        tm.end(objective ? 2 : 1);
    }
    EP_CUDA(ctx, cudaGetLastError());
    return EP_OK;
}

}  // namespace ep
