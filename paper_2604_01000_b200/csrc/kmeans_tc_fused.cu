// Fused assign-and-accumulate pass of Lloyd K-Means (Algorithm 3, the clustering step) for few centroids
// (K <= 64, d <= 128) on the tensor cores: one read of the embedding matrix per iteration.
//
// kmeans_tc_fused: a persistent block per SM streams 128-row tiles of X through a ring of shared-memory
// stages (TMA, 128-byte swizzle).  The TF32-rounded copy of all K centroids sits in shared memory for the
// whole launch.  Four kinds of warps work on consecutive tiles at the same time, handing tiles on through
// mbarriers (every wait has a time limit):
//   1. one thread issues tcgen05.mma kind::tf32: scores [128 x K] into one of two TMEM accumulators;
//   2. four screen warps, one row per thread and no barrier between them, read the accumulator back and
//      keep the two smallest packed (score | column) keys.  If the second is farther from the first than
//      the TF32 error bound of that row allows, the first is provably the fp32 argmin and becomes the
//      label.  Otherwise the row id goes to the warp's list of undecided rows, with the set of centroids
//      inside the bound;
//   3. two sorting warps (alternating tiles) group the tile's decided rows by label, stably;
//   4. eight accumulate warps, each owning up to KMAX/8 clusters with one 16-byte column chunk per lane, add
//      the rows of their clusters, in row order, from the shared-memory tile into registers.  Which warp owns
//      which cluster is settled per launch from the block's own counts of the previous iteration, so that
//      uneven clusters still give the warps even work; a cluster's rows are added by one warp in row order
//      whoever that is, so the sums do not depend on it.
// After its last tile the block settles the rows its screen warps left undecided: their squared distances
// sum_j (x_j - c_j)^2 to the listed centroids in fp32 (lowest index wins ties), the label, and the row added to
// the block's sums after all decided rows, in list order.  No floating-point atomics anywhere: the order of
// every addition is fixed by the launch shape and the lists, so results repeat bit for bit.
//
// All Lloyd iterations of a call run inside ONE launch (a cooperative launch: the blocks are resident together).
// After an iteration's tiles the blocks meet on a grid-wide barrier (a counter, polled with a time limit), block k
// turns the published partial sums into the new centroid k (fp64, fixed order), they meet again, and the next
// iteration's tiles start: no launch gap, no prologue and no second kernel between iterations.
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
constexpr int MAX_KB = 8;               // d <= 256
constexpr int MAX_STAGES = 8;
constexpr int THREADS = 512;            // warp 0 TMA, 1 MMA, 2..3 sorting (2 also owns TMEM), 4..7 screen, 8..15 accumulate
constexpr int S_WARP0 = 4;
constexpr int A_WARP0 = 8;
constexpr int A_WARPS = 8;
constexpr int MAX_K = 64;
constexpr int LATE_WARPS = THREADS / 32;   // every warp of the block works on the undecided rows
constexpr int MAX_LATE_CHUNK = 256;        // undecided rows held in shared memory at a time

// Phase clocks for tuning (compiled in with -DEP_PHASE_CLOCKS only): thread 0 of a warp set adds up how long
// it waited and how long it worked, into the diagnostic counters.
#ifdef EP_PHASE_CLOCKS
#define EP_CLK_DECL long long pc_wait = 0, pc_work = 0, pc_t = clock64();
#define EP_CLK(var)                        \
    {                                      \
        const long long now_ = clock64();  \
        var += now_ - pc_t;                \
        pc_t = now_;                       \
    }
#define EP_CLK_OUT(cond, iw, ik)                                      \
    if (counters && (cond)) {                                         \
        atomicAdd(&counters[iw], (unsigned long long)pc_wait);        \
        atomicAdd(&counters[ik], (unsigned long long)pc_work);        \
    }
#else
#define EP_CLK_DECL
#define EP_CLK(var)
#define EP_CLK_OUT(cond, iw, ik)
#endif

struct FusedShared {
    uint64_t x_full[MAX_STAGES], x_empty[MAX_STAGES];
    uint64_t c_full;
    uint64_t t_full[2], t_empty[2];
    uint64_t lab_full[2], lab_empty[2];
    uint64_t ord_full[2], ord_empty[2];
    uint64_t plan_full;
    uint64_t drain;                     // after an abort: the MMAs still in flight have completed
    uint32_t tmem_base;
    int abort;
    uint8_t lab[2][BM];                 // sorting key of each row of the tile; MAX_K = not to be accumulated here
    uint16_t order[2][BM];              // the tile's rows grouped by sorting key, ascending row inside a key, each as
                                        // its byte offset inside a k-block with the swizzle term in bits 4..6
    int goff[2][MAX_K + 1];             // first position of each label in order[]
    int hcnt[2][MAX_K + 1];             // scratch of the two sorting warps; hcnt[1] first holds the weights of the
                                        // clusters while warp 3 shares the accumulate work out
    int cnt[MAX_K];                     // rows per sorting key that this block decided
    uint8_t plan_sorted[MAX_K];         // clusters by descending weight
    uint8_t keymap[MAX_K + 1];          // cluster -> sorting key = owner warp * OWN + slot; [MAX_K] = MAX_K
    int8_t kof[MAX_K];                  // sorting key -> cluster, -1 = no cluster
    alignas(16) float cn[MAX_K];
    uint64_t late_bar[LATE_WARPS];      // one per warp: its undecided rows of the current chunk have arrived
    int late_n[4];                      // entries in each screen warp's list of undecided rows
    int late_cum[5];                    // their running totals
};
// With 64 centroids of 128 floats, three 64 KB stages fit beside this block and the centroid tile only while it
// stays within 3 KB; a fourth of the pass's speed hangs on the third stage.
static_assert(sizeof(FusedShared) <= 3072, "FusedShared has outgrown the room beside three stages");
static_assert(MAX_LATE_CHUNK <= 2 * BM, "the labels of a chunk of undecided rows reuse FusedShared::lab");

// 16 accumulator columns, issued without waiting: several of these go out before one tmem_wait().
template <int O, int VN>
__device__ __forceinline__ void tmem_issue16(uint32_t taddr, uint32_t (&v)[VN]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[O + 0]), "=r"(v[O + 1]), "=r"(v[O + 2]), "=r"(v[O + 3]), "=r"(v[O + 4]), "=r"(v[O + 5]), "=r"(v[O + 6]),
          "=r"(v[O + 7]), "=r"(v[O + 8]), "=r"(v[O + 9]), "=r"(v[O + 10]), "=r"(v[O + 11]), "=r"(v[O + 12]),
          "=r"(v[O + 13]), "=r"(v[O + 14]), "=r"(v[O + 15])
        : "r"(taddr + O)
        : "memory");
}
// a += x where i < n, as four predicated additions: no branch, whatever the compiler thinks of the condition.
__device__ __forceinline__ void add_if_less(float4 &a, const float4 &x, int i, int n) {
    asm("{\n.reg .pred p;\n"
        "setp.lt.s32 p, %8, %9;\n"
        "@p add.rn.f32 %0, %0, %4;\n"
        "@p add.rn.f32 %1, %1, %5;\n"
        "@p add.rn.f32 %2, %2, %6;\n"
        "@p add.rn.f32 %3, %3, %7;\n}"
        : "+f"(a.x), "+f"(a.y), "+f"(a.z), "+f"(a.w)
        : "f"(x.x), "f"(x.y), "f"(x.z), "f"(x.w), "r"(i), "r"(n));
}
__device__ __forceinline__ void tmem_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Every block of the (cooperative) grid has arrived `target` times in total.  Bounded: after GRID_WAIT_CLOCKS, or
// once this block has given up elsewhere, the block's abort flag is set and false comes back.
constexpr long long GRID_WAIT_CLOCKS = 4000000000ll;
__device__ __noinline__ bool grid_barrier(unsigned *bar, unsigned target, volatile int *abort_flag) {
    __syncthreads();
    if (threadIdx.x == 0) {
        // the arrival releases what this block wrote (the __syncthreads above ordered the other threads' writes before
        // it); the acquiring load that sees the last arrival makes every block's writes visible here
        asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(bar) : "memory");
        const long long t0 = clock64();
        for (unsigned spins = 0;; ++spins) {
            unsigned seen;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(bar) : "memory");
            if (seen >= target || *abort_flag) break;
            if ((spins & 31u) == 31u && clock64() - t0 > GRID_WAIT_CLOCKS) {
                *abort_flag = 1;
                break;
            }
        }
    }
    __syncthreads();
    return *abort_flag == 0;
}

// Sums of four doubles per thread over the block, in a fixed order: a butterfly inside each warp, then the warps'
// results in warp order (red: 4 x 16 doubles of shared memory).  Every thread gets the four totals.
__device__ __forceinline__ void block_sum4(double (&v)[4], double *red) {
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1)
#pragma unroll
        for (int i = 0; i < 4; ++i) v[i] += __shfl_xor_sync(FULL, v[i], o);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0)
#pragma unroll
        for (int i = 0; i < 4; ++i) red[i * (THREADS / 32) + warp] = v[i];
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        double t = 0.0;
#pragma unroll
        for (int w = 0; w < THREADS / 32; ++w) t += red[i * (THREADS / 32) + w];
        v[i] = t;
    }
}

__device__ __forceinline__ float tf32_nearest(float x) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return __uint_as_float(r);
}

// The centroid update shared out over the whole grid: a unit is W four-float columns of one cluster (W a power of
// two, at most 32), so that K x ceil(d / 4W) units keep about every block busy and a block pulls only 16 W bytes of
// each slab.  Groups of W threads take contiguous shares of the slabs in slab order; the groups of a warp are added by
// a butterfly, the warps in warp order: a fixed tree.  The unit writes its columns of c_k and of the TF32 copy, and to
// tpart[unit] its share of (n_k |c|^2 - 2 c.S_k, |c'|^2, |c' - tf32(c')|^2); whoever needs |c'|^2, the residual or the
// objective of a cluster adds the shares of its units in unit order (cluster_terms).  buf: 4 x 16 x 32 + 64 doubles.
constexpr int UPDATE_MAX_CHUNKS = 16;
__device__ __forceinline__ int update_chunk_width(int K, int d4, int grid) {
    int W = 1;
    while (W < 32 && (K * ((d4 + W - 1) / W) > grid || (d4 + W - 1) / W > UPDATE_MAX_CHUNKS)) W <<= 1;
    return W;
}
__device__ __noinline__ void update_unit(int k, int c, int W, int K, int d, int parts, const float *psum, const int *pcnt,
                                            float *C, float *ct, double *tpart_unit, int keep_centroids, double *buf) {
    const int d4 = d >> 2;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = THREADS / W, g = threadIdx.x / W, q = threadIdx.x & (W - 1);
    const int col = c * W + q;                                   // this thread's four columns
    double *red = buf + 4 * (THREADS / 32) * 32;
    // every load is issued before anything waits on one
    double sums[4] = {0.0, 0.0, 0.0, 0.0};
    for (int p = threadIdx.x; p < parts; p += THREADS) sums[0] += (double)__ldcg(pcnt + (size_t)p * K + k);
    float4 c4 = make_float4(0.f, 0.f, 0.f, 0.f);
    if (g == 0 && col < d4) c4 = __ldcg(reinterpret_cast<const float4 *>(C) + (size_t)k * d4 + col);
    double part[4] = {0.0, 0.0, 0.0, 0.0};
    if (col < d4) {
        const int p0 = (int)((long long)parts * g / G), p1 = (int)((long long)parts * (g + 1) / G);
        const float4 *src = reinterpret_cast<const float4 *>(psum) + (size_t)k * d4 + col;
        const size_t pitch = (size_t)K * d4;
#pragma unroll 1
        for (int pb = p0; pb < p1; pb += 4) {
            float4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                v[u] = pb + u < p1 ? __ldcg(src + (size_t)(pb + u) * pitch) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                part[0] += (double)v[u].x;
                part[1] += (double)v[u].y;
                part[2] += (double)v[u].z;
                part[3] += (double)v[u].w;
            }
        }
    }
    block_sum4(sums, red);
    const long long n = (long long)sums[0];                     // counts are far below 2^53: exact
    for (int o = 16; o >= W; o >>= 1)                            // the groups of this warp (lanes that differ above q)
#pragma unroll
        for (int i = 0; i < 4; ++i) part[i] += __shfl_xor_sync(FULL, part[i], o);
    __syncthreads();
    if (lane < W)
#pragma unroll
        for (int i = 0; i < 4; ++i) buf[(i * (THREADS / 32) + warp) * 32 + lane] = part[i];
    __syncthreads();
    if (warp == 0) {
        double t[3] = {0.0, 0.0, 0.0};                          // n |c|^2 - 2 c.S, |c'|^2, |c' - tf32(c')|^2 of these columns
        if (lane < W && col < d4) {
            const float cold[4] = {c4.x, c4.y, c4.z, c4.w};
            float cnew[4], crnd[4];
            double cs = 0.0, cc = 0.0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                double S = 0.0;
                for (int w = 0; w < THREADS / 32; ++w) S += buf[(i * (THREADS / 32) + w) * 32 + lane];
                cnew[i] = (n > 0 && !keep_centroids) ? (float)(S / (double)n) : cold[i];
                crnd[i] = tf32_nearest(cnew[i]);
                const double lo = (double)cnew[i] - (double)crnd[i];
                cs += (double)cold[i] * S;
                cc += (double)cold[i] * (double)cold[i];
                t[1] += (double)cnew[i] * (double)cnew[i];
                t[2] += lo * lo;
            }
            t[0] = (double)n * cc - 2.0 * cs;
            reinterpret_cast<float4 *>(C)[(size_t)k * d4 + col] = make_float4(cnew[0], cnew[1], cnew[2], cnew[3]);
            reinterpret_cast<float4 *>(ct)[(size_t)k * d4 + col] = make_float4(crnd[0], crnd[1], crnd[2], crnd[3]);
        }
        for (int o = W >> 1; o >= 1; o >>= 1)
#pragma unroll
            for (int i = 0; i < 3; ++i) t[i] += __shfl_xor_sync(FULL, t[i], o);
        if (lane == 0) {
            tpart_unit[0] = t[0];
            tpart_unit[1] = t[1];
            tpart_unit[2] = t[2];
        }
    }
    __syncthreads();
}
// A cluster's (objective term, |c|^2, residual |c - tf32(c)|) from the shares of its units, in unit order.
__device__ __forceinline__ void cluster_terms(const double *tpart, int k, int chunks, double &obj, float &cnorm, float &clo) {
    double t0 = 0.0, t1 = 0.0, t2 = 0.0;
    for (int c = 0; c < chunks; ++c) {
        const double *u = tpart + (size_t)(k * chunks + c) * 4;
        t0 += __ldcg(u + 0);
        t1 += __ldcg(u + 1);
        t2 += __ldcg(u + 2);
    }
    obj = t0;
    cnorm = (float)t1;
    clo = (float)(sqrt(t2) * 1.000001);
}

// J of an iteration = sum_i |x_i|^2 + sum_k (n_k |c_k|^2 - 2 c_k.S_k), both summed in a fixed order, by one block.
__device__ __noinline__ void objective_of_iteration(const double *x2part, int x2n, const double *objterm, int K, double *red,
                                                    double *out) {
    double t[4] = {0.0, 0.0, 0.0, 0.0};
    for (int i = threadIdx.x; i < x2n; i += THREADS) t[0] += x2part[i];
    for (int k = threadIdx.x; k < K; k += THREADS) t[1] += __ldcg(objterm + k);
    block_sum4(t, red);
    if (threadIdx.x == 0) *out = t[0] + t[1];
}

// KMAX = 16, 32 or 64: upper bound of K.  VPL = 16-byte chunks of a row per lane: 1 for d <= 128 with tiles of 128
// rows, 2 for d <= 256 with tiles of 64 rows (the stage stays 64 KB; the MMA still spans 128 TMEM lanes, the upper
// 64 of which then hold scores of whatever follows the tile in shared memory and are never read).
// rownorm[i] = (|x_i|, |x_i - trunc_tf32(x_i)|); clo[k] = |c_k - tf32(c_k)|; cn = |c_k|^2 padded with a huge value;
// centroids = the fp32 centroids themselves (map_c covers their TF32-rounded copy).  Block b leaves the sums of its
// rows in psum[b][K][d] and their counts in pcnt[b][K].  late_list[(4 b + w) late_cap ..] is scratch for the rows
// screen warp w cannot decide (x = row id, y and z = mask of the centroids within the bound); the block settles
// them itself after its last tile, late_chunk rows at a time.
// From the second iteration on (from the first when use_prev0 says so) pcnt[b] holds this block's counts of the previous
// iteration over the same tiles; they weigh the clusters when these are shared out among the accumulate warps (any
// sharing gives the same sums).
// update_here != 0: the launch runs T iterations (T = 1 with keep_centroids: labels against the given centroids only);
// after each, the centroids, cn, their TF32 copy ct (what map_c covers) and clo are rewritten in place by the blocks
// themselves, the cluster terms of the objective go to objterm[K], and block 0 writes objective[iteration] (when asked
// for) from them and the x2n partial sums of squares x2part.  grid_bar: one word, zero before the launch.
// update_here == 0 (T = 1): the launch ends once the sums are published; a separate kernel updates the centroids.
// counters (profiling only): [0] rows screened, [3] rows left undecided by the screening, [5] / [6] clocks block 0
// spent from an iteration's start to its sums being published / from there to the end of the update.
// PERSISTENT = update_here, known at compile time: the one-iteration instance carries none of the loop's bookkeeping.
template <int KMAX, int VPL, bool PERSISTENT>
__global__ void __launch_bounds__(THREADS, 1)
kmeans_tc_fused(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_c,
                const float *__restrict__ emb, float *centroids, float *cn, float *ct, float *clo,
                const float2 *__restrict__ rownorm, int64_t N,
                int d, int K, int npad, int num_kb, int stages, uint32_t idesc, uint32_t tmem_cols, uint32_t key_mask,
                int32_t *__restrict__ assign, float *psum, int *pcnt,
                int4 *late_list, int64_t late_cap, int late_chunk, int T, int update_here, int use_prev0, int keep_centroids,
                double *objterm, double *objective, const double *__restrict__ x2part, int x2n, int x_one_box,
                unsigned *grid_bar,
                unsigned long long *counters, int *status) {
    // The swizzled tiles need 1024-byte alignment.  The array is used as declared (no pointer arithmetic
    // through integers), so that every access below stays a shared-memory instruction; should a launch
    // ever place it differently, the block reports that and leaves before touching anything.
    extern __shared__ __align__(1024) uint8_t smem[];
    if ((smem_u32(smem) & 1023u) != 0u || npad != KMAX) {
        if (threadIdx.x == 0) ep_raise(status, EP_ERR_CUDA);
        return;
    }
    constexpr int BMR = BM / VPL;                      // rows per tile
    constexpr int SWARPS = BMR / 32;                   // screen warps with rows
    constexpr int X_KB_BYTES = BMR * 128;              // one k-block of a row tile
    const int stage_bytes = num_kb * X_KB_BYTES;
    const int c_kb_bytes = KMAX * 128;                 // the host passes npad == KMAX
    uint8_t *x_smem = smem;                                          // [stages][num_kb][128 rows][128 B]
    uint8_t *c_smem = x_smem + (size_t)stages * stage_bytes;         // [num_kb][npad rows][128 B]
    FusedShared *sh = reinterpret_cast<FusedShared *>(c_smem + (size_t)num_kb * c_kb_bytes);
    volatile int *abort_flag = &sh->abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int d4 = d >> 2;
    const int64_t num_tiles = (N + BMR - 1) / BMR;

    if (threadIdx.x == 0) {
#pragma unroll 1
        for (int i = 0; i < MAX_STAGES; ++i) {
            mbar_init(&sh->x_full[i], 1);
            mbar_init(&sh->x_empty[i], A_WARPS);
        }
        mbar_init(&sh->c_full, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sh->t_full[i], 1);
            mbar_init(&sh->t_empty[i], SWARPS);   // the screen warps
            mbar_init(&sh->lab_full[i], SWARPS);
            mbar_init(&sh->lab_empty[i], 1);  // a sorting warp
            mbar_init(&sh->ord_full[i], 1);
            mbar_init(&sh->ord_empty[i], A_WARPS);
        }
        mbar_init(&sh->plan_full, 1);
        mbar_init(&sh->drain, 1);
#pragma unroll 1
        for (int i = 0; i < LATE_WARPS; ++i) mbar_init(&sh->late_bar[i], 1);
        sh->abort = 0;
        sh->tmem_base = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // Between two iterations every barrier of the pipeline rests between phases (every tile was loaded, screened,
    // sorted and accumulated).  A barrier that went through an odd number of phases gets one more, empty one (thread 0
    // supplies all of its arrivals): then all of them stand where they stood at the start, and the tile counters of
    // all warp sets begin every iteration at zero, with the parities of a fresh launch.
    auto even_out_phases = [&](uint32_t tiles, uint32_t chunks) {
        auto flip = [&](uint64_t *bar, uint32_t count, uint32_t phases) {
            if (phases & 1u)
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
        };
#pragma unroll 1
        for (uint32_t st = 0; st < (uint32_t)stages; ++st) {
            const uint32_t ph = st < tiles ? (tiles - st + (uint32_t)stages - 1u) / (uint32_t)stages : 0u;
            flip(&sh->x_full[st], 1, ph);
            flip(&sh->x_empty[st], A_WARPS, ph);
        }
#pragma unroll 1
        for (uint32_t b = 0; b < 2; ++b) {
            const uint32_t ph = b < tiles ? (tiles - b + 1u) / 2u : 0u;
            flip(&sh->t_full[b], 1, ph);
            flip(&sh->t_empty[b], SWARPS, ph);
            flip(&sh->lab_full[b], SWARPS, ph);
            flip(&sh->lab_empty[b], 1, ph);
            flip(&sh->ord_full[b], 1, ph);
            flip(&sh->ord_empty[b], A_WARPS, ph);
        }
        flip(&sh->c_full, 1, 1u);
        flip(&sh->plan_full, 1, 1u);
#pragma unroll 1
        for (int w = 0; w < LATE_WARPS; ++w) flip(&sh->late_bar[w], 1, chunks);
    };
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
    const uint32_t nt = num_tiles > (int64_t)blockIdx.x ? (uint32_t)((num_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x) : 0u;   // tiles of this block
    constexpr uint32_t it_base = 0u, ipar = 0u;
    uint32_t grid_arrivals = 0;
    if (PERSISTENT != (update_here != 0)) {                // the host picks the instance that matches
        if (threadIdx.x == 0) ep_raise(status, EP_ERR_CUDA);
        T = 0;
    }

#pragma unroll 1
    for (int iter = 0; iter < (PERSISTENT ? T : min(T, 1)); ++iter) {
    const int use_prev = (PERSISTENT && iter > 0) || use_prev0;
    uint32_t chunk_it = 0;
    const long long clk_start = clock64();
    if (threadIdx.x < 4) sh->late_n[threadIdx.x] = 0;
    // |c|^2 and the TF32 residual of every centroid: from the caller's arrays, or (after an update inside this launch)
    // from the shares the update's units left, which every block adds up in the same order
    float *clo_s = reinterpret_cast<float *>(sh->hcnt[0]);      // warp 2's scratch, not in use before its first tile
    double *tpart = reinterpret_cast<double *>(grid_bar + 64);
    const int upd_W = update_chunk_width(K, d >> 2, (int)gridDim.x), upd_chunks = ((d >> 2) + upd_W - 1) / upd_W;
    for (int k = threadIdx.x; k < MAX_K; k += blockDim.x) {
        sh->cnt[k] = 0;
        float cnk = CUDART_INF_F, clk = 0.f;                     // beyond K: a huge norm, so that no row goes there
        if (k < K) {
            if (PERSISTENT && iter > 0) {
                double obj;
                cluster_terms(tpart, k, upd_chunks, obj, cnk, clk);
            } else {
                cnk = __ldcg(cn + k);
                clk = __ldcg(clo + k);
            }
        } else if (k < KMAX) {
            cnk = __ldcg(cn + k);
        }
        sh->cn[k] = cnk;
        clo_s[k] = clk;
    }
    __syncthreads();

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer: the whole warp runs the
        // loop (warp-uniform control flow and operands), one elected lane issues.  x_one_box: map_x is the
        // three-dimensional view of X and one box brings a whole tile; else one box per k-block.
        {
            // the centroids' TF32 copy of this iteration (written by other blocks through ordinary stores)
            asm volatile("fence.proxy.async;" ::: "memory");
            mbar_expect_tx_elected(&sh->c_full, (uint32_t)(num_kb * c_kb_bytes));
#pragma unroll 1
            for (int kb = 0; kb < num_kb; ++kb)
                tma_load_2d_elected(smem_u32(c_smem) + (uint32_t)(kb * c_kb_bytes), &map_c, kb * KBLK, 0, &sh->c_full);
            uint32_t it = it_base, s = 0, ph = 0;             // ring stage and phase of the next tile: counters, no division
            for (int64_t tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++it, ph ^= (++s == (uint32_t)stages), s = s == (uint32_t)stages ? 0u : s) {
                if (!__all_sync(FULL, mbar_wait(&sh->x_empty[s], ph ^ 1u, abort_flag))) break;
                mbar_expect_tx_elected(&sh->x_full[s], (uint32_t)stage_bytes);
                const uint32_t dst = smem_u32(x_smem) + s * (uint32_t)stage_bytes;
                if (x_one_box) {
                    tma_load_3d_elected(dst, &map_x, 0, (int)(tile * BMR), 0, &sh->x_full[s]);
                } else {
#pragma unroll 1
                    for (int kb = 0; kb < num_kb; ++kb)
                        tma_load_2d_elected(dst + (uint32_t)(kb * X_KB_BYTES), &map_x, kb * KBLK, (int)(tile * BMR), &sh->x_full[s]);
                }
            }
            if (lane == 0 && *abort_flag) {
                // On the way out after an abort: the loads already issued get time to land, so that nothing of this
                // block's own still writes into its shared memory when it leaves.
                mbar_wait_quiet(&sh->c_full, ipar, DRAIN_LIMIT_CLOCKS);
#pragma unroll 1
                for (uint32_t j = it > (uint32_t)stages ? it - (uint32_t)stages : 0u; j < it; ++j)
                    mbar_wait_quiet(&sh->x_full[j % (uint32_t)stages], (j / (uint32_t)stages) & 1u, DRAIN_LIMIT_CLOCKS);
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer: the whole warp runs the loop,
        // one elected lane issues (see the elected forms in tc_device.cuh)
        {
            bool ok = __all_sync(FULL, mbar_wait(&sh->c_full, ipar, abort_flag));
            uint32_t it = it_base, s = 0, ph = 0;
            for (int64_t tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++it, ph ^= (++s == (uint32_t)stages), s = s == (uint32_t)stages ? 0u : s) {
                const uint32_t buf = it & 1u, use = (it >> 1) & 1u;
                if (!(ok = __all_sync(FULL, mbar_wait(&sh->t_empty[buf], use ^ 1u, abort_flag)))) break;
                if (!(ok = __all_sync(FULL, mbar_wait(&sh->x_full[s], ph, abort_flag)))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * (uint32_t)KMAX;
                const uint32_t a_addr = smem_u32(x_smem) + s * (uint32_t)stage_bytes, b_addr = smem_u32(c_smem);
                static_assert(KBLK == 32, "umma_tf32_kblock_elected issues the four K-steps of a 32-float k-block");
#pragma unroll 1
                for (int kb = 0; kb < num_kb; ++kb)
                    umma_tf32_kblock_elected(d_tmem, umma_desc(a_addr + (uint32_t)(kb * X_KB_BYTES)),
                                             umma_desc(b_addr + (uint32_t)(kb * c_kb_bytes)), idesc, (uint32_t)kb);
                umma_commit_elected(&sh->t_full[buf]);
            }
            if (__any_sync(FULL, !ok || *abort_flag)) {
                // after an abort the accumulators are given back at the end of the kernel: first every MMA issued
                // here must have completed (the commit comes from the lane that issued them: the same election)
                umma_commit_elected(&sh->drain);                  // only ever used once: the block leaves after an abort
                if (lane == 0) mbar_wait_quiet(&sh->drain, 0u, DRAIN_LIMIT_CLOCKS);
            }
        }
    }
    if (warp == 2 || warp == 3) {
        // ---------------------------------------------------------------- sorting warps: warp 2 takes the
        // block's even tiles, warp 3 the odd ones.  A stable counting sort of the tile's 128 rows by label,
        // so that an accumulate warp finds the rows of a cluster as one run, in row order.
        const uint32_t hw = (uint32_t)warp - 2u;
        const unsigned lt = (1u << lane) - 1u;
        if (warp == 3) {
            // Which accumulate warp owns which cluster: heaviest cluster first, each to the warp with the least
            // weight so far that still has a free slot (OWN slots per warp).  The weight of a cluster is the number
            // of rows it got from this block's tiles in the previous iteration (+ 1), so the warps end up with
            // about the same number of rows per tile however uneven the clusters are.
            // (runs once per launch: its loops stay rolled, the kernel's code is large as it is)
            constexpr int OWN = KMAX / A_WARPS;
            int *plan_cnt = sh->hcnt[1];               // this warp's own scratch, not yet in use
#pragma unroll 1
            for (int k = lane; k <= MAX_K; k += 32) sh->keymap[k] = (uint8_t)MAX_K;
#pragma unroll 1
            for (int q = lane; q < MAX_K; q += 32) {
                sh->kof[q] = (int8_t)-1;
                int w = 0;
                if (q < K) w = 1 + (use_prev ? min(max(__ldcg(pcnt + (size_t)blockIdx.x * K + q), 0), 1 << 24) : 0);
                plan_cnt[q] = w;
            }
            __syncwarp();
#pragma unroll 1
            for (int k = lane; k < K; k += 32) {
                const int mine = plan_cnt[k];
                int rank = 0;
#pragma unroll 1
                for (int j = 0; j < K; ++j) {
                    const int o = plan_cnt[j];
                    rank += (o > mine || (o == mine && j < k)) ? 1 : 0;
                }
                sh->plan_sorted[rank] = (uint8_t)k;
            }
            __syncwarp();
            unsigned load = 0u;
            int taken = 0;
#pragma unroll 1
            for (int r = 0; r < K; ++r) {
                const int k = sh->plan_sorted[r];
                const unsigned key = (lane < A_WARPS && taken < OWN) ? ((load << 3) | (unsigned)lane) : 0xFFFFFFFFu;
                const unsigned best = __reduce_min_sync(FULL, key);
                if (lane < A_WARPS && key == best) {
                    sh->keymap[k] = (uint8_t)(lane * OWN + taken);
                    sh->kof[lane * OWN + taken] = (int8_t)k;
                    ++taken;
                    load += (unsigned)plan_cnt[k];
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh->plan_full);
        }
        EP_CLK_DECL
        for (uint32_t j = 0; j < nt; ++j) {
            const uint32_t it = it_base + j;
            if ((it & 1u) != hw) continue;             // warp 2 takes the even tiles of the running count, warp 3 the odd ones
            const uint32_t par = hw, use = (it >> 1) & 1u;
            EP_CLK(pc_work)
            if (!mbar_wait(&sh->lab_full[par], use, abort_flag)) break;
            EP_CLK(pc_wait)
            int l[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) l[j] = j < SWARPS ? (int)sh->lab[par][j * 32 + lane] : MAX_K;
            for (int i = lane; i <= MAX_K; i += 32) sh->hcnt[hw][i] = 0;
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh->lab_empty[par]);
            int before[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const unsigned peers = __match_any_sync(FULL, l[j]);
                const int leader = __ffs(peers) - 1;
                int old = 0;
                if (lane == leader) {
                    old = sh->hcnt[hw][l[j]];
                    sh->hcnt[hw][l[j]] = old + __popc(peers);
                }
                before[j] = __shfl_sync(FULL, old, leader) + __popc(peers & lt);
                __syncwarp();
            }
            const int t0 = sh->hcnt[hw][2 * lane], t1 = sh->hcnt[hw][2 * lane + 1];
            int inc = t0 + t1;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int up = __shfl_up_sync(FULL, inc, o);
                if (lane >= o) inc += up;
            }
            const int ex = inc - t0 - t1;
            if (t0) atomicAdd(&sh->cnt[2 * lane], t0);       // integer: exact whatever the order
            if (t1) atomicAdd(&sh->cnt[2 * lane + 1], t1);
            EP_CLK(pc_work)
            if (!mbar_wait(&sh->ord_empty[par], use ^ 1u, abort_flag)) break;
            EP_CLK(pc_wait)
            sh->goff[par][2 * lane] = ex;
            sh->goff[par][2 * lane + 1] = ex + t0;
            if (lane == 31) sh->goff[par][MAX_K] = inc;
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (l[j] < MAX_K) {
                    const int r = j * 32 + lane;
                    sh->order[par][sh->goff[par][l[j]] + before[j]] = (uint16_t)((r << 7) | ((r & 7) << 4));
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh->ord_full[par]);
        }
        EP_CLK_OUT(warp == 2 && lane == 0, 4, 5)
    } else if (warp >= S_WARP0 && warp < A_WARP0) {
        // ---------------------------------------------------------------- screen warps: one row per thread,
        // each warp on its own (no barrier between them): TMEM lanes 32 sw .. 32 sw + 31 = rows of the tile
        const int sw = warp - S_WARP0;
        const int stid = threadIdx.x - S_WARP0 * 32;       // row in tile
        float m2 = 0.f, ml = 0.f;                          // largest centroid norm and rounding residual
#pragma unroll 1
        for (int k = lane; k < K; k += 32) {
            m2 = fmaxf(m2, sh->cn[k]);
            ml = fmaxf(ml, clo_s[k]);
        }
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) {
            m2 = fmaxf(m2, __shfl_xor_sync(FULL, m2, o));
            ml = fmaxf(ml, __shfl_xor_sync(FULL, ml, o));
        }
        const float cmax2 = m2, clomax = ml;
        const float cmax = sqrtf(cmax2) * 1.000001f;
        const unsigned lt = (1u << lane) - 1u;
        int4 *late_rows = late_list + ((size_t)blockIdx.x * 4 + sw) * late_cap;
        int late_n = 0;
        unsigned n_rows = 0;
        EP_CLK_DECL

        float2 nr_next = make_float2(0.f, 0.f);            // this row's norms, fetched one tile ahead
        if (sw < SWARPS && (int64_t)blockIdx.x * BMR + stid < N) nr_next = __ldg(rownorm + (int64_t)blockIdx.x * BMR + stid);

        bool planned = mbar_wait(&sh->plan_full, ipar, abort_flag);
        uint32_t it = it_base;
        for (int64_t tile = blockIdx.x; planned && sw < SWARPS && tile < num_tiles; tile += gridDim.x, ++it) {
            const uint32_t buf = it & 1u, use = (it >> 1) & 1u, par = it & 1u;
            const int64_t row = tile * BMR + stid;
            const float2 nr = nr_next;
            {
                const int64_t nrow = (tile + gridDim.x) * BMR + stid;
                if (nrow < N) nr_next = __ldg(rownorm + nrow);
            }
            EP_CLK(pc_work)
            if (!mbar_wait(&sh->t_full[buf], use, abort_flag)) break;
            EP_CLK(pc_wait)
            tc_fence_after();
            // ---- all of this row's screened products into registers, then the accumulator is free again
            const uint32_t taddr = tmem_base + ((uint32_t)(sw * 32) << 16) + buf * (uint32_t)KMAX;
            uint32_t v[KMAX];
            tmem_issue16<0>(taddr, v);                     // npad == KMAX: no test inside the tile loop depends on K
            if constexpr (KMAX > 16) tmem_issue16<16>(taddr, v);
            if constexpr (KMAX > 32) {
                tmem_issue16<32>(taddr, v);
                tmem_issue16<48>(taddr, v);
            }
            tmem_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh->t_empty[buf]);
            float key1[4], key2[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) key1[i] = key2[i] = __uint_as_float(KEY_INIT);
#pragma unroll
            for (int c = 0; c < KMAX; c += 16) {
#pragma unroll
                for (int j4 = 0; j4 < 16; j4 += 4) {
                    const float4 n4 = *reinterpret_cast<const float4 *>(&sh->cn[c + j4]);
                    const float nn[4] = {n4.x, n4.y, n4.z, n4.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float sc = fmaf(-2.f, __uint_as_float(v[c + j4 + j]), nn[j]);
                        v[c + j4 + j] = __float_as_uint(sc);
                        keep_two(key1[j], key2[j],
                                 __uint_as_float((__float_as_uint(sc) & key_mask) | (uint32_t)(c + j4 + j)));
                    }
                }
            }
            const float lo01 = fminf(key1[0], key1[1]), hi01 = fminf(fmaxf(key1[0], key1[1]), fminf(key2[0], key2[1]));
            const float lo23 = fminf(key1[2], key1[3]), hi23 = fminf(fmaxf(key1[2], key1[3]), fminf(key2[2], key2[3]));
            const float k1 = fminf(lo01, lo23);
            const float k2 = fminf(fmaxf(lo01, lo23), fminf(hi01, hi23));
            const float thr = k1 + 2.f * screen_allowance(nr.x, nr.y, cmax, cmax2, clomax, d);
            const int i1 = (int)(__float_as_uint(k1) & IDX_MASK);
            const bool live = row < N;
            const bool decided = k2 > thr && i1 < K;       // the best screened score cannot be overtaken
            const bool undecided = live && !decided;
            const int label = (live && decided) ? i1 : MAX_K;   // MAX_K: not accumulated by this kernel
            const unsigned todo = __ballot_sync(FULL, undecided);
            if (todo) {
                // Rows that the screening cannot decide are not settled here: their ids go, in row order, to
                // this warp's list, each with the set of centroids whose screened score is within the allowance
                // of the row's best (bit c of the two mask words); the block settles them after its last tile.
                if (undecided) {
                    uint32_t mlo = 0u, mhi = 0u;
#pragma unroll
                    for (int c = 0; c < KMAX; ++c) {
                        const uint32_t hit = __uint_as_float(v[c]) <= thr ? 1u : 0u;
                        if (c < 32)
                            mlo |= hit << (c & 31);
                        else
                            mhi |= hit << (c & 31);
                    }
                    mlo &= K >= 32 ? 0xFFFFFFFFu : (1u << K) - 1u;     // columns beyond K are padding
                    mhi &= K >= 64 ? 0xFFFFFFFFu : K > 32 ? (1u << (K - 32)) - 1u : 0u;
                    if (EP_INDEX_OK(late_n + __popc(todo & lt), late_cap, status))
                        late_rows[(size_t)late_n + __popc(todo & lt)] = make_int4((int)row, (int)mlo, (int)mhi, 0);
                }
                late_n += __popc(todo);
            }
            if (live) {
                if (decided) assign[row] = label;
                ++n_rows;
            }
            // ---- hand the labels to the sorting warp
            EP_CLK(pc_work)
            if (!mbar_wait(&sh->lab_empty[par], use ^ 1u, abort_flag)) break;
            EP_CLK(pc_wait)
            sh->lab[par][stid] = sh->keymap[label];        // the sorting key: owner warp, then the owner's slot
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh->lab_full[par]);
        }
        EP_CLK_OUT(stid == 0, 1, 2)
        if (lane == 0) sh->late_n[sw] = late_n;
        if (counters) {
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) n_rows += __shfl_xor_sync(FULL, n_rows, o);
            if (lane == 0) {
                atomicAdd(&counters[0], (unsigned long long)n_rows);
                atomicAdd(&counters[3], (unsigned long long)late_n);
            }
        }
    } else if (warp >= A_WARP0) {
        // ---------------------------------------------------------------- accumulate warps
        const int aw = warp - A_WARP0;                     // owns the clusters with sorting keys aw OWN .. aw OWN + OWN - 1
        constexpr int OWN = KMAX / A_WARPS;
        const uint32_t lx = (uint32_t)(lane & 7) << 4;     // a lane's place inside a 128-byte swizzle row, before the swizzle
        float4 acc[OWN][VPL];                              // this lane's 16-byte chunks of a row are lane, lane + 32
#pragma unroll
        for (int i = 0; i < OWN; ++i)
#pragma unroll
            for (int v = 0; v < VPL; ++v) acc[i][v] = make_float4(0.f, 0.f, 0.f, 0.f);
        bool planned = mbar_wait(&sh->plan_full, ipar, abort_flag);
        EP_CLK_DECL
        uint32_t it = it_base, s = 0, ph = 0;
        for (int64_t tile = blockIdx.x; planned && tile < num_tiles; tile += gridDim.x, ++it, ph ^= (++s == (uint32_t)stages), s = s == (uint32_t)stages ? 0u : s) {
            const uint32_t par = it & 1u, use = (it >> 1) & 1u;
            const uint8_t *xl = x_smem + (size_t)s * stage_bytes + (size_t)(lane >> 3) * X_KB_BYTES;   // this lane's first k-block
            EP_CLK(pc_work)
            if (!mbar_wait(&sh->ord_full[par], use, abort_flag)) break;
            if (!mbar_wait(&sh->x_full[s], ph, abort_flag)) break;   // long complete: makes the tile visible here
            EP_CLK(pc_wait)
            // The rows of this warp's clusters are one stretch of order[], slot after slot; lane i holds where
            // slot i starts (lane OWN: where the stretch ends).
            const int bl = sh->goff[par][aw * OWN + min(lane, OWN)];
            auto load_row = [&](float4 (&x)[VPL], uint32_t o) {
#pragma unroll
                for (int v = 0; v < VPL; ++v)
                    x[v] = lane + 32 * v < d4 ? *reinterpret_cast<const float4 *>(xl + (size_t)(4 * v) * X_KB_BYTES + (o ^ lx))
                                              : make_float4(0.f, 0.f, 0.f, 0.f);
            };
#pragma unroll
            for (int i = 0; i < OWN; ++i) {
                const int p1 = __shfl_sync(FULL, bl, i + 1);
                for (int p = __shfl_sync(FULL, bl, i); p < p1; p += 4) {       // four rows at a time: loads first, adds in row order
                    float4 x[4][VPL];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {              // a run's last group is not padded with repeated reads
                        if (p + u < p1) {
                            load_row(x[u], (uint32_t)sh->order[par][p + u] & 0x3FF0u);
                        } else {
#pragma unroll
                            for (int v = 0; v < VPL; ++v) x[u][v] = make_float4(0.f, 0.f, 0.f, 0.f);
                        }
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u)
#pragma unroll
                        for (int v = 0; v < VPL; ++v) add_if_less(acc[i][v], x[u][v], p + u, p1);
                }
            }
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&sh->x_empty[s]);
                mbar_arrive(&sh->ord_empty[par]);
            }
        }
        EP_CLK_OUT(aw == 0 && lane == 0, 6, 7)
        // ---- this block's sums of the decided rows go to shared memory, where the undecided rows are added to them.
        // The table takes the place of the first tiles of the ring, so every accumulate warp must have read its last
        // row first (all eight arrive here whatever happened; nobody else touches the ring any more).
        asm volatile("bar.sync 2, %0;" ::"n"(A_WARPS * 32) : "memory");
        float4 *acc_s = reinterpret_cast<float4 *>(x_smem);                 // [K][d4]
#pragma unroll
        for (int i = 0; i < OWN; ++i) {
            const int k = planned ? (int)sh->kof[aw * OWN + i] : -1;
            if (k >= 0 && k < K) {
#pragma unroll
                for (int v = 0; v < VPL; ++v)
                    if (lane + 32 * v < d4) acc_s[(size_t)k * d4 + lane + 32 * v] = acc[i][v];
            }
        }
    }
    __syncthreads();
    if (sh->abort != 0) break;
    {
        // ---------------------------------------------------------------- the rows the screening left undecided
        // All 16 warps.  The ring is free now: it holds the block's sums (acc_s, above), the fp32 centroids (cs) and
        // late_chunk rows at a time (rows_s), fetched by bulk copies, a warp's share on a barrier of its own.
        //   1. warp w settles rows w per .. w per + per - 1 of the chunk: squared distances sum_j (x_j - c_j)^2 to the
        //      centroids the row's mask names (all K if the mask is empty, which NaN scores cause), eight per
        //      reduction, lowest index winning ties; the label goes to assign[] and to late_lab[].
        //   2. warp w adds the chunk's rows with label k = w (mod 16), in list order, to acc_s[k]: one warp per
        //      cluster, so every sum has one fixed order.
        float4 *acc_s = reinterpret_cast<float4 *>(x_smem);                 // [K][d4]
        float4 *cs = acc_s + (size_t)K * d4;                                // [K][d4]
        float4 *rows_s = cs + (size_t)K * d4;                               // [late_chunk][d4]
        uint8_t *late_lab = &sh->lab[0][0];                                 // [late_chunk] labels of the chunk's rows, 255 = none
        const float4 *C4 = reinterpret_cast<const float4 *>(centroids);
#pragma unroll 1
        for (int i = threadIdx.x; i < K * d4; i += THREADS) cs[i] = __ldcg(C4 + i);
        if (threadIdx.x == 0) {
            int run = 0;
#pragma unroll 1
            for (int w = 0; w < 4; ++w) {
                sh->late_cum[w] = run;
                run += min(max(sh->late_n[w], 0), (int)late_cap);
            }
            sh->late_cum[4] = run;
        }
        __syncthreads();
        const int total = sh->late_cum[4];
        const int cum1 = sh->late_cum[1], cum2 = sh->late_cum[2], cum3 = sh->late_cum[3];
        const int4 *lists = late_list + (size_t)blockIdx.x * 4 * late_cap;
        const int slot = lane_chunk_slot(lane);
        const uint32_t row_bytes = (uint32_t)d * 4u;
#pragma unroll 1
        for (int p0 = 0; p0 < total; p0 += late_chunk, ++chunk_it) {
            // ---- 1. fetch and settle this warp's rows: an even share of the chunk, at most 32
            const int cn_rows = min(late_chunk, total - p0);
            const int per = (cn_rows + LATE_WARPS - 1) / LATE_WARPS;
            const int pw = p0 + warp * per;
            const int nw = max(0, min(per, total - pw));
            int4 e = make_int4(-1, 0, 0, 0);
            if (lane < nw) {
                const int p = pw + lane;
                const int w = (p >= cum1) + (p >= cum2) + (p >= cum3);
                e = lists[(size_t)w * late_cap + (p - sh->late_cum[w])];
                if (e.x < 0 || e.x >= N) e.x = -1;                          // never index outside the matrix
            }
            const unsigned have = __ballot_sync(FULL, e.x >= 0);
            bool arrived = true;
            if (have) {
                if (lane == 0) mbar_expect_tx(&sh->late_bar[warp], (uint32_t)__popc(have) * row_bytes);
                __syncwarp();
                if (e.x >= 0)
                    bulk_load_1d(rows_s + (size_t)(warp * per + lane) * d4, emb + (size_t)e.x * d, row_bytes, &sh->late_bar[warp]);
                arrived = mbar_wait(&sh->late_bar[warp], chunk_it & 1u, abort_flag);
            } else if (lane == 0) {
                mbar_arrive(&sh->late_bar[warp]);                           // keeps this barrier's phase in step with the chunks
            }
#pragma unroll 1
            for (int r = 0; r < nw; ++r) {
                const int row = __shfl_sync(FULL, e.x, r);
                const uint32_t mlo = (uint32_t)__shfl_sync(FULL, e.y, r), mhi = (uint32_t)__shfl_sync(FULL, e.z, r);
                if (row < 0 || !arrived) {
                    if (lane == 0) late_lab[warp * per + r] = 255;
                    continue;
                }
                float4 x[VPL];
#pragma unroll
                for (int v = 0; v < VPL; ++v)
                    x[v] = lane + 32 * v < d4 ? rows_s[(size_t)(warp * per + r) * d4 + lane + 32 * v] : make_float4(0.f, 0.f, 0.f, 0.f);
                unsigned long long m = ((unsigned long long)mhi << 32) | mlo;
                if (K < 64) m &= (1ull << K) - 1ull;
                if (m == 0ull) m = K < 64 ? (1ull << K) - 1ull : ~0ull;
                float best = CUDART_INF_F;
                int bidx = 0x7fffffff;
                if (__popcll(m) <= 2) {
                    // the usual near tie, between two centroids: two sums side by side
                    // |x - c|^2 itself, not |c|^2 - 2 x.c: these rows are the near ties, and the direct form
                    // resolves a gap relative to the distance even when the norms are far larger than it
                    const int k0 = __ffsll((long long)m) - 1;
                    const unsigned long long rest = m & (m - 1);
                    const int k1 = rest ? __ffsll((long long)rest) - 1 : k0;
                    float a0 = 0.f, a1 = 0.f;
#pragma unroll
                    for (int v = 0; v < VPL; ++v) {
                        if (lane + 32 * v < d4) {
                            a0 = dist4(x[v], cs[(size_t)k0 * d4 + lane + 32 * v], a0);
                            a1 = dist4(x[v], cs[(size_t)k1 * d4 + lane + 32 * v], a1);
                        }
                    }
#pragma unroll
                    for (int o = 16; o >= 1; o >>= 1) {
                        a0 += __shfl_xor_sync(FULL, a0, o);
                        a1 += __shfl_xor_sync(FULL, a1, o);
                    }
                    const int lab2 = (a1 < a0 || !(a0 == a0)) ? k1 : k0;      // k0 < k1: it keeps a tie
                    if (lane == 0) {
                        assign[row] = lab2;
                        late_lab[warp * per + r] = (uint8_t)lab2;
                    }
                    continue;
                }
                while (m) {
                    float a[KC];
                    int myk = -1;
#pragma unroll
                    for (int kk = 0; kk < KC; ++kk) {        // the next eight named centroids (fewer at the end)
                        a[kk] = 0.f;
                        if (m) {
                            const int k = __ffsll((long long)m) - 1;
                            m &= m - 1;
                            if (kk == slot) myk = k;
#pragma unroll
                            for (int v = 0; v < VPL; ++v)
                                if (lane + 32 * v < d4) a[kk] = dist4(x[v], cs[(size_t)k * d4 + lane + 32 * v], a[kk]);
                        }
                    }
                    // |x - c|^2 itself, not |c|^2 - 2 x.c: these rows are the near ties, and the direct form
                    // resolves a gap relative to the distance even when the norms are far larger than it
                    float sc = reduce8_transposed(a, lane);
                    if (myk >= 0) {
                        sc = (sc == sc) ? sc : CUDART_INF_F;
                        if (sc < best || (sc == best && myk < bidx)) {
                            best = sc;
                            bidx = myk;
                        }
                    }
                }
#pragma unroll
                for (int o = 16; o >= 4; o >>= 1) {          // the eight slots differ in lane bits 4, 3, 2
                    const float ov = __shfl_xor_sync(FULL, best, o);
                    const int oi = __shfl_xor_sync(FULL, bidx, o);
                    if (ov < best || (ov == best && oi < bidx)) {
                        best = ov;
                        bidx = oi;
                    }
                }
                if (bidx < 0 || bidx >= K) bidx = 0;         // a row of NaNs still gets a valid label
                if (lane == 0 && EP_INDEX_OK(warp * per + r, late_chunk, status)) {
                    assign[row] = bidx;
                    late_lab[warp * per + r] = (uint8_t)bidx;
                }
            }
            __syncthreads();
            // ---- 2. add the chunk's rows to the sums of their clusters
#pragma unroll 1
            for (int j0 = 0; j0 < cn_rows; j0 += 32) {
                const int lab = j0 + lane < cn_rows ? (int)late_lab[j0 + lane] : 255;
                const bool mine = lab < K && (lab & (LATE_WARPS - 1)) == warp;
                if (mine) atomicAdd(&sh->cnt[sh->keymap[lab]], 1);           // integer: exact whatever the order
                unsigned mm = __ballot_sync(FULL, mine);
                while (mm) {
                    const int b = __ffs(mm) - 1;
                    mm &= mm - 1;
                    const int k = __shfl_sync(FULL, lab, b);
#pragma unroll
                    for (int v = 0; v < VPL; ++v) {
                        if (lane + 32 * v < d4) {
                            const float4 xr = rows_s[(size_t)(j0 + b) * d4 + lane + 32 * v];
                            float4 t = acc_s[(size_t)k * d4 + lane + 32 * v];
                            t.x += xr.x;
                            t.y += xr.y;
                            t.z += xr.z;
                            t.w += xr.w;
                            acc_s[(size_t)k * d4 + lane + 32 * v] = t;
                        }
                    }
                }
            }
            __syncthreads();                                 // the next chunk overwrites rows_s and late_lab
        }
        // ---- publish this block's sums and counts
        float4 *out = reinterpret_cast<float4 *>(psum) + (size_t)blockIdx.x * K * d4;
#pragma unroll 1
        for (int i = threadIdx.x; i < K * d4; i += THREADS) out[i] = acc_s[i];
#pragma unroll 1
        for (int k = threadIdx.x; k < K; k += blockDim.x) pcnt[(size_t)blockIdx.x * K + k] = sh->cnt[min((int)sh->keymap[k], MAX_K - 1)];

        if (!PERSISTENT) break;
        // ---- the centroid update, by the blocks themselves: every block has published, block k (and k + grid, ...)
        // folds cluster k, and everybody meets again before the next iteration reads the new centroids
        const long long clk_published = clock64();
        grid_arrivals += gridDim.x;
        if (!grid_barrier(grid_bar, grid_arrivals, abort_flag)) break;
        double *buf = reinterpret_cast<double *>(x_smem);     // the block's sums are published: the ring is free again
#pragma unroll 1
        for (int u = blockIdx.x; u < K * upd_chunks; u += gridDim.x)
            update_unit(u / upd_chunks, u % upd_chunks, upd_W, K, d, (int)gridDim.x, psum, pcnt, centroids, ct,
                        tpart + (size_t)u * 4, keep_centroids, buf);
        asm volatile("fence.proxy.async;" ::: "memory");      // ct is next read by the TMA loads of other blocks
        grid_arrivals += gridDim.x;
        if (!grid_barrier(grid_bar, grid_arrivals, abort_flag)) break;
        if (threadIdx.x == 0) even_out_phases(nt, chunk_it);      // nothing of this iteration is in flight any more
        if (blockIdx.x == 0) {
            // the caller's arrays (what a later launch, or the objective below, reads) from the units' shares
            for (int k = threadIdx.x; k < K; k += THREADS) {
                double obj;
                float cnk, clk;
                cluster_terms(tpart, k, upd_chunks, obj, cnk, clk);
                objterm[k] = obj;
                cn[k] = cnk;
                clo[k] = clk;
            }
            __syncthreads();
        }
        if (counters && blockIdx.x == 0 && threadIdx.x == 0) {
            const long long clk_end = clock64();
            atomicAdd(&counters[5], (unsigned long long)(clk_published - clk_start));
            atomicAdd(&counters[6], (unsigned long long)(clk_end - clk_published));
        }
        if (objective && blockIdx.x == 0) objective_of_iteration(x2part, x2n, objterm, K, buf + 4 * THREADS, objective + iter);
    }
    }   // iterations
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) ep_raise(status, EP_ERR_TIMEOUT);
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
    int npad, num_kb, stages, grid, late_chunk, x_one_box;
    int64_t late_cap;
    size_t smem;
    uint32_t tmem_cols;
};

size_t kmeans_tcf_state_bytes() { return sizeof(TcFusedState); }

// Columns of the score tile: the kernel instance's KMAX, so that nothing inside its tile loop depends on K.
static inline int tcf_npad(int K) { return K <= 16 ? 16 : K <= 32 ? 32 : 64; }

static inline int tcf_tile_rows(int d) { return d <= 128 ? BM : BM / 2; }

static size_t tcf_fixed_smem(int d, int K) {
    const int num_kb = (d + KBLK - 1) / KBLK;
    return (size_t)num_kb * tcf_npad(K) * 128 + sizeof(FusedShared);
}

static inline size_t tcf_stage_bytes(int d) { return (size_t)((d + KBLK - 1) / KBLK) * tcf_tile_rows(d) * 128; }

static inline int tcf_stages(const ep_ctx *ctx, int d, int K) {
    const size_t fixed = tcf_fixed_smem(d, K);
    if (fixed >= (size_t)ctx->smem_optin) return 0;
    return (int)std::min<size_t>(MAX_STAGES, ((size_t)ctx->smem_optin - fixed) / tcf_stage_bytes(d));
}

// Undecided rows the block holds in shared memory at a time once its tiles are done: what the ring leaves beside
// the block's sums and the fp32 centroids (K x d floats each), in whole rows, a multiple of the warps.
static inline int tcf_late_chunk(const ep_ctx *ctx, int d, int K) {
    const size_t ring = (size_t)tcf_stages(ctx, d, K) * tcf_stage_bytes(d), tables = 2 * (size_t)K * d * 4;
    if (ring <= tables) return 0;
    const size_t rows = (ring - tables) / ((size_t)d * 4);
    return (int)std::min<size_t>(MAX_LATE_CHUNK, rows / LATE_WARPS * LATE_WARPS);
}

bool kmeans_tcf_shape_ok(const ep_ctx *ctx, int d, int K) {
    if (d < KBLK || d > MAX_KB * KBLK || K < 1 || K > MAX_K) return false;
    if (d > 128 && K > 32) return false;   // the kernel instances for 64-row tiles stop at 32 columns
    return tcf_stages(ctx, d, K) >= 2 && tcf_late_chunk(ctx, d, K) >= LATE_WARPS;
}

int kmeans_tcf_grid(const ep_ctx *ctx, int64_t N, int d) {
    return (int)std::max<int64_t>(1, std::min<int64_t>(ctx->sm_count, ceil_div(N, tcf_tile_rows(d))));
}

// Entries of one screen warp's list of undecided rows: every row it can ever see.
int64_t kmeans_tcf_late_cap(const ep_ctx *ctx, int64_t N, int d) {
    return ceil_div(ceil_div(N, tcf_tile_rows(d)), kmeans_tcf_grid(ctx, N, d)) * 32;
}

// rownorm[i] = (|x_i|, |x_i - trunc_tf32(x_i)|): what the error bound of both tensor-core paths needs of a row.
int kmeans_row_norms(ep_ctx *ctx, const float *emb, int64_t N, int d, float2 *rownorm, cudaStream_t stream) {
    Timed tm(ctx, stream, EP_TIMER_KMEANS_UPDATE);
    row_norms<<<(int)std::min<int64_t>((int64_t)ctx->sm_count * 16, ceil_div(N, 8)), 256, 0, stream>>>(emb, N, d, rownorm);
    tm.end(1);
    EP_CUDA(ctx, cudaGetLastError());
    return EP_OK;
}

int kmeans_tcf_prepare(ep_ctx *ctx, const float *emb, int64_t N, int d, int K, const float *ct, TcFusedState *st) {
    st->npad = tcf_npad(K);
    st->num_kb = (d + KBLK - 1) / KBLK;
    st->stages = tcf_stages(ctx, d, K);
    st->smem = tcf_fixed_smem(d, K) + (size_t)st->stages * tcf_stage_bytes(d);
    st->late_chunk = tcf_late_chunk(ctx, d, K);
    st->grid = kmeans_tcf_grid(ctx, N, d);
    st->late_cap = kmeans_tcf_late_cap(ctx, N, d);
    uint32_t cols = 32;
    while (cols < 2u * (uint32_t)st->npad) cols <<= 1;
    st->tmem_cols = cols;
    // one box per tile where the rows are whole k-blocks; else (and should the driver refuse the view) a box per k-block
    st->x_one_box = (d % KBLK == 0 && tc_encode_rowtile_map(&st->map_x, emb, N, d, tcf_tile_rows(d))) ? 1 : 0;
    if ((!st->x_one_box && !tc_encode_kblock_map(&st->map_x, emb, N, d, tcf_tile_rows(d))) ||
        !tc_encode_kblock_map(&st->map_c, ct, K, d, st->npad))
        return fail(ctx, EP_ERR_CUDA, "cuTensorMapEncodeTiled failed for N=%lld d=%d K=%d", (long long)N, d, K);
    return EP_OK;
}

template <int KMAX, int VPL>
static int tcf_launch(ep_ctx *ctx, const TcFusedState &st, const float *emb, float *centroids, float *cn, float *ct, float *clo,
                      const float2 *rownorm, int64_t N, int d, int K, int32_t *assign, float *psum, int *pcnt,
                      int4 *late_list, int T, int update_here, int use_prev0, int keep_centroids, double *objterm,
                      double *objective, const double *x2part, int x2n, unsigned *grid_bar, cudaStream_t stream) {
    auto kern = update_here ? kmeans_tc_fused<KMAX, VPL, true> : kmeans_tc_fused<KMAX, VPL, false>;
    EP_CUDA(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)st.smem));
    unsigned long long *counters =
        ctx->opt_profile ? reinterpret_cast<unsigned long long *>(ctx->d_status + EP_COUNTER_WORD0) : nullptr;
    if (update_here) EP_CUDA(ctx, cudaMemsetAsync(grid_bar, 0, sizeof(unsigned), stream));
    Timed tm(ctx, stream, EP_TIMER_KMEANS_ASSIGN);
    CUtensorMap map_x = st.map_x, map_c = st.map_c;
    int npad = st.npad, num_kb = st.num_kb, stages = st.stages, late_chunk = st.late_chunk;
    uint32_t idesc = umma_idesc_tf32_m128(st.npad), tmem_cols = st.tmem_cols, key_mask = ~IDX_MASK;
    int64_t late_cap = st.late_cap;
    int x_one_box = st.x_one_box;
    int *status = ctx->d_status;
    void *args[] = {&map_x, &map_c, &emb, &centroids, &cn, &ct, &clo, &rownorm, &N, &d, &K, &npad, &num_kb, &stages, &idesc,
                    &tmem_cols, &key_mask, &assign, &psum, &pcnt, &late_list, &late_cap, &late_chunk, &T, &update_here, &use_prev0,
                    &keep_centroids,
                    &objterm, &objective, &x2part, &x2n, &x_one_box, &grid_bar, &counters, &status};
    if (update_here)   // one block per SM, all resident together: they meet on a grid-wide barrier twice per iteration
        EP_CUDA(ctx, cudaLaunchCooperativeKernel(reinterpret_cast<void *>(kern), dim3(st.grid), dim3(THREADS), args, st.smem, stream));
    else
        EP_CUDA(ctx, cudaLaunchKernel(reinterpret_cast<void *>(kern), dim3(st.grid), dim3(THREADS), args, st.smem, stream));
    tm.end(1);
    EP_CUDA(ctx, cudaGetLastError());
    return EP_OK;
}

// update_here: all T Lloyd iterations (assignment, accumulation, centroid update, objective) in one launch; on return
// of the stream work assign = labels of the last iteration, centroids / cn / ct / clo = those after the last update.
// Otherwise one assignment + accumulation pass (T is taken as 1): block b leaves its sums in psum[b][K][d] and its counts
// in pcnt[b][K] for the caller's update kernel; use_prev0 = pcnt still holds the counts of the iteration before.
int kmeans_tcf_run(ep_ctx *ctx, const TcFusedState &st, const float *emb, float *centroids, float *cn, float *ct, float *clo,
                   const float2 *rownorm, int64_t N, int d, int K, int32_t *assign, float *psum, int *pcnt, void *late_list_ws,
                   int T, bool update_here, bool use_prev0, bool keep_centroids, double *objterm, double *objective,
                   const double *x2part, int x2n, unsigned *grid_bar, cudaStream_t stream) {
    int4 *late_list = static_cast<int4 *>(late_list_ws);
    const int vpl = d <= 128 ? 1 : 2;
    if (!update_here) T = 1;
#define EP_TCF(KM, V)                                                                                                        \
    tcf_launch<KM, V>(ctx, st, emb, centroids, cn, ct, clo, rownorm, N, d, K, assign, psum, pcnt, late_list, T,             \
                      update_here ? 1 : 0, use_prev0 ? 1 : 0, keep_centroids ? 1 : 0, objterm, objective, x2part, x2n, grid_bar, stream)
    return vpl == 2 ? (K <= 16 ? EP_TCF(16, 2) : EP_TCF(32, 2)) : K <= 16 ? EP_TCF(16, 1) : K <= 32 ? EP_TCF(32, 1) : EP_TCF(64, 1);
#undef EP_TCF
}

}  // namespace ep
