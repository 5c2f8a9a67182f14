// Partition-ordered vertex permutation (Section 4.5.1): a stable counting sort of the vertex ids
// by label, done as least-significant-digit passes over 8-bit digits (one pass for K <= 256).
// Each pass: per-tile digit histogram -> exclusive scan over (digit, tile) -> stable scatter.
#include "ep_common.cuh"

#include <algorithm>
#include <mutex>

namespace {

constexpr int RADIX = 256;
constexpr int SORT_WARPS = 8;
constexpr int SORT_ITEMS = 16;                                  // 32-element steps per warp per tile
constexpr int SORT_TILE = SORT_WARPS * 32 * SORT_ITEMS;         // 4096 keys per block
constexpr int SCAN_THREADS = 1024;
constexpr int SCAN_ITEMS = 4;
constexpr int SCAN_TILE = SCAN_THREADS * SCAN_ITEMS;
constexpr unsigned FULL = 0xffffffffu;

// hist[digit * ntiles + tile] = keys of this tile whose digit (key >> shift) & 255 equals `digit`.
// When label_limit > 0 (first pass) a key outside [0, label_limit) raises EP_ERR_BAD_INDEX; such a key is
// still sorted by its digits, so nothing is read or written out of bounds.
__global__ void __launch_bounds__(SORT_WARPS * 32) digit_histogram(const int32_t *__restrict__ keys, int64_t N,
                                                                    int shift, int ntiles, int32_t *hist,
                                                                    int label_limit, int *status) {
    __shared__ int cnt[RADIX];
    cnt[threadIdx.x] = 0;
    __syncthreads();
    const int64_t base = (int64_t)blockIdx.x * SORT_TILE;
    if (base + SORT_TILE <= N && (reinterpret_cast<uintptr_t>(keys) & 15u) == 0) {
        // a full tile of an aligned array: all of a thread's keys are on their way before the first is counted
        const int4 *src = reinterpret_cast<const int4 *>(keys + base);
        int4 k4[SORT_ITEMS / 4];
#pragma unroll
        for (int i = 0; i < SORT_ITEMS / 4; ++i) k4[i] = __ldg(src + i * (SORT_WARPS * 32) + threadIdx.x);
#pragma unroll
        for (int i = 0; i < SORT_ITEMS / 4; ++i) {
            const int kk[4] = {k4[i].x, k4[i].y, k4[i].z, k4[i].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (label_limit > 0 && (unsigned)kk[j] >= (unsigned)label_limit) ep_raise(status, EP_ERR_BAD_INDEX);
                atomicAdd(&cnt[(kk[j] >> shift) & (RADIX - 1)], 1);
            }
        }
    } else {
#pragma unroll 4
        for (int i = 0; i < SORT_ITEMS; ++i) {
            int64_t idx = base + i * (SORT_WARPS * 32) + threadIdx.x;
            if (idx < N) {
                const int key = keys[idx];
                if (label_limit > 0 && (unsigned)key >= (unsigned)label_limit) ep_raise(status, EP_ERR_BAD_INDEX);
                atomicAdd(&cnt[(key >> shift) & (RADIX - 1)], 1);
            }
        }
    }
    __syncthreads();
    hist[(size_t)threadIdx.x * ntiles + blockIdx.x] = cnt[threadIdx.x];
}

// Exclusive scan, level 1: each block scans SCAN_TILE int32 values in place and records its total.
__global__ void __launch_bounds__(SCAN_THREADS) scan_tiles(int32_t *data, int64_t n, int32_t *totals) {
    __shared__ int warp_sum[32];
    const int64_t base = (int64_t)blockIdx.x * SCAN_TILE + (int64_t)threadIdx.x * SCAN_ITEMS;
    int v[SCAN_ITEMS];
    int s = 0;
#pragma unroll
    for (int i = 0; i < SCAN_ITEMS; ++i) {
        v[i] = (base + i < n) ? data[base + i] : 0;
        s += v[i];
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = s;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(FULL, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) warp_sum[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        int w = warp_sum[lane];
        int winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(FULL, winc, o);
            if (lane >= o) winc += t;
        }
        warp_sum[lane] = winc - w;
        if (lane == 31) totals[blockIdx.x] = winc;
    }
    __syncthreads();
    int run = warp_sum[warp] + inc - s;
#pragma unroll
    for (int i = 0; i < SCAN_ITEMS; ++i) {
        if (base + i < n) data[base + i] = run;
        run += v[i];
    }
}

// Level 2: one block turns the tile totals into exclusive offsets (sequential over chunks of 1024).
__global__ void __launch_bounds__(SCAN_THREADS) scan_totals(int32_t *totals, int n) {
    __shared__ int warp_sum[32];
    __shared__ int carry_s;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int base = 0; base < n; base += SCAN_THREADS) {
        int i = base + threadIdx.x;
        int v = i < n ? totals[i] : 0;
        int inc = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(FULL, inc, o);
            if (lane >= o) inc += t;
        }
        if (lane == 31) warp_sum[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            int w = warp_sum[lane];
            int winc = w;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int t = __shfl_up_sync(FULL, winc, o);
                if (lane >= o) winc += t;
            }
            warp_sum[lane] = winc - w;
        }
        __syncthreads();
        int carry = carry_s;
        int excl = carry + warp_sum[warp] + inc - v;
        if (i < n) totals[i] = excl;
        __syncthreads();
        if (threadIdx.x == SCAN_THREADS - 1) carry_s = excl + v;
        __syncthreads();
    }
}

// Level 3: add each tile's offset.
__global__ void __launch_bounds__(SCAN_THREADS) scan_add(int32_t *data, int64_t n, const int32_t *__restrict__ totals) {
    const int add = totals[blockIdx.x];
    const int64_t base = (int64_t)blockIdx.x * SCAN_TILE + (int64_t)threadIdx.x * SCAN_ITEMS;
#pragma unroll
    for (int i = 0; i < SCAN_ITEMS; ++i)
        if (base + i < n) data[base + i] += add;
}

// Stable scatter of one pass.  Warp w of a block owns the contiguous keys [w*512, (w+1)*512) of the
// tile and walks them 32 at a time; a key's rank among equal digits is (keys of lower warps) +
// (earlier keys of this warp) + (lower lanes of this step), which is exactly its original order.
//   vals_in  == nullptr: the value of key i is i itself (first pass)
//   keys_out == nullptr: keys are not needed afterwards (last pass)
//   inv_out  != nullptr: also writes inv_out[value] = destination (last pass)
__global__ void __launch_bounds__(SORT_WARPS * 32, 4) digit_scatter(const int32_t *__restrict__ keys_in,
                                                                  const int32_t *__restrict__ vals_in, int64_t N,
                                                                  int shift, int ntiles,
                                                                  const int32_t *__restrict__ offsets,
                                                                  int32_t *__restrict__ keys_out,
                                                                  int32_t *__restrict__ vals_out,
                                                                  int32_t *__restrict__ inv_out) {
    __shared__ int cnt[SORT_WARPS][RADIX];
    __shared__ int gbase[RADIX], dstart[RADIX], wtot[SORT_WARPS];
    __shared__ int sval[SORT_TILE], skey[SORT_TILE];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < SORT_WARPS * RADIX; i += blockDim.x) (&cnt[0][0])[i] = 0;
    // this digit's place in the output: asked for now, needed only after the ranking (the tiles' offsets of one digit
    // lie ntiles words apart, so every thread's word is a cache line of its own and takes its time)
    const int my_gbase = __ldg(offsets + (size_t)threadIdx.x * ntiles + blockIdx.x);
    __syncthreads();

    const int64_t base = (int64_t)blockIdx.x * SORT_TILE + (int64_t)warp * (32 * SORT_ITEMS);
    int key[SORT_ITEMS], rank[SORT_ITEMS];
    const unsigned lt = (1u << lane) - 1u;
#pragma unroll
    for (int i = 0; i < SORT_ITEMS; ++i) {
        const int64_t idx = base + i * 32 + lane;
        const bool ok = idx < N;
        key[i] = ok ? keys_in[idx] : 0;
        const int dg = ok ? ((key[i] >> shift) & (RADIX - 1)) : (RADIX + lane);   // idle lanes match nobody
        const unsigned peers = __match_any_sync(FULL, dg);
        const int leader = __ffs(peers) - 1;
        int before = 0;
        if (ok && lane == leader) {
            before = cnt[warp][dg];
            cnt[warp][dg] = before + __popc(peers);
        }
        before = __shfl_sync(FULL, before, leader);
        rank[i] = before + __popc(peers & lt);
        __syncwarp();
    }
    gbase[threadIdx.x] = my_gbase;
    __syncthreads();
    {   // per digit: turn the warps' counts into exclusive offsets inside the tile, and the digits' totals
        // into the place where each digit's run starts in the tile's sorted order
        const int dg = threadIdx.x;
        int run = 0;
#pragma unroll
        for (int w = 0; w < SORT_WARPS; ++w) {
            int c = cnt[w][dg];
            cnt[w][dg] = run;
            run += c;
        }
        int inc = run;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(FULL, inc, o);
            if (lane >= o) inc += t;
        }
        if (lane == 31) wtot[warp] = inc;
        __syncthreads();
        int add = 0;
        for (int w = 0; w < warp; ++w) add += wtot[w];
        dstart[dg] = add + inc - run;
    }
    __syncthreads();
    // stage the tile in sorted order, so that the global writes below go out as contiguous runs per digit
#pragma unroll
    for (int i = 0; i < SORT_ITEMS; ++i) {
        const int64_t idx = base + i * 32 + lane;
        if (idx < N) {
            const int dg = (key[i] >> shift) & (RADIX - 1);
            const int within = cnt[warp][dg] + rank[i];
            const int val = vals_in ? vals_in[idx] : (int)idx;
            const int lp = dstart[dg] + within;
            sval[lp] = val;
            skey[lp] = key[i];
            if (inv_out) inv_out[val] = gbase[dg] + within;
        }
    }
    __syncthreads();
    const int ntile = (int)min((int64_t)SORT_TILE, N - (int64_t)blockIdx.x * SORT_TILE);
    for (int q = threadIdx.x; q < ntile; q += blockDim.x) {
        const int k = skey[q];
        const int dg = (k >> shift) & (RADIX - 1);
        const int dst = gbase[dg] + (q - dstart[dg]);
        vals_out[dst] = sval[q];
        if (keys_out) keys_out[dst] = k;
    }
}

int passes_for(int K) {
    int bits = 0;
    while ((int64_t(1) << bits) < K) ++bits;
    return std::max(1, (bits + 7) / 8);
}

}  // namespace

namespace ep {

struct SortBuffers {
    int32_t *hist, *totals, *keys[2], *vals[2];
};

static size_t sort_layout(int64_t N, int K, void *ws, SortBuffers *out) {
    Arena a(ws);
    SortBuffers b{};
    const int64_t ntiles = ceil_div(N, SORT_TILE);
    const int64_t nhist = ntiles * RADIX;
    b.hist = a.take<int32_t>(nhist);
    b.totals = a.take<int32_t>(ceil_div(nhist, SCAN_TILE));
    const int passes = passes_for(K);
    if (passes > 1) {
        b.keys[0] = a.take<int32_t>(N);
        b.vals[0] = a.take<int32_t>(N);
    }
    if (passes > 2) {
        b.keys[1] = a.take<int32_t>(N);
        b.vals[1] = a.take<int32_t>(N);
    }
    if (out) *out = b;
    return a.used;
}

size_t reorder_workspace_bytes(int64_t N, int K) { return sort_layout(N, K, nullptr, nullptr); }

int reorder_run(ep_ctx *ctx, const int32_t *assign, int64_t N, int K, int32_t *perm, int32_t *inv_perm, void *workspace,
                cudaStream_t stream, bool timed) {
    SortBuffers b;
    sort_layout(N, K, workspace, &b);
    const int ntiles = (int)ceil_div(N, SORT_TILE);
    const int64_t nhist = (int64_t)ntiles * RADIX;
    const int nscan = (int)ceil_div(nhist, SCAN_TILE);
    const int passes = passes_for(K);
    const int32_t *kin = assign, *vin = nullptr;
    const int saved_profile = ctx->opt_profile;
    if (!timed) ctx->opt_profile = 0;
    Timed tm(ctx, stream, EP_TIMER_REORDER);
    ctx->opt_profile = saved_profile;
    // four blocks of the scatter kernel per SM need most of the SM's memory as shared memory
    EP_CUDA(ctx, cudaFuncSetAttribute(digit_scatter, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared));
    for (int p = 0; p < passes; ++p) {
        const bool last = (p == passes - 1);
        int32_t *kout = last ? nullptr : b.keys[p & 1];
        int32_t *vout = last ? perm : b.vals[p & 1];
        digit_histogram<<<ntiles, SORT_WARPS * 32, 0, stream>>>(kin, N, 8 * p, ntiles, b.hist, p == 0 ? K : 0,
                                                               ctx->d_status);
        scan_tiles<<<nscan, SCAN_THREADS, 0, stream>>>(b.hist, nhist, b.totals);
        scan_totals<<<1, SCAN_THREADS, 0, stream>>>(b.totals, nscan);
        scan_add<<<nscan, SCAN_THREADS, 0, stream>>>(b.hist, nhist, b.totals);
        digit_scatter<<<ntiles, SORT_WARPS * 32, 0, stream>>>(kin, vin, N, 8 * p, ntiles, b.hist, kout, vout,
                                                             last ? inv_perm : nullptr);
        kin = kout;
        vin = vout;
    }
    tm.end(5 * passes);
    EP_CUDA(ctx, cudaGetLastError());
    return EP_OK;
}

}  // namespace ep

// ---------------------------------------------------------------------------------------------------
// ep_reorder_static: the single-pass sort above with its scratch in a device array owned by the
// library instead of a caller workspace, for callers that cannot obtain device memory themselves.
// ---------------------------------------------------------------------------------------------------
namespace {

constexpr int64_t STATIC_MAX_N = EP_REORDER_STATIC_MAX_N;
constexpr int STATIC_MAX_K = EP_REORDER_STATIC_MAX_K;
constexpr int64_t STATIC_TILES = (STATIC_MAX_N + SORT_TILE - 1) / SORT_TILE;
constexpr int64_t STATIC_HIST = STATIC_TILES * RADIX;                        // per-tile digit counts
constexpr int64_t STATIC_TOTALS = (STATIC_HIST + SCAN_TILE - 1) / SCAN_TILE; // one total per scan block
constexpr int64_t STATIC_HEAD = 64;                                          // status word, padded to 256 bytes
constexpr int64_t STATIC_WORDS = STATIC_HEAD + STATIC_HIST + (STATIC_TOTALS + 63) / 64 * 64;
static_assert(STATIC_MAX_K <= RADIX, "the static variant is the one-pass sort");

// About 1 MB in every GPU that loads the library, from load until the process exits.
static __device__ __align__(256) int32_t g_static_scratch[STATIC_WORDS];

constexpr int STATIC_MAX_DEVICES = 64;
int32_t *g_static_ptr[STATIC_MAX_DEVICES];   // device address of g_static_scratch on each device, once resolved
std::mutex g_static_mutex;

}  // namespace

extern "C" int ep_reorder_static(const int32_t *assign, int64_t N, int32_t K, int32_t *perm, int32_t *inv_perm,
                                 int32_t *device_status, void *cuda_stream) {
    if (!assign || !perm) return EP_ERR_INVALID_ARG;
    if (!ep::aligned(assign, 4) || !ep::aligned(perm, 4) || (inv_perm && !ep::aligned(inv_perm, 4)) ||
        (device_status && !ep::aligned(device_status, 4)))
        return EP_ERR_INVALID_ARG;
    if (N < 1 || K < 1) return EP_ERR_INVALID_ARG;
    if (N > STATIC_MAX_N || K > STATIC_MAX_K) return EP_ERR_UNSUPPORTED;   // beyond the built-in scratch

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return EP_ERR_CUDA;
    if (dev < 0 || dev >= STATIC_MAX_DEVICES) return EP_ERR_UNSUPPORTED;
    int32_t *base = nullptr;
    {
        // g_static_scratch names a host-side handle here, not device memory: the address a kernel may
        // use has to be asked for, once per device, while that device is current.
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_ptr[dev]) {
            void *p = nullptr;
            if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return EP_ERR_CUDA;
            g_static_ptr[dev] = static_cast<int32_t *>(p);
        }
        base = g_static_ptr[dev];
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int *status = device_status ? device_status : base;   // the array's first word when the caller wants none
    int32_t *hist = base + STATIC_HEAD;
    int32_t *totals = hist + STATIC_HIST;

    const int ntiles = (int)ep::ceil_div(N, SORT_TILE);
    const int64_t nhist = (int64_t)ntiles * RADIX;
    const int nscan = (int)ep::ceil_div(nhist, SCAN_TILE);
    // The array still holds the previous call's counts.  The status word is the only part read before
    // it is written; every histogram and total this call reads is rewritten by its own kernels first.
    if (cudaMemsetAsync(status, 0, sizeof(int), stream) != cudaSuccess) return EP_ERR_CUDA;
    digit_histogram<<<ntiles, SORT_WARPS * 32, 0, stream>>>(assign, N, 0, ntiles, hist, K, status);
    scan_tiles<<<nscan, SCAN_THREADS, 0, stream>>>(hist, nhist, totals);
    scan_totals<<<1, SCAN_THREADS, 0, stream>>>(totals, nscan);
    scan_add<<<nscan, SCAN_THREADS, 0, stream>>>(hist, nhist, totals);
    digit_scatter<<<ntiles, SORT_WARPS * 32, 0, stream>>>(assign, nullptr, N, 0, ntiles, hist, nullptr, perm, inv_perm);
    return cudaGetLastError() == cudaSuccess ? EP_OK : EP_ERR_CUDA;
}
