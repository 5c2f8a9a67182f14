// Partition-ordered vertex permutation (Section 4.5.1): a stable counting sort of the vertex ids by label, done as
// least-significant-digit passes over digits of 4, 6 or 8 bits (one pass for K <= 256, two 6-bit passes for K = 4096).
//
// One launch per pass.  The blocks of a pass, one of 1024 threads per SM, are all resident at once (a cooperative
// launch) and each owns a contiguous run of tiles of the key array:
//   1. the block counts the digits of its run in shared memory and publishes the counts, one row per block;
//   2. one grid-wide barrier (a counter every block increments, then polls with a time limit);
//   3. from the rows of all blocks every block derives, on its own, where each digit's keys of ITS run start in
//      the output (the digits' totals scanned, plus the counts of the blocks before it);
//   4. the block scatters its run tile by tile, keeping the running output position of every digit in shared memory.
//      Inside a tile a key's rank among equal digits is (keys of lower warps) + (earlier keys of its warp), found with
//      one vote per digit bit, which is exactly its original order; the tile is staged in sorted order in shared
//      memory so that the global writes of one digit leave as contiguous runs.
// Integer work only: exactly one output is correct and it does not depend on the schedule.
#include "ep_common.cuh"

#include <algorithm>
#include <mutex>

namespace {

constexpr int SORT_THREADS = 1024;                              // one block per SM: the count matrix stays a few rows
constexpr int SORT_WARPS = SORT_THREADS / 32;
constexpr int SORT_ITEMS = 16;                                  // 32-key steps per warp per tile
constexpr int SORT_TILE = SORT_WARPS * 32 * SORT_ITEMS;         // 16384 keys per tile
constexpr int MAX_RADIX = 256;
constexpr int SORT_MAX_GRID = 512;                              // blocks the count matrix of a workspace has room for
constexpr long long GRID_WAIT_LIMIT_CLOCKS = 4000000000ll;      // ~2 s: far beyond any legitimate wait
constexpr unsigned FULL = 0xffffffffu;

struct PassArgs {
    const int32_t *keys_in;      // N keys
    const int32_t *vals_in;      // their values, or nullptr: the value of key i is i itself (first pass)
    int64_t N;
    int shift;                   // the pass sorts by (key >> shift) & (2^BITS - 1)
    int items;                   // 32-key steps per warp and tile (<= SORT_ITEMS): a tile is 1024 * items keys
    int tiles_per_block;
    int32_t *counts;             // [gridDim.x][2^BITS]: digit counts of every block's run
    unsigned *barrier;           // zero before the launch
    int32_t *keys_out;           // nullptr: keys are not needed afterwards (last pass)
    int32_t *vals_out;
    int32_t *inv_out;            // not nullptr: also inv_out[value] = destination (last pass)
    int label_limit;             // > 0: a key outside [0, label_limit) raises EP_ERR_BAD_INDEX (it is still sorted by
                                 // its digits, so nothing is read or written out of bounds)
    int *status;
};

// The lanes of the warp whose digit equals this lane's, from one vote per digit bit.  `valid` lanes only match valid
// lanes (the ragged last tile); PARTIAL = false skips that vote.
template <int BITS, bool PARTIAL>
__device__ __forceinline__ unsigned same_digit_lanes(int digit, bool valid) {
    unsigned peers = FULL;
    if (PARTIAL) {
        const unsigned v = __ballot_sync(FULL, valid);
        peers = valid ? v : ~v;
    }
#pragma unroll
    for (int b = 0; b < BITS; ++b) {
        const bool bit = (digit >> b) & 1;
        const unsigned v = __ballot_sync(FULL, bit);
        peers &= bit ? v : ~v;
    }
    return peers;
}

// Dynamic shared memory of a pass: the staged tile (values, digits, keys if they go on) and the per-warp counters.
template <int BITS, bool KEYS_OUT>
constexpr size_t pass_smem_bytes() {
    return (size_t)SORT_TILE * (KEYS_OUT ? 9 : 5) + (size_t)SORT_WARPS * (1 << BITS) * 4;
}

// FIXED: a.items == SORT_ITEMS (long inputs), known at compile time so that the 16 steps carry no test.
template <int BITS, bool KEYS_OUT, bool FIXED>
__global__ void __launch_bounds__(SORT_THREADS, 1) radix_pass(const PassArgs a) {
    constexpr int RADIX = 1 << BITS;
    constexpr int DMASK = RADIX - 1;
    constexpr int PARTS = SORT_THREADS / RADIX;  // threads that share one digit's column of the count matrix
    extern __shared__ __align__(16) int sort_smem[];
    int *sval = sort_smem;                                         // [SORT_TILE]
    int *skey = sval + SORT_TILE;                                  // [SORT_TILE] when KEYS_OUT
    int (*cnt)[RADIX] = reinterpret_cast<int (*)[RADIX]>(skey + (KEYS_OUT ? SORT_TILE : 0));   // [SORT_WARPS][RADIX]: per warp and
                                                 // digit: counts, then exclusive positions inside the tile
    uint8_t *sdig = reinterpret_cast<uint8_t *>(&cnt[SORT_WARPS][0]);   // [SORT_TILE]
    __shared__ int run[RADIX];                   // where the next key of each digit of this block's run goes
    __shared__ int delta[RADIX];                 // tile: output position - staged position, per digit
    __shared__ int wtot[SORT_WARPS];
    __shared__ int gave_up;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int items = FIXED ? SORT_ITEMS : a.items;
    const int tile_keys = SORT_WARPS * 32 * items;
    const int64_t ntiles = (a.N + tile_keys - 1) / tile_keys;
    const int64_t t0 = (int64_t)blockIdx.x * a.tiles_per_block;
    const int64_t t1 = min(ntiles, t0 + a.tiles_per_block);
    const int64_t k0 = t0 * tile_keys, k1 = min(a.N, t1 * tile_keys);

    // ---- 1. digit counts of this block's run
    for (int i = threadIdx.x; i < SORT_WARPS * RADIX; i += SORT_THREADS) (&cnt[0][0])[i] = 0;
    if (threadIdx.x == 0) gave_up = 0;
    __syncthreads();
    {
        bool bad = false;
        const bool vec = (reinterpret_cast<uintptr_t>(a.keys_in) & 15u) == 0;
        const int64_t kv = vec ? k0 + ((k1 - k0) & ~int64_t(3)) : k0;     // 16-byte loads up to here
        constexpr int AHEAD = 4;                                          // 16-byte loads in flight per thread
        for (int64_t i0 = k0 + (int64_t)threadIdx.x * 4; i0 < kv; i0 += (int64_t)SORT_THREADS * 4 * AHEAD) {
            int4 k4[AHEAD];
#pragma unroll
            for (int u = 0; u < AHEAD; ++u) {
                const int64_t i = i0 + (int64_t)u * SORT_THREADS * 4;
                k4[u] = i < kv ? __ldg(reinterpret_cast<const int4 *>(a.keys_in + i)) : make_int4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < AHEAD; ++u) {
                if (i0 + (int64_t)u * SORT_THREADS * 4 >= kv) break;
                const int kk[4] = {k4[u].x, k4[u].y, k4[u].z, k4[u].w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    bad |= a.label_limit > 0 && (unsigned)kk[j] >= (unsigned)a.label_limit;
                    atomicAdd(&cnt[warp][(kk[j] >> a.shift) & DMASK], 1);
                }
            }
        }
        for (int64_t i = kv + threadIdx.x; i < k1; i += SORT_THREADS) {
            const int key = a.keys_in[i];
            bad |= a.label_limit > 0 && (unsigned)key >= (unsigned)a.label_limit;
            atomicAdd(&cnt[warp][(key >> a.shift) & DMASK], 1);
        }
        if (bad) ep_raise(a.status, EP_ERR_BAD_INDEX);
    }
    __syncthreads();
    if (threadIdx.x < RADIX) {
        int c = 0;
#pragma unroll
        for (int w = 0; w < SORT_WARPS; ++w) c += cnt[w][threadIdx.x];
        a.counts[(size_t)blockIdx.x * RADIX + threadIdx.x] = c;
    }

    // ---- 2. every block's row is published: one barrier across the grid (all blocks are resident)
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(a.barrier, 1u);
        const long long t_start = clock64();
        for (unsigned spins = 0;; ++spins) {
            unsigned seen;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(a.barrier) : "memory");
            if (seen >= gridDim.x) break;
            if ((spins & 31u) == 31u && clock64() - t_start > GRID_WAIT_LIMIT_CLOCKS) {
                gave_up = 1;
                break;
            }
            __nanosleep(100);
        }
    }
    __syncthreads();
    if (gave_up) {
        if (threadIdx.x == 0) ep_raise(a.status, EP_ERR_TIMEOUT);
        return;
    }

    // ---- 3. where this block's keys of each digit start: totals of the lower digits + counts of the lower blocks.
    // PARTS threads share a digit's column, each adding every PARTS-th row; the partial sums meet in shared memory.
    {
        const int dg = threadIdx.x & DMASK, part = threadIdx.x >> BITS;
        int below = 0, total = 0;
        const int32_t *col = a.counts + dg;
#pragma unroll 8
        for (int b = part; b < (int)gridDim.x; b += PARTS) {
            const int v = __ldcg(col + (size_t)b * RADIX);
            below += b < (int)blockIdx.x ? v : 0;
            total += v;
        }
        int *pb = sval, *pt = sval + SORT_THREADS;            // PARTS * RADIX = SORT_THREADS values each; no tile is staged yet
        pb[threadIdx.x] = below;
        pt[threadIdx.x] = total;
        __syncthreads();
        below = total = 0;
        if (threadIdx.x < RADIX) {
#pragma unroll
            for (int q = 0; q < PARTS; ++q) {
                below += pb[q * RADIX + threadIdx.x];
                total += pt[q * RADIX + threadIdx.x];
            }
        }
        int inc = total;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(FULL, inc, o);
            if (lane >= o) inc += t;
        }
        if (lane == 31) wtot[warp] = inc;
        __syncthreads();
        int add = 0;
        for (int w = 0; w < warp; ++w) add += wtot[w];
        if (threadIdx.x < RADIX) run[threadIdx.x] = add + inc - total + below;
        __syncthreads();
    }

    // ---- 4. stable scatter of the run, tile by tile
    const unsigned lt = (1u << lane) - 1u;
    for (int64_t tile = t0; tile < t1; ++tile) {
        const int64_t base = tile * tile_keys + (int64_t)warp * (32 * items);
        const bool full = (tile + 1) * tile_keys <= a.N;
        for (int i = threadIdx.x; i < SORT_WARPS * RADIX; i += SORT_THREADS) (&cnt[0][0])[i] = 0;
        int key[SORT_ITEMS], packed[SORT_ITEMS];         // packed = rank among the warp's equal digits << 8 | digit
#pragma unroll
        for (int i = 0; i < SORT_ITEMS; ++i) {
            const int64_t idx = base + i * 32 + lane;
            key[i] = (i < items && (full || idx < a.N)) ? a.keys_in[idx] : 0;
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < SORT_ITEMS; ++i) {
            if (i >= items) break;
            const bool ok = full || base + i * 32 + lane < a.N;
            const int dg = (key[i] >> a.shift) & DMASK;
            const unsigned peers = full ? same_digit_lanes<BITS, false>(dg, true) : same_digit_lanes<BITS, true>(dg, ok);
            // every lane reads its digit's running count in this warp; the lowest lane of each group of equal digits
            // then moves it on (one predicated store, no branch and no exchange between lanes)
            volatile int *slot = &cnt[warp][dg];
            const int before = *slot;
            __syncwarp();
            if (ok && (peers & lt) == 0u) *slot = before + __popc(peers);
            __syncwarp();
            packed[i] = ((before + __popc(peers & lt)) << 8) | dg;
        }
        __syncthreads();
        {   // per digit: the warps' counts become exclusive positions inside the tile's sorted order
            int tc = 0;
            if (threadIdx.x < RADIX) {
#pragma unroll
                for (int w = 0; w < SORT_WARPS; ++w) {
                    const int c = cnt[w][threadIdx.x];
                    cnt[w][threadIdx.x] = tc;
                    tc += c;
                }
            }
            int inc = tc;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(FULL, inc, o);
                if (lane >= o) inc += t;
            }
            if (lane == 31) wtot[warp] = inc;
            __syncthreads();
            int add = 0;
            for (int w = 0; w < warp; ++w) add += wtot[w];
            if (threadIdx.x < RADIX) {
                const int dstart = add + inc - tc;        // where this digit's run starts in the staged tile
#pragma unroll
                for (int w = 0; w < SORT_WARPS; ++w) cnt[w][threadIdx.x] += dstart;
                delta[threadIdx.x] = run[threadIdx.x] - dstart;
                run[threadIdx.x] += tc;
            }
        }
        __syncthreads();
        // stage the tile in sorted order, so that the global writes below go out as contiguous runs per digit
#pragma unroll
        for (int i = 0; i < SORT_ITEMS; ++i) {
            const int64_t idx = base + i * 32 + lane;
            if (i < items && (full || idx < a.N)) {
                const int dg = packed[i] & 255;
                const int lp = cnt[warp][dg] + (packed[i] >> 8);
                const int val = a.vals_in ? a.vals_in[idx] : (int)idx;
                if (!EP_INDEX_OK(lp, tile_keys, a.status)) continue;
                sval[lp] = val;
                sdig[lp] = (uint8_t)dg;
                if (KEYS_OUT) skey[lp] = key[i];
                if (a.inv_out && EP_INDEX_OK(val, a.N, a.status) && EP_INDEX_OK(lp + delta[dg], a.N, a.status))
                    a.inv_out[val] = lp + delta[dg];
            }
        }
        __syncthreads();
        const int ntile = (int)min((int64_t)tile_keys, a.N - tile * tile_keys);
        for (int q = threadIdx.x; q < ntile; q += SORT_THREADS) {
            const int dst = q + delta[sdig[q]];
            if (!EP_INDEX_OK(dst, a.N, a.status)) continue;
            a.vals_out[dst] = sval[q];
            if (KEYS_OUT) a.keys_out[dst] = skey[q];
        }
        __syncthreads();                                 // the next tile overwrites the counters and the staged tile
    }
}

// Digit width of the passes for K labels: as few passes as 8-bit digits allow, each as narrow as that permits.
struct PassPlan {
    int passes, bits;
};

PassPlan plan_passes(int K) {
    int total = 0;
    while ((int64_t(1) << total) < K) ++total;
    total = std::max(total, 1);
    const int passes = (total + 7) / 8;
    const int per = (total + passes - 1) / passes;
    return {passes, per <= 4 ? 4 : per <= 6 ? 6 : 8};
}

typedef void (*PassKernel)(const PassArgs);

struct PassLaunch {
    PassKernel kern;
    size_t smem;
};

template <int BITS>
PassLaunch pass_kernel_of(bool keys_out, bool fixed) {
    if (keys_out)
        return fixed ? PassLaunch{radix_pass<BITS, true, true>, pass_smem_bytes<BITS, true>()}
                     : PassLaunch{radix_pass<BITS, true, false>, pass_smem_bytes<BITS, true>()};
    return fixed ? PassLaunch{radix_pass<BITS, false, true>, pass_smem_bytes<BITS, false>()}
                 : PassLaunch{radix_pass<BITS, false, false>, pass_smem_bytes<BITS, false>()};
}

PassLaunch pass_kernel(int bits, bool keys_out, bool fixed) {
    if (bits == 4) return pass_kernel_of<4>(keys_out, fixed);
    if (bits == 6) return pass_kernel_of<6>(keys_out, fixed);
    return pass_kernel_of<8>(keys_out, fixed);
}

// One pass on the stream: the grid-barrier word cleared, then the cooperative launch of one block per SM.
cudaError_t launch_pass(int bits, bool keys_out, int sm_count, int max_grid, PassArgs args, cudaStream_t stream) {
    // Tiles as large as they come (16 steps per warp) when every block has several; otherwise the steps per tile are
    // chosen so that the keys spread evenly over one block per SM in as few tiles as possible.
    const int blocks = std::max(1, std::min(sm_count, max_grid));
    const int64_t per_block = (args.N + blocks - 1) / blocks;                             // keys per block, evenly
    const int64_t tiles_each = std::max<int64_t>(1, (per_block + SORT_TILE - 1) / SORT_TILE);
    const int64_t keys_per_tile = (per_block + tiles_each - 1) / tiles_each;
    args.items = (int)std::min<int64_t>(SORT_ITEMS, std::max<int64_t>(1, (keys_per_tile + SORT_WARPS * 32 - 1) / (SORT_WARPS * 32)));
    const PassLaunch pl = pass_kernel(bits, keys_out, args.items == SORT_ITEMS);
    cudaError_t e = cudaFuncSetAttribute(pl.kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem);
    if (e != cudaSuccess) return e;
    const int64_t tile_keys = (int64_t)SORT_WARPS * 32 * args.items;
    const int64_t ntiles = (args.N + tile_keys - 1) / tile_keys;
    int grid = (int)std::max<int64_t>(1, std::min<int64_t>(blocks, ntiles));
    args.tiles_per_block = (int)((ntiles + grid - 1) / grid);
    grid = (int)((ntiles + args.tiles_per_block - 1) / args.tiles_per_block);
    e = cudaMemsetAsync(args.barrier, 0, sizeof(unsigned), stream);
    if (e != cudaSuccess) return e;
    void *params[] = {&args};
    return cudaLaunchCooperativeKernel(reinterpret_cast<void *>(pl.kern), dim3(grid), dim3(SORT_THREADS), params, pl.smem, stream);
}

}  // namespace

namespace ep {

struct SortBuffers {
    int32_t *counts;
    unsigned *barrier;
    int32_t *keys[2], *vals[2];
};

static size_t sort_layout(int64_t N, int K, void *ws, SortBuffers *out) {
    Arena a(ws);
    SortBuffers b{};
    b.counts = a.take<int32_t>((size_t)SORT_MAX_GRID * MAX_RADIX);
    b.barrier = a.take<unsigned>(64);
    const int passes = plan_passes(K).passes;
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
    const PassPlan plan = plan_passes(K);
    const int32_t *kin = assign, *vin = nullptr;
    const int saved_profile = ctx->opt_profile;
    if (!timed) ctx->opt_profile = 0;
    Timed tm(ctx, stream, EP_TIMER_REORDER);
    ctx->opt_profile = saved_profile;
    for (int p = 0; p < plan.passes; ++p) {
        const bool last = (p == plan.passes - 1);
        PassArgs args{};
        args.keys_in = kin;
        args.vals_in = vin;
        args.N = N;
        args.shift = plan.bits * p;
        args.counts = b.counts;
        args.barrier = b.barrier;
        args.keys_out = last ? nullptr : b.keys[p & 1];
        args.vals_out = last ? perm : b.vals[p & 1];
        args.inv_out = last ? inv_perm : nullptr;
        args.label_limit = p == 0 ? K : 0;
        args.status = ctx->d_status;
        EP_CUDA(ctx, launch_pass(plan.bits, !last, ctx->sm_count, SORT_MAX_GRID, args, stream));
        kin = args.keys_out;
        vin = args.vals_out;
    }
    tm.end(plan.passes);
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
constexpr int STATIC_MAX_GRID = 512;                                         // rows of digit counts the array holds
constexpr int64_t STATIC_HEAD = 64;                                          // status word and barrier word, padded to 256 bytes
constexpr int64_t STATIC_WORDS = STATIC_HEAD + (int64_t)STATIC_MAX_GRID * MAX_RADIX;
static_assert(STATIC_MAX_K <= MAX_RADIX, "the static variant is the one-pass sort");

// About 0.5 MB in every GPU that loads the library, from load until the process exits.
static __device__ __align__(256) int32_t g_static_scratch[STATIC_WORDS];

}  // namespace

extern "C" int ep_reorder_static(const int32_t *assign, int64_t N, int32_t K, int32_t *perm, int32_t *inv_perm,
                                 int32_t *device_status, void *cuda_stream) {
    if (!assign || !perm) return EP_ERR_INVALID_ARG;
    if (!ep::aligned(assign, 4) || !ep::aligned(perm, 4) || (inv_perm && !ep::aligned(inv_perm, 4)) ||
        (device_status && !ep::aligned(device_status, 4)))
        return EP_ERR_INVALID_ARG;
    if (N < 1 || K < 1) return EP_ERR_INVALID_ARG;
    if (N > STATIC_MAX_N || K > STATIC_MAX_K) return EP_ERR_UNSUPPORTED;   // beyond the built-in scratch

    int dev = -1, sm_count = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return EP_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sm_count < 1) return EP_ERR_CUDA;
    // g_static_scratch names a host-side handle here, not device memory: the address a kernel may use has to be
    // asked for while the device it is wanted on is current.  Asked on every call (it allocates nothing once the
    // library's code is loaded on the device), so no cached address can outlive a reset of the device.
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return EP_ERR_CUDA;
    int32_t *base = static_cast<int32_t *>(p);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int *status = device_status ? device_status : base;   // the array's first word when the caller wants none

    // The array still holds the previous call's counts.  The status word and the barrier word are the only parts
    // read before they are written; every count this call reads is rewritten by its own kernel first.
    if (cudaMemsetAsync(status, 0, sizeof(int), stream) != cudaSuccess) return EP_ERR_CUDA;
    PassArgs args{};
    args.keys_in = assign;
    args.vals_in = nullptr;
    args.N = N;
    args.shift = 0;
    args.counts = base + STATIC_HEAD;
    args.barrier = reinterpret_cast<unsigned *>(base + 1);
    args.keys_out = nullptr;
    args.vals_out = perm;
    args.inv_out = inv_perm;
    args.label_limit = K;
    args.status = status;
    if (launch_pass(plan_passes(K).bits, false, sm_count, STATIC_MAX_GRID, args, stream) != cudaSuccess) {
        cudaGetLastError();
        return EP_ERR_CUDA;
    }
    return EP_OK;
}
