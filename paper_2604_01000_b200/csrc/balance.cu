// Migration policy M(P, S, C) (Algorithm 4: random migration in proportion to free capacity) and the balancing
// loop of Algorithm 3 that applies it to one vertex set until no partition is above its capacity.
//
// One application, all on the device:
//   loads     L_i = |{v in S : P(v) = i}| (block-local counts, then integer atomics);
//   plan      one block: m_i = max(L_i - C, 0), the free capacity of the underloaded partitions laid end to end
//             (cum_j), F, and where each partition's vertices start once S is sorted by partition;
//   order     S sorted by (partition, degree, vertex id) with the stable radix sort of reorder.cu over the key
//             P(v) (D + 1) + deg(v), D the caller's bound on the degree; vertices outside S go last;
//   move      vertex v of an overloaded partition i moves iff its position inside the partition's run is below
//             m_i, i.e. it is among the m_i smallest degrees (equal degrees: lower id first); it goes to the
//             partition j whose stretch of the free capacity holds t = floor(rand_words[v] F / 2^32).
// Random words are an input: nothing here draws numbers, and only integers are compared, so exactly one
// result is correct.
#include "ep_common.cuh"

#include <algorithm>

namespace {

constexpr int BAL_MAX_K = 1024;

// state[0] = sum of m_i (vertices to move), state[1] = F, state[2] = vertices moved or -1 (no free capacity)
constexpr int BAL_STATE_WORDS = 4;

template <typename RowT>
__global__ void __launch_bounds__(256) balance_loads(const RowT *__restrict__ rowptr, const int32_t *__restrict__ assign,
                                                     const uint8_t *__restrict__ member, int64_t N, int K,
                                                     long long max_degree, unsigned long long *load, int *status) {
    __shared__ unsigned int local[BAL_MAX_K];
    for (int k = threadIdx.x; k < K; k += blockDim.x) local[k] = 0u;
    __syncthreads();
    unsigned bad = 0;
    for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < N; v += (int64_t)gridDim.x * blockDim.x) {
        if (member && !member[v]) continue;
        const int a = assign[v];
        const long long deg = (long long)rowptr[v + 1] - (long long)rowptr[v];
        if ((unsigned)a >= (unsigned)K || deg < 0 || deg > max_degree) {
            bad = 1;                                        // such a vertex is left where it is and not counted
            continue;
        }
        atomicAdd(&local[a], 1u);
    }
    if (bad) ep_raise(status, EP_ERR_BAD_INDEX);
    __syncthreads();
    for (int k = threadIdx.x; k < K; k += blockDim.x)
        if (local[k]) atomicAdd(&load[k], (unsigned long long)local[k]);
}

// One block.  over[i] = m_i; cum[j] = free capacity of the underloaded partitions up to and including j;
// start[i] = number of vertices of S in partitions below i.
__global__ void __launch_bounds__(32) balance_plan(const unsigned long long *__restrict__ load, int K, long long capacity,
                                                   long long *over, long long *cum, long long *start, long long *state) {
    if (threadIdx.x != 0) return;
    long long F = 0, total = 0, run = 0;
    for (int j = 0; j < K; ++j) {
        const long long L = (long long)load[j];
        over[j] = L > capacity ? L - capacity : 0;
        total += over[j];
        if (L < capacity) F += capacity - L;
        cum[j] = F;
        start[j] = run;
        run += L;
    }
    state[0] = total;
    state[1] = F;
    state[2] = (total > 0 && F == 0) ? -1 : total;
    state[3] = 0;
}

template <typename RowT>
__global__ void __launch_bounds__(256) balance_keys(const RowT *__restrict__ rowptr, const int32_t *__restrict__ assign,
                                                    const uint8_t *__restrict__ member, int64_t N, int K,
                                                    long long max_degree, int32_t *__restrict__ key) {
    const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= N) return;
    const int a = assign[v];
    const long long deg = (long long)rowptr[v + 1] - (long long)rowptr[v];
    const bool counted = (!member || member[v]) && (unsigned)a < (unsigned)K && deg >= 0 && deg <= max_degree;
    key[v] = counted ? (int32_t)((long long)a * (max_degree + 1) + deg) : (int32_t)((long long)K * (max_degree + 1));
}

__global__ void __launch_bounds__(256) balance_move(int32_t *__restrict__ assign, const int32_t *__restrict__ key,
                                                    const int32_t *__restrict__ position, int64_t N, int K,
                                                    long long max_degree, const uint32_t *__restrict__ rand_words,
                                                    const long long *__restrict__ over, const long long *__restrict__ cum,
                                                    const long long *__restrict__ start, const long long *__restrict__ state) {
    __shared__ long long over_s[BAL_MAX_K], cum_s[BAL_MAX_K], start_s[BAL_MAX_K];
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
        over_s[k] = over[k];
        cum_s[k] = cum[k];
        start_s[k] = start[k];
    }
    __syncthreads();
    const long long F = state[1];
    if (state[2] <= 0) return;                               // nothing to move, or nowhere to move it
    const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= N) return;
    const long long kv = key[v];
    const int a = (int)(kv / (max_degree + 1));              // K for the vertices that are not counted
    if (a >= K || over_s[a] == 0) return;
    if ((long long)position[v] - start_s[a] >= over_s[a]) return;
    const unsigned long long t = ((unsigned long long)rand_words[v] * (unsigned long long)F) >> 32;
    int lo = 0, hi = K - 1;                                  // first partition whose cumulative capacity exceeds t
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if ((unsigned long long)cum_s[mid] > t)
            hi = mid;
        else
            lo = mid + 1;
    }
    assign[v] = lo;
}

}  // namespace

namespace ep {

struct BalanceBuffers {
    unsigned long long *load;
    long long *over, *cum, *start, *state;
    int32_t *key, *order, *position;
    void *sort_ws;
};

static int64_t balance_keys_total(int K, int64_t max_degree) { return (int64_t)K * (max_degree + 1) + 1; }

bool balance_shape_ok(int64_t N, int K, int64_t max_degree) {
    return N >= 1 && N < (int64_t(1) << 31) && K >= 1 && K <= BAL_MAX_K && max_degree >= 0 && max_degree < (int64_t(1) << 31) &&
           balance_keys_total(K, max_degree) <= (int64_t(1) << 30);
}

static size_t balance_layout(int64_t N, int K, int64_t max_degree, void *ws, BalanceBuffers *out) {
    Arena a(ws);
    BalanceBuffers b{};
    b.load = a.take<unsigned long long>(K);
    b.over = a.take<long long>(K);
    b.cum = a.take<long long>(K);
    b.start = a.take<long long>(K);
    b.state = a.take<long long>(BAL_STATE_WORDS);
    b.key = a.take<int32_t>(N);
    b.order = a.take<int32_t>(N);
    b.position = a.take<int32_t>(N);
    b.sort_ws = a.take<char>(reorder_workspace_bytes(N, (int)balance_keys_total(K, max_degree)));
    if (out) *out = b;
    return a.used;
}

size_t balance_workspace_bytes(int64_t N, int K, int64_t max_degree) {
    return balance_layout(N, K, max_degree, nullptr, nullptr);
}

template <typename RowT>
static int migrate_launch(ep_ctx *ctx, const RowT *rowptr, int64_t N, int K, const uint8_t *member, int64_t capacity,
                          int64_t max_degree, const uint32_t *rand_words, int32_t *assign, long long *state_out,
                          const BalanceBuffers &b, cudaStream_t stream) {
    Timed tm(ctx, stream, EP_TIMER_BALANCE);
    EP_CUDA(ctx, cudaMemsetAsync(b.load, 0, sizeof(unsigned long long) * K, stream));
    const int lgrid = (int)std::max<int64_t>(1, std::min<int64_t>((int64_t)ctx->sm_count * 4, ceil_div(N, 256)));
    balance_loads<RowT><<<lgrid, 256, 0, stream>>>(rowptr, assign, member, N, K, (long long)max_degree, b.load, ctx->d_status);
    balance_plan<<<1, 32, 0, stream>>>(b.load, K, (long long)capacity, b.over, b.cum, b.start, b.state);
    int kernels = 2;
    if (rand_words) {
        const unsigned nblk = (unsigned)ceil_div(N, 256);
        balance_keys<RowT><<<nblk, 256, 0, stream>>>(rowptr, assign, member, N, K, (long long)max_degree, b.key);
        tm.end(kernels + 1);
        kernels = 0;
        int rc = reorder_run(ctx, b.key, N, (int)balance_keys_total(K, max_degree), b.order, b.position, b.sort_ws, stream,
                             /*timed=*/false);
        if (rc != EP_OK) return rc;
        Timed tm2(ctx, stream, EP_TIMER_BALANCE);
        balance_move<<<nblk, 256, 0, stream>>>(assign, b.key, b.position, N, K, (long long)max_degree, rand_words, b.over,
                                              b.cum, b.start, b.state);
        tm2.end(1);
    } else {
        tm.end(kernels);
    }
    if (state_out)
        EP_CUDA(ctx, cudaMemcpyAsync(state_out, b.state, sizeof(long long) * BAL_STATE_WORDS, cudaMemcpyDeviceToDevice, stream));
    EP_CUDA(ctx, cudaGetLastError());
    return EP_OK;
}

int migrate_run(ep_ctx *ctx, const void *rowptr, bool rowptr64, int64_t N, int K, const uint8_t *member, int64_t capacity,
                int64_t max_degree, const uint32_t *rand_words, int32_t *assign, long long *state_out, void *workspace,
                cudaStream_t stream) {
    BalanceBuffers b;
    balance_layout(N, K, max_degree, workspace, &b);
    if (rowptr64)
        return migrate_launch<int64_t>(ctx, static_cast<const int64_t *>(rowptr), N, K, member, capacity, max_degree,
                                       rand_words, assign, state_out, b, stream);
    return migrate_launch<int32_t>(ctx, static_cast<const int32_t *>(rowptr), N, K, member, capacity, max_degree, rand_words,
                                   assign, state_out, b, stream);
}

// The device copy of the last plan's state, for the host loop of ep_balance.
const long long *balance_state_ptr(int64_t N, int K, int64_t max_degree, void *workspace) {
    BalanceBuffers b;
    balance_layout(N, K, max_degree, workspace, &b);
    return b.state;
}

}  // namespace ep
