// Self-test of the bounded device wait.  Every wait inside the tensor-core kernels (on an mbarrier that a TMA copy,
// an MMA or another warp completes) goes through eptc::mbar_wait, which gives up after a number of clocks, raises the
// block's abort flag and lets the kernel report EP_ERR_TIMEOUT instead of hanging.  In the production kernels no
// wait ever runs out, so this one-block kernel makes one run out on purpose, in the only safe way: it waits, with a
// short limit, on a barrier that by construction receives no arrival.  Nothing faults, traps or spins without end.
#include "ep_common.cuh"
#include "tc_device.cuh"

namespace {

using namespace eptc;

// Warp 0 waits with the caller's limit and gives up; warp 1 waits on the same barrier with the library's ordinary
// limit (about 2 s) and must leave as soon as warp 0 has raised the abort flag, long before its own limit.
// out[0] = clocks warp 0 waited, out[1] = clocks warp 1 waited, out[2] = what the two waits returned (bit 0, bit 1).
__global__ void __launch_bounds__(64) wait_timeout_probe(long long limit, int *status, long long *out) {
    __shared__ uint64_t bar;
    __shared__ int abort_s;
    __shared__ int results;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_s = 0;
        results = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const long long t0 = clock64();
    const bool ok = threadIdx.x < 32 ? mbar_wait(&bar, 0u, &abort_s, limit) : mbar_wait(&bar, 0u, &abort_s);
    const long long waited = clock64() - t0;
    if ((threadIdx.x & 31) == 0) {
        out[threadIdx.x >> 5] = waited;
        if (ok) atomicOr(&results, 1 << (threadIdx.x >> 5));
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        out[2] = results;
        if (abort_s) ep_raise(status, EP_ERR_TIMEOUT);
        asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(smem_u32(&bar)) : "memory");
    }
}

}  // namespace

extern "C" int ep_selftest_wait_timeout(ep_ctx *ctx, int64_t limit_clocks, int64_t *waited /* [dev] 3 x int64 */,
                                        void *cuda_stream) {
    if (!ctx) return EP_ERR_INVALID_ARG;
    if (!waited || !ep::aligned(waited, 8)) return ep::fail(ctx, EP_ERR_INVALID_ARG, "null or misaligned pointer");
    if (limit_clocks < 1000 || limit_clocks > 200000000)
        return ep::fail(ctx, EP_ERR_INVALID_ARG, "limit_clocks must lie in [1e3, 2e8] (at most about 0.1 s)");
    ep::DeviceGuard g(ctx->device);
    wait_timeout_probe<<<1, 64, 0, static_cast<cudaStream_t>(cuda_stream)>>>((long long)limit_clocks, ctx->d_status,
                                                                             reinterpret_cast<long long *>(waited));
    ctx->launches += 1;
    EP_CUDA(ctx, cudaGetLastError());
    return EP_OK;
}
