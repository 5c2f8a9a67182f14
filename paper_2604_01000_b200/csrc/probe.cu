// Yardsticks for the label gather of the edge-cut pass (Section 2.1.1, Eq. 1: one label lookup per stored entry).
// The pass streams the column ids at HBM speed; what binds it is the lookup of one small label per entry at a
// random vertex.  These kernels do nothing but that lookup (the column ids streamed the same way, one byte
// gathered per entry, the bytes summed), so that the edge-cut pass can be held against the rate at which this GPU
// serves such gathers at all:
//   gather_global   the byte table in global memory (L1 / L2), as the edge-cut pass reads it when the labels do
//                   not fit in shared memory;
//   gather_cluster  the byte table spread over the shared memory of a thread-block cluster, every lookup a
//                   ld.shared::cluster from the block that holds the vertex's slice;
//   gather_texture  the byte table in global memory, read through a texture object (the texture units' own
//                   address and tag path instead of the load/store unit's).
#include "ep_common.cuh"

#include <algorithm>

namespace {

constexpr int PB_THREADS = 256;
constexpr int PB_VEC = 8;
constexpr int PB_TILE = PB_THREADS * PB_VEC * 4;      // entries per block step, as in the edge-cut pass
constexpr int PC_THREADS = 1024;
constexpr int PC_TILE = PC_THREADS * PB_VEC * 4;
constexpr unsigned FULL = 0xffffffffu;

__device__ __forceinline__ void block_add(unsigned long long v, unsigned long long *out) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(FULL, v, o);
    if ((threadIdx.x & 31) == 0 && v) atomicAdd(out, v);
}

__global__ void __launch_bounds__(PB_THREADS, 4) gather_global(const int32_t *__restrict__ colidx, int64_t nnz,
                                                             const uint8_t *__restrict__ table, int64_t N,
                                                             unsigned long long *sum) {
    const int64_t ntiles = (nnz + PB_TILE - 1) / PB_TILE;
    unsigned long long mine = 0ull;
    for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const int64_t e0 = tile * PB_TILE;
        const int ne = (int)min((int64_t)PB_TILE, nnz - e0);
        int4 c[PB_VEC];
#pragma unroll
        for (int i = 0; i < PB_VEC; ++i) {
            const int q = (i * PB_THREADS + threadIdx.x) * 4;
            if (q + 3 < ne) {
                c[i] = __ldcs(reinterpret_cast<const int4 *>(colidx + e0) + (q >> 2));
            } else {
                c[i].x = q + 0 < ne ? colidx[e0 + q + 0] : -1;
                c[i].y = q + 1 < ne ? colidx[e0 + q + 1] : -1;
                c[i].z = q + 2 < ne ? colidx[e0 + q + 2] : -1;
                c[i].w = -1;
            }
        }
        unsigned t = 0;
#pragma unroll
        for (int i = 0; i < PB_VEC; ++i) {
            const int cols[4] = {c[i].x, c[i].y, c[i].z, c[i].w};
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if ((unsigned)cols[j] < (unsigned)N) t += __ldg(table + cols[j]);
        }
        mine += t;
    }
    block_add(mine, sum);
}

__global__ void __launch_bounds__(PB_THREADS, 4) gather_texture(const int32_t *__restrict__ colidx, int64_t nnz,
                                                              cudaTextureObject_t table, int64_t N,
                                                              unsigned long long *sum) {
    const int64_t ntiles = (nnz + PB_TILE - 1) / PB_TILE;
    unsigned long long mine = 0ull;
    for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const int64_t e0 = tile * PB_TILE;
        const int ne = (int)min((int64_t)PB_TILE, nnz - e0);
        int4 c[PB_VEC];
#pragma unroll
        for (int i = 0; i < PB_VEC; ++i) {
            const int q = (i * PB_THREADS + threadIdx.x) * 4;
            if (q + 3 < ne) {
                c[i] = __ldcs(reinterpret_cast<const int4 *>(colidx + e0) + (q >> 2));
            } else {
                c[i].x = q + 0 < ne ? colidx[e0 + q + 0] : -1;
                c[i].y = q + 1 < ne ? colidx[e0 + q + 1] : -1;
                c[i].z = q + 2 < ne ? colidx[e0 + q + 2] : -1;
                c[i].w = -1;
            }
        }
        unsigned t = 0;
#pragma unroll
        for (int i = 0; i < PB_VEC; ++i) {
            const int cols[4] = {c[i].x, c[i].y, c[i].z, c[i].w};
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if ((unsigned)cols[j] < (unsigned)N) t += tex1Dfetch<unsigned char>(table, cols[j]);
        }
        mine += t;
    }
    block_add(mine, sum);
}

// Block r of a cluster holds table bytes [r * slice, (r + 1) * slice) in its shared memory.  magic = ceil(2^32 / slice).
__global__ void __launch_bounds__(PC_THREADS, 1) gather_cluster(const int32_t *__restrict__ colidx, int64_t nnz,
                                                              const uint8_t *__restrict__ table, int64_t N,
                                                              uint32_t slice, uint32_t magic, int csize,
                                                              unsigned long long *sum) {
    extern __shared__ __align__(16) uint8_t tab[];
    uint32_t rank;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    const int64_t lo = (int64_t)rank * slice;
    for (uint32_t i = threadIdx.x; i < slice; i += PC_THREADS) tab[i] = lo + i < N ? table[lo + i] : 0;
    // every block of the cluster has filled its slice before anyone reads it
    asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    const uint32_t base = (uint32_t)__cvta_generic_to_shared(tab);
    const int64_t ntiles = (nnz + PC_TILE - 1) / PC_TILE;
    unsigned long long mine = 0ull;
    for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const int64_t e0 = tile * PC_TILE;
        const int ne = (int)min((int64_t)PC_TILE, nnz - e0);
        int4 c[PB_VEC];
#pragma unroll
        for (int i = 0; i < PB_VEC; ++i) {
            const int q = (i * PC_THREADS + threadIdx.x) * 4;
            if (q + 3 < ne) {
                c[i] = __ldcs(reinterpret_cast<const int4 *>(colidx + e0) + (q >> 2));
            } else {
                c[i].x = q + 0 < ne ? colidx[e0 + q + 0] : -1;
                c[i].y = q + 1 < ne ? colidx[e0 + q + 1] : -1;
                c[i].z = q + 2 < ne ? colidx[e0 + q + 2] : -1;
                c[i].w = -1;
            }
        }
        unsigned t = 0;
#pragma unroll
        for (int i = 0; i < PB_VEC; ++i) {
            const int cols[4] = {c[i].x, c[i].y, c[i].z, c[i].w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t col = (uint32_t)cols[j];
                if (col < (uint32_t)N) {
                    uint32_t r = __umulhi(col, magic);            // col / slice, at most one too high
                    if (r * slice > col) r -= 1;
                    r = min(r, (uint32_t)csize - 1u);
                    const uint32_t off = min(col - r * slice, slice - 1u);
                    uint32_t addr, v;
                    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(addr) : "r"(base + off), "r"(r));
                    asm volatile("ld.shared::cluster.u8 %0, [%1];" : "=r"(v) : "r"(addr));
                    t += v;
                }
            }
        }
        mine += t;
    }
    // no block leaves while another may still read its slice
    asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    block_add(mine, sum);
}

}  // namespace

extern "C" int ep_probe_gather(ep_ctx *ctx, const int32_t *colidx, int64_t nnz, const uint8_t *table, int64_t N,
                               int32_t cluster_size, uint64_t *sum, void *cuda_stream) {
    using namespace ep;
    if (!ctx) return EP_ERR_INVALID_ARG;
    if (!colidx || !table || !sum) return fail(ctx, EP_ERR_INVALID_ARG, "null pointer");
    if (!aligned(colidx, 16) || !aligned(sum, 8)) return fail(ctx, EP_ERR_INVALID_ARG, "misaligned pointer");
    if (N < 1 || N >= (int64_t(1) << 31) || nnz < 1 || nnz >= (int64_t(1) << 40))
        return fail(ctx, EP_ERR_INVALID_ARG, "shape out of range: N=%lld nnz=%lld", (long long)N, (long long)nnz);
    if (cluster_size != -1 && cluster_size != 0 && cluster_size != 2 && cluster_size != 4 && cluster_size != 8 &&
        cluster_size != 16)
        return fail(ctx, EP_ERR_INVALID_ARG, "cluster_size must be -1 (texture), 0 (global memory), 2, 4, 8 or 16");
    DeviceGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    auto *out = reinterpret_cast<unsigned long long *>(sum);
    EP_CUDA(ctx, cudaMemsetAsync(out, 0, sizeof(unsigned long long), st));
    if (cluster_size == 0) {
        const int grid = (int)std::min<int64_t>(ceil_div(nnz, PB_TILE), (int64_t)ctx->sm_count * 4);
        gather_global<<<grid, PB_THREADS, 0, st>>>(colidx, nnz, table, N, out);
        ctx->launches += 1;
        EP_CUDA(ctx, cudaGetLastError());
        return EP_OK;
    }
    if (cluster_size == -1) {
        int max_linear = 0, tex_align = 0;
        EP_CUDA(ctx, cudaDeviceGetAttribute(&max_linear, cudaDevAttrMaxTexture1DLinearWidth, ctx->device));
        EP_CUDA(ctx, cudaDeviceGetAttribute(&tex_align, cudaDevAttrTextureAlignment, ctx->device));
        if (N > (int64_t)max_linear)
            return fail(ctx, EP_ERR_UNSUPPORTED, "%lld table bytes exceed the widest linear texture (%d)", (long long)N, max_linear);
        if (tex_align > 0 && !aligned(table, (size_t)tex_align))
            return fail(ctx, EP_ERR_INVALID_ARG, "the table must be aligned to %d bytes for the texture path", tex_align);
        if (ctx->probe_tex == 0 || ctx->probe_tex_ptr != table || ctx->probe_tex_n != (long long)N) {
            if (ctx->probe_tex) {                              // a kernel of an earlier call may still read through it
                EP_CUDA(ctx, cudaDeviceSynchronize());
                cudaDestroyTextureObject((cudaTextureObject_t)ctx->probe_tex);
                ctx->probe_tex = 0;
            }
            cudaResourceDesc res = {};
            res.resType = cudaResourceTypeLinear;
            res.res.linear.devPtr = const_cast<uint8_t *>(table);
            res.res.linear.desc = cudaCreateChannelDesc<unsigned char>();
            res.res.linear.sizeInBytes = (size_t)N;
            cudaTextureDesc td = {};
            td.readMode = cudaReadModeElementType;
            cudaTextureObject_t tex = 0;
            EP_CUDA(ctx, cudaCreateTextureObject(&tex, &res, &td, nullptr));
            ctx->probe_tex = (unsigned long long)tex;
            ctx->probe_tex_ptr = table;
            ctx->probe_tex_n = (long long)N;
        }
        const int grid = (int)std::min<int64_t>(ceil_div(nnz, PB_TILE), (int64_t)ctx->sm_count * 4);
        gather_texture<<<grid, PB_THREADS, 0, st>>>(colidx, nnz, (cudaTextureObject_t)ctx->probe_tex, N, out);
        ctx->launches += 1;
        EP_CUDA(ctx, cudaGetLastError());
        return EP_OK;
    }
    const uint32_t slice = (uint32_t)(ceil_div(ceil_div(N, cluster_size), 16) * 16);
    if ((size_t)slice + 1024 > (size_t)ctx->smem_optin)
        return fail(ctx, EP_ERR_UNSUPPORTED, "%lld table bytes do not fit the shared memory of %d blocks", (long long)N, cluster_size);
    const uint32_t magic = (uint32_t)(((uint64_t(1) << 32) + slice - 1) / slice);
    EP_CUDA(ctx, cudaFuncSetAttribute(gather_cluster, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)slice));
    if (cluster_size > 8) EP_CUDA(ctx, cudaFuncSetAttribute(gather_cluster, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(PC_THREADS);
    cfg.dynamicSmemBytes = slice;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)cluster_size;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    cfg.gridDim = dim3((unsigned)cluster_size);
    int nclusters = 0;
    if (cudaOccupancyMaxActiveClusters(&nclusters, gather_cluster, &cfg) != cudaSuccess || nclusters < 1) {
        cudaGetLastError();
        return fail(ctx, EP_ERR_UNSUPPORTED, "no cluster of %d blocks with %u bytes of shared memory each fits this device", cluster_size, slice);
    }
    nclusters = (int)std::min<int64_t>(nclusters, ceil_div(ceil_div(nnz, PC_TILE), cluster_size));
    cfg.gridDim = dim3((unsigned)(nclusters * cluster_size));
    EP_CUDA(ctx, cudaLaunchKernelEx(&cfg, gather_cluster, colidx, nnz, table, N, slice, magic, (int)cluster_size, out));
    ctx->launches += 1;
    return EP_OK;
}
