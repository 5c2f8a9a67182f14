// Device helpers of the tensor-core K-Means kernels: mbarrier waits with a time limit, TMA tile
// loads, tcgen05 (UMMA) descriptors and issue, TMEM loads, and the packed-key bookkeeping.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace eptc {

constexpr long long WAIT_LIMIT_CLOCKS = 4000000000ll;   // ~2 s: far beyond any legitimate wait
constexpr uint32_t KEY_INIT = 0x7F7FFFFFu;              // FLT_MAX: above every real key
constexpr uint32_t IDX_MASK = 127u;                     // a key's low 7 mantissa bits hold a column index

// UMMA instruction descriptor: D = f32, A = B = tf32, both K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t umma_idesc_tf32_m128(int n) {
    return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24);
}

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Waits for the phase of the given parity, but never for ever: after `limit` clocks, or once
// another thread has given up, it sets the block's abort flag and returns false.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag,
                                          long long limit = WAIT_LIMIT_CLOCKS) {
    const uint32_t addr = smem_u32(bar);
    long long t0 = 0;
    for (uint32_t spins = 0;; ++spins) {
        uint32_t ok;
        asm volatile(
            "{\n.reg .pred p;\n"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
            "selp.u32 %0, 1, 0, p;\n}"
            : "=r"(ok)
            : "r"(addr), "r"(parity)
            : "memory");
        if (ok) return true;
        if (*abort_flag) return false;
        if (spins == 64) t0 = clock64();
        if (spins > 64 && (spins & 63) == 0 && clock64() - t0 > limit) {
            *abort_flag = 1;
            return false;
        }
    }
}

// The same wait without the abort flag, for a block that is already on its way out after an abort: it gives the
// copies and MMAs the block has in flight `limit` clocks to finish (their completion is what flips the phase), so
// that nothing of its own still writes to its shared memory or TMEM when it releases them.
__device__ __forceinline__ bool mbar_wait_quiet(uint64_t *bar, uint32_t parity, long long limit) {
    const uint32_t addr = smem_u32(bar);
    const long long t0 = clock64();
    for (uint32_t spins = 0;; ++spins) {
        uint32_t ok;
        asm volatile(
            "{\n.reg .pred p;\n"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
            "selp.u32 %0, 1, 0, p;\n}"
            : "=r"(ok)
            : "r"(addr), "r"(parity)
            : "memory");
        if (ok) return true;
        if ((spins & 63) == 63 && clock64() - t0 > limit) return false;
    }
}
constexpr long long DRAIN_LIMIT_CLOCKS = 20000000ll;   // ~10 ms per barrier on the way out

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int x, int y, uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}

// "Elected" forms for a warp that runs its issue loop as a whole (all lanes wait, count and compute the same
// operands) and lets one lane, chosen by elect.sync, issue.  The operands of TMA and MMA instructions are
// warp-level values; with the loop inside `if (lane == 0)` the same instructions cost far more issue time
// (measured in the fused small-K kernel: 82 -> 54 clocks per tcgen05.mma, which had been the slowest link of the
// pipeline for 256-column rows).
__device__ __forceinline__ void mbar_expect_tx_elected(uint64_t *bar, uint32_t bytes) {
    asm volatile("{\n.reg .pred pe;\nelect.sync _|pe, 0xffffffff;\n"
                 "@pe mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n}" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void tma_load_2d_elected(uint32_t dst, const CUtensorMap *map, int x, int y, uint64_t *bar) {
    asm volatile("{\n.reg .pred pe;\nelect.sync _|pe, 0xffffffff;\n"
                 "@pe cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n}"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void tma_load_3d_elected(uint32_t dst, const CUtensorMap *map, int x, int y, int z,
                                                    uint64_t *bar) {
    asm volatile("{\n.reg .pred pe;\nelect.sync _|pe, 0xffffffff;\n"
                 "@pe cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];\n}"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
                 : "memory");
}
// The four K-steps (8 floats each) of one 128-byte k-block; the first one overwrites the accumulator when
// accumulate_first == 0.
__device__ __forceinline__ void umma_tf32_kblock_elected(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                         uint32_t accumulate_first) {
    asm volatile(
        "{\n.reg .pred pe, pa, pt;\n.reg .b64 a1, a2, a3, b1, b2, b3;\n"
        "elect.sync _|pe, 0xffffffff;\n"
        "setp.ne.b32 pa, %4, 0;\n"
        "setp.eq.b32 pt, 0, 0;\n"
        "add.s64 a1, %1, 2;\nadd.s64 a2, %1, 4;\nadd.s64 a3, %1, 6;\n"
        "add.s64 b1, %2, 2;\nadd.s64 b2, %2, 4;\nadd.s64 b3, %2, 6;\n"
        "@pe tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, pa;\n"
        "@pe tcgen05.mma.cta_group::1.kind::tf32 [%0], a1, b1, %3, pt;\n"
        "@pe tcgen05.mma.cta_group::1.kind::tf32 [%0], a2, b2, %3, pt;\n"
        "@pe tcgen05.mma.cta_group::1.kind::tf32 [%0], a3, b3, %3, pt;\n}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate_first)
        : "memory");
}
__device__ __forceinline__ void umma_commit_elected(uint64_t *bar) {
    asm volatile("{\n.reg .pred pe;\nelect.sync _|pe, 0xffffffff;\n"
                 "@pe tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n}"
                 ::"r"(smem_u32(bar))
                 : "memory");
}

// Plain bulk copy of `bytes` (a multiple of 16, both addresses 16-byte aligned) from global to this block's shared
// memory; the barrier receives the bytes as they land.
__device__ __forceinline__ void bulk_load_1d(void *dst, const void *src, uint32_t bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// Shared-memory operand descriptor: K-major rows of 128 bytes, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
    return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
           (2ull << 61);
}

__device__ __forceinline__ void umma_tf32(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n.reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The barrier receives one arrival when every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 32 consecutive accumulator columns of this thread's TMEM lane: the load is only issued here; v holds the
// columns after tmem_ld_wait(v).
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}

// Waits for every TMEM load this thread has issued.  The registers pass through the statement so that no use
// of them can be scheduled ahead of the wait.
__device__ __forceinline__ void tmem_ld_wait(uint32_t (&v)[32]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
                   "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15]),
                   "+r"(v[16]), "+r"(v[17]), "+r"(v[18]), "+r"(v[19]), "+r"(v[20]), "+r"(v[21]), "+r"(v[22]),
                   "+r"(v[23]), "+r"(v[24]), "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), "+r"(v[28]), "+r"(v[29]),
                   "+r"(v[30]), "+r"(v[31])
                 :
                 : "memory");
}

// 16 consecutive accumulator columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Smallest of three (one instruction on sm_100).
__device__ __forceinline__ float fmin3(float a, float b, float c) {
    float r;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// Keeps the two smallest keys seen.  A key is a score whose low 7 mantissa bits hold the column's
// index inside its group, compared as a float, so one min/max pair carries value and index.
__device__ __forceinline__ void keep_two(float &b1, float &b2, float key) {
    const float t = fmaxf(key, b1);
    b1 = fminf(key, b1);
    b2 = fminf(b2, t);
}

// Error allowance of a screened score s~ = |c|^2 - 2 fl(x~.c~) against the fp32 score, for a row x and
// any centroid c.  x~ is what the tensor core makes of x (it drops the low 13 mantissa bits, or rounds:
// either way |x - x~| <= |x - trunc(x)| element by element), c~ the TF32-rounded copy the update kernel
// stores.  x.c - x~.c~ = (x - x~).c + x~.(c - c~), so by Cauchy-Schwarz
//     |x.c - x~.c~| <= xlo * cmax + xnorm * clomax
// with xlo = |x - trunc(x)|_2 measured on this very row and clomax = max_k |c_k - c~_k|_2 measured on the
// centroids.  The products x~_j c~_j are exact in fp32; summing d of them and the final fma lose at most
// (d + 2) 2^-23 of |x||c| each way, allowed for as d 2^-20; overwriting 7 mantissa bits with the index
// moves a score by < 2^-16 of itself.
__device__ __forceinline__ float screen_allowance(float xnorm, float xlo, float cmax, float cmax2, float clomax, int d) {
    const float a = xnorm * cmax;
    return 2.002f * (xlo * cmax + xnorm * clomax) + a * ((float)d * 9.6e-7f) + 1.6e-5f * (cmax2 + 2.f * a);
}


}  // namespace eptc
