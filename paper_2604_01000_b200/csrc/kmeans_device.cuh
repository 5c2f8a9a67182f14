// Device helpers shared by the K-Means translation units: streaming loads, the lane-sliced dot
// product and the transposed warp reduction.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace epk {

constexpr int KC = 8;                 // centroids reduced together by one butterfly
constexpr unsigned FULL = 0xffffffffu;

__device__ __forceinline__ float4 ldg_stream(const float4 *p) {
    float4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w)
                 : "l"(p));
    return r;
}

__device__ __forceinline__ float dot4(const float4 &a, const float4 &b, float acc) {
    acc = fmaf(a.x, b.x, acc);
    acc = fmaf(a.y, b.y, acc);
    acc = fmaf(a.z, b.z, acc);
    acc = fmaf(a.w, b.w, acc);
    return acc;
}

// acc + |a - b|^2 over four coordinates: the squared distance in its direct form.  Every term is
// non-negative and each difference is rounded once, so the result is accurate relative to the DISTANCE
// (a few units in the last place), whatever the norms of a and b are; |b|^2 - 2 a.b is only accurate
// relative to those norms.
__device__ __forceinline__ float dist4(const float4 &a, const float4 &b, float acc) {
    const float tx = a.x - b.x, ty = a.y - b.y, tz = a.z - b.z, tw = a.w - b.w;
    acc = fmaf(tx, tx, acc);
    acc = fmaf(ty, ty, acc);
    acc = fmaf(tz, tz, acc);
    acc = fmaf(tw, tw, acc);
    return acc;
}

// Sums 8 per-lane values across the warp with 9 shuffles instead of 40: each exchange halves the
// number of values a lane still carries.  On return every lane holds the warp-wide total of value
// index ((lane>>4)&1)*4 + ((lane>>3)&1)*2 + ((lane>>2)&1).  The additions pair lanes l and l^16, then
// l^8, l^4, l^2, l^1: the same tree, hence bit for bit the same sum, as warp_sum below.
__device__ __forceinline__ float reduce8_transposed(const float (&a)[KC], int lane) {
    const bool h16 = lane & 16, h8 = lane & 8, h4 = lane & 4;
    float b[4], c[2];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float send = h16 ? a[i] : a[i + 4];
        float keep = h16 ? a[i + 4] : a[i];
        b[i] = keep + __shfl_xor_sync(FULL, send, 16);
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        float send = h8 ? b[i] : b[i + 2];
        float keep = h8 ? b[i + 2] : b[i];
        c[i] = keep + __shfl_xor_sync(FULL, send, 8);
    }
    float send = h4 ? c[0] : c[1];
    float keep = h4 ? c[1] : c[0];
    float v = keep + __shfl_xor_sync(FULL, send, 4);
    v += __shfl_xor_sync(FULL, v, 2);
    v += __shfl_xor_sync(FULL, v, 1);
    return v;
}

__device__ __forceinline__ int lane_chunk_slot(int lane) {
    return ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1);
}

// Warp-wide sum of one value, pairing lanes in the order 16, 8, 4, 2, 1.
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1) v += __shfl_xor_sync(FULL, v, m);
    return v;
}

}  // namespace epk
