// Fragment helpers of the mma.sync kernels for quantised (byte) caches: bytes -> f16 A fragments, f16 MMAs, the
// quantising store of appended rows, and the power-of-two scaling that keeps query rows inside f16's range.
#pragma once
#include <cuda_fp16.h>

#include "common.cuh"

namespace lethe {
namespace {

__device__ __forceinline__ void mma_f16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// two e4m3 bytes (low 16 bits of x) -> f16x2, byte 0 in the low half
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t x) {
    uint32_t y;
    asm("{ .reg .b16 lo; cvt.u16.u32 lo, %1; cvt.rn.f16x2.e4m3x2 %0, lo; }" : "=r"(y) : "r"(x));
    return y;
}
// Bytes `sel_lo` and `sel_hi` (0..3) of x -> f16x2.  An e5m2 byte is the upper byte of the half of the same value,
// so one byte permute does it; e4m3 goes through the conversion instruction.
template <bool E5M2, int SEL_LO, int SEL_HI>
__device__ __forceinline__ uint32_t bytes_to_f16x2(uint32_t x) {
    if constexpr (E5M2) return __byte_perm(x, 0u, 0x0404 | (SEL_LO << 4) | (SEL_HI << 12));  // [0, lo, 0, hi]
    else if constexpr (SEL_LO == 0 && SEL_HI == 1) return e4m3x2_to_f16x2(x);                 // the low 16 bits as they are
    else if constexpr (SEL_LO == 2 && SEL_HI == 3) return e4m3x2_to_f16x2(x >> 16);
    else return e4m3x2_to_f16x2(__byte_perm(x, 0u, 0x4400 | SEL_LO | (SEL_HI << 4)));        // [lo, hi, 0, 0]
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
    __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
// two fp32 -> two e4m3 bytes (round to nearest even, saturating), `lo` in the low byte
template <bool E5M2>
__device__ __forceinline__ uint32_t f32x2_to_fp8x2(float lo, float hi) {
    uint32_t y;
    if (E5M2) asm("{ .reg .b16 r; cvt.rn.satfinite.e5m2x2.f32 r, %2, %1; cvt.u32.u16 %0, r; }" : "=r"(y) : "f"(lo), "f"(hi));
    else asm("{ .reg .b16 r; cvt.rn.satfinite.e4m3x2.f32 r, %2, %1; cvt.u32.u16 %0, r; }" : "=r"(y) : "f"(lo), "f"(hi));
    return y;
}
// bf16 pair (as stored) -> f16x2
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t x) {
    const float lo = __uint_as_float(x << 16), hi = __uint_as_float(x & 0xffff0000u);
    return pack_f16(lo, hi);
}
// two bf16 values times a power of two -> two f16 values (exact while the products are within f16's range)
__device__ __forceinline__ uint32_t bf16x2_to_f16x2_scaled(uint32_t x, float mul) {
    return pack_f16(__uint_as_float(x << 16) * mul, __uint_as_float(x & 0xffff0000u) * mul);
}
// The divisor (a power of two, returned in `div`) that brings the largest magnitude of a query row into [128, 256), and
// its inverse (the return value).  The row is spread over the four lanes that share gq = lane >> 2; w holds this lane's
// bf16 pairs.
template <int KS>
__device__ __forceinline__ float query_row_scale(const uint2 (&w)[KS], float& div) {
    float big = 0.f;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
        big = fmaxf(big, fmaxf(fabsf(__uint_as_float(w[ks].x << 16)), fabsf(__uint_as_float(w[ks].x & 0xffff0000u))));
        big = fmaxf(big, fmaxf(fabsf(__uint_as_float(w[ks].y << 16)), fabsf(__uint_as_float(w[ks].y & 0xffff0000u))));
    }
    big = fmaxf(big, __shfl_xor_sync(0xffffffffu, big, 1));
    big = fmaxf(big, __shfl_xor_sync(0xffffffffu, big, 2));
    int ex = (int)((__float_as_uint(big) >> 23) & 0xffu) - 7;  // biased exponent of the divisor
    ex = big > 0.f && big < INFINITY ? min(max(ex, 2), 252) : 127;
    div = __uint_as_float((uint32_t)ex << 23);
    return __uint_as_float((uint32_t)(254 - ex) << 23);
}

}  // namespace
}  // namespace lethe
