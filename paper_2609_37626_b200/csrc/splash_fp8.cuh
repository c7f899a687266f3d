// Building blocks shared by the e4m3 decode kernels: 8-bit MMA issue, conversions, swizzle.
#pragma once

#include <cuda_fp16.h>

#include "splash_umma.cuh"

namespace splash {
namespace umma {

__host__ __device__ constexpr uint32_t make_idesc_e4m3(int M, int N, int a_mn_major, int b_e5m2 = 0, int b_mn_major = 0,
                                                        int a_e5m2 = 0) {
    // fp32 accumulate (bit 4); A / B formats E4M3 (= 0) or E5M2 (= 1) in bits 7..9 / 10..12
    return (1u << 4) | ((uint32_t)a_e5m2 << 7) | ((uint32_t)b_e5m2 << 10) | ((uint32_t)a_mn_major << 15) |
           ((uint32_t)b_mn_major << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ void umma_e4m3(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// two floats -> two e4m3 bytes (first argument in the low byte), round to nearest, saturating
__device__ __forceinline__ uint16_t to_e4m3x2(float lo, float hi) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ uint16_t to_e5m2x2(float lo, float hi) {
    uint16_t r;
    asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float2 from_e4m3x2(uint16_t v) {
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(v));
    __half2 h = *reinterpret_cast<__half2 *>(&h2);
    return __half22float2(h);
}
// The same split in packed f16 arithmetic: two floats -> (e4m3 pair, e5m2 pair of the residuals), five instructions.
// The detour through f16 (11 significant bits, values below 65,504) costs nothing that the 2-bit mantissa of the
// residual does not already cost; the residual itself is exact in f16.
__device__ __forceinline__ void split_e4m3_e5m2_x2(float lo, float hi, uint16_t &main, uint16_t &rest) {
    uint32_t h2, back, res;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(h2) : "f"(hi), "f"(lo));
    asm("cvt.rn.satfinite.e4m3x2.f16x2 %0, %1;" : "=h"(main) : "r"(h2));
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(back) : "h"(main));
    asm("sub.rn.f16x2 %0, %1, %2;" : "=r"(res) : "r"(h2), "r"(back));
    asm("cvt.rn.satfinite.e5m2x2.f16x2 %0, %1;" : "=h"(rest) : "r"(res));
}
// Two floats -> (e4m3 pair, e4m3 pair of the residuals) in packed f16 arithmetic, for the query operands: the value
// passes through f16 (11 significant bits against the 8 of the bf16 query it comes from), the residual is exact in f16.
__device__ __forceinline__ void split_e4m3_e4m3_x2(float lo, float hi, uint16_t &main, uint16_t &rest) {
    uint32_t h2, back, res;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(h2) : "f"(hi), "f"(lo));
    asm("cvt.rn.satfinite.e4m3x2.f16x2 %0, %1;" : "=h"(main) : "r"(h2));
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(back) : "h"(main));
    asm("sub.rn.f16x2 %0, %1, %2;" : "=r"(res) : "r"(h2), "r"(back));
    asm("cvt.rn.satfinite.e4m3x2.f16x2 %0, %1;" : "=h"(rest) : "r"(res));
}
// Two floats -> (e4m3 pair, e4m3 pair of 16 x the residuals): the residual of an e4m3 rounding is at most 2^-4 of
// the value, so 16 x residual fits the format whenever the value does, and keeps three significant bits.  For kernels
// that accumulate the two terms separately and add them as hi + lo / 16.
__device__ __forceinline__ void split_e4m3_e4m3x16_x2(float lo, float hi, uint16_t &main, uint16_t &rest) {
    uint32_t h2, back, res;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(h2) : "f"(hi), "f"(lo));
    asm("cvt.rn.satfinite.e4m3x2.f16x2 %0, %1;" : "=h"(main) : "r"(h2));
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(back) : "h"(main));
    asm("sub.rn.f16x2 %0, %1, %2;" : "=r"(res) : "r"(h2), "r"(back));
    asm("mul.rn.f16x2 %0, %1, %2;" : "=r"(res) : "r"(res), "r"(0x4C004C00u));     // x 16
    asm("cvt.rn.satfinite.e4m3x2.f16x2 %0, %1;" : "=h"(rest) : "r"(res));
}
__device__ __forceinline__ float fast_log2(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float fast_rcp(float x) {
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

}  // namespace umma
}  // namespace splash
