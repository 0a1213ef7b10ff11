// The one rotation every RoPE kernel of the library applies to a packed pair.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

namespace ll {

// Rotate one packed bf16 pair (low half = element 2j, high half = element 2j+1) by the
// angle whose (cos, sin) is cs, in fp32.
__device__ __forceinline__ void rotate_pair_f32(uint32_t packed, float2 cs, float &r0, float &r1)
{
    float a = __uint_as_float(packed << 16);
    float b = __uint_as_float(packed & 0xffff0000u);
    r0 = fmaf(a, cs.x, -(b * cs.y));
    r1 = fmaf(a, cs.y, b * cs.x);
}

// The same with one rounding to bf16 at the end.
__device__ __forceinline__ uint32_t rotate_pair(uint32_t packed, float2 cs)
{
    float r0, r1;
    rotate_pair_f32(packed, cs, r0, r1);
    __nv_bfloat162 o = __floats2bfloat162_rn(r0, r1);   // .x (low half) = r0
    return *reinterpret_cast<uint32_t *>(&o);
}

// Two fp32 values to two E4M3 codes (round to nearest even, saturating at +-448); `lo` lands in
// the low byte.
__device__ __forceinline__ uint32_t cvt_e4m3x2(float lo, float hi)
{
    uint16_t d;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(d) : "f"(hi), "f"(lo));
    return d;
}

// Two E4M3 codes (low 16 bits of `codes`) to two bf16 values, exactly (every E4M3 value is a
// bf16 value); the low byte's value lands in the low half.
__device__ __forceinline__ uint32_t e4m3x2_to_bf16x2(uint32_t codes)
{
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)codes));
    const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&h2));
    __nv_bfloat162 o = __floats2bfloat162_rn(f.x, f.y);
    return *reinterpret_cast<uint32_t *>(&o);
}

}  // namespace ll
