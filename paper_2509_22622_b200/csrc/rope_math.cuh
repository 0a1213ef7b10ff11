// The one rotation every RoPE kernel of the library applies to a packed pair.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

namespace ll {

// Rotate one packed bf16 pair (low half = element 2j, high half = element 2j+1) by the
// angle whose (cos, sin) is cs, in fp32, with one rounding to bf16 at the end.
__device__ __forceinline__ uint32_t rotate_pair(uint32_t packed, float2 cs)
{
    float a = __uint_as_float(packed << 16);
    float b = __uint_as_float(packed & 0xffff0000u);
    float r0 = fmaf(a, cs.x, -(b * cs.y));
    float r1 = fmaf(a, cs.y, b * cs.x);
    __nv_bfloat162 o = __floats2bfloat162_rn(r0, r1);   // .x (low half) = r0
    return *reinterpret_cast<uint32_t *>(&o);
}

}  // namespace ll
