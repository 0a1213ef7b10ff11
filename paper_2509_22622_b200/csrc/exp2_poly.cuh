// 2^x for pairs of fp32 values: on the special-function unit, and on the FMA pipe (a clamped
// range reduction and a cubic), for kernels whose exponentials would otherwise all queue on the
// special-function unit.
#pragma once
#include <cstdint>

#include "ptx.cuh"

namespace ll {
namespace ptx {

__device__ __forceinline__ float as_f(uint32_t u) { return __uint_as_float(u); }
__device__ __forceinline__ uint32_t as_u(float f) { return __float_as_uint(f); }

// 2^x for two values on the special-function unit.
__device__ __forceinline__ uint64_t exp2_sfu2(uint64_t x2)
{
    float x0, x1;
    unpack2(x2, x0, x1);
    return pack2(ex2(x0), ex2(x1));
}

// 2^x for two scores on the FMA pipe, x = s * c - m (c = log2(e)/sqrt(D), m the row's reference).
// The scale-and-shift itself does the clamping: y = sat(s * c/128 + (kPolyLow - m)/128) is
// (x + kPolyLow)/128 held to [0, 1], i.e. x held to [-kPolyLow, 128 - kPolyLow].  Then
// 128 y = j + f with j = floor(128 y) read from the low mantissa bits of 128 y + 1.5 * 2^23
// (rounded down), 2^f by a cubic with maximum relative error 7.5e-5 on [0, 1) whose
// coefficients carry the factor 2^-kPolyLow, and j added to the result's exponent field.
// A score below the range gives a weight of 2^-kPolyLow instead of less (irrelevant against a
// row sum >= 1); one above it gives just under 2^(128 - kPolyLow) = 256, which the caller's
// check on the sums (kSafeSum) catches.  NaN scores clamp to the bottom of the range.
constexpr int kPolyLow = 120;
struct PolyRow {
    float cs, bias;                 // c / 128 and (kPolyLow - m) / 128
};
__device__ __forceinline__ uint64_t exp2_poly2(float s0, float s1, const PolyRow &r)
{
    constexpr float kMagic = 12582912.f;
    constexpr float kUnit = 0x1p-120f;
    static_assert(kPolyLow == 120, "the cubic's coefficients carry 2^-kPolyLow");
    const uint64_t y2 = pack2(fma_sat(s0, r.cs, r.bias), fma_sat(s1, r.cs, r.bias));
    const uint64_t r2 = fma2_rm(y2, pack2(128.f, 128.f), pack2(kMagic, kMagic));
    const uint64_t nj2 = fma2(r2, pack2(-1.f, -1.f), pack2(kMagic, kMagic));          // -floor(128 y), exact
    const uint64_t f2 = fma2(y2, pack2(128.f, 128.f), nj2);                           // 128 y - j, exact
    uint64_t p2 = fma2(f2, pack2(0.07802491635f * kUnit, 0.07802491635f * kUnit),
                       pack2(0.22606660426f * kUnit, 0.22606660426f * kUnit));
    p2 = fma2(p2, f2, pack2(0.69583368301f * kUnit, 0.69583368301f * kUnit));
    p2 = fma2(p2, f2, pack2(0.99992519617f * kUnit, 0.99992519617f * kUnit));
    float p0, p1, r0, r1;
    unpack2(p2, p0, p1);
    unpack2(r2, r0, r1);
    return pack2(as_f(mad_lo(as_u(r0), 1u << 23, as_u(p0))), as_f(mad_lo(as_u(r1), 1u << 23, as_u(p1))));
}

}  // namespace ptx
}  // namespace ll
