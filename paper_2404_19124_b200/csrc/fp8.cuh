// e4m3 (1 sign, 4 exponent, 3 mantissa bits, bias 7, largest finite value 448, no infinities) helpers
// for the reduced-precision copy of the vocabulary head: a row x of bf16 values is stored as bytes
// q_i = e4m3(x_i / s) with one fp32 scale s = max|x| / 448 per row, so x_i ~ s * value(q_i).
#pragma once

#include "spec_common.cuh"

namespace spec {

constexpr float kE4m3Max = 448.0f;

// Two floats -> two e4m3 bytes, round to nearest even, saturating; `lo` lands in the low byte.
__device__ __forceinline__ uint32_t e4m3x2(float lo, float hi) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return (uint32_t)r;
}

// Eight floats scaled by `inv` -> eight consecutive e4m3 bytes.
__device__ __forceinline__ uint2 e4m3x8(const float (&x)[8], float inv) {
    uint2 o;
    o.x = e4m3x2(x[0] * inv, x[1] * inv) | (e4m3x2(x[2] * inv, x[3] * inv) << 16);
    o.y = e4m3x2(x[4] * inv, x[5] * inv) | (e4m3x2(x[6] * inv, x[7] * inv) << 16);
    return o;
}

__device__ __forceinline__ float row_scale_of(float amax) { return amax > 0.0f ? amax / kE4m3Max : 1.0f; }

}  // namespace spec
