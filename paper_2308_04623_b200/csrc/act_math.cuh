// Element-wise arithmetic shared by the kernels that turn fp32 activations into tensor-core operands: the GELU of the
// feed-forward block and the bf16 hi / lo split.  Every producer of an operand uses these, so that the value a
// projection multiplies does not depend on which kernel prepared it.
#pragma once
#include <cuda_bf16.h>
#include <cstdint>

namespace act {
// GELU, tanh form: 0.5 z (1 + tanh u) = z / (1 + exp(-2u)),  u = sqrt(2 / pi) (z + 0.044715 z^3)
__device__ __forceinline__ float gelu_tanh_fast(float z) {
    const float u2 = 1.5957691216057308f * (z + 0.044715f * z * z * z);
    return __fdividef(z, 1.0f + __expf(-u2));
}
// four floats -> four bf16 (round to nearest even), in memory order
__device__ __forceinline__ uint2 pack4_bf16(float a, float b, float c, float d) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
    return make_uint2(*reinterpret_cast<const uint32_t *>(&lo), *reinterpret_cast<const uint32_t *>(&hi));
}
// eight floats -> their bf16 values (hi) and the bf16 of what that rounding left (lo), 16 bytes each
__device__ __forceinline__ void split8_bf16(const float (&v)[8], uint4 &hi, uint4 &lo) {
    const uint2 h0 = pack4_bf16(v[0], v[1], v[2], v[3]), h1 = pack4_bf16(v[4], v[5], v[6], v[7]);
    hi = make_uint4(h0.x, h0.y, h1.x, h1.y);
    const uint32_t hw[4] = {h0.x, h0.y, h1.x, h1.y};
    float r[8];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        r[2 * q] = v[2 * q] - __uint_as_float(hw[q] << 16);
        r[2 * q + 1] = v[2 * q + 1] - __uint_as_float(hw[q] & 0xffff0000u);
    }
    const uint2 l0 = pack4_bf16(r[0], r[1], r[2], r[3]), l1 = pack4_bf16(r[4], r[5], r[6], r[7]);
    lo = make_uint4(l0.x, l0.y, l1.x, l1.y);
}
} // namespace act
