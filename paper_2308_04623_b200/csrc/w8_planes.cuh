// Activations for the 8-bit tensor-core kind: a value as four e4m3 planes.
//
// The 8-bit kind of tcgen05.mma wants both operands in an 8-bit format.  The weights are e4m3 codes in HBM; an
// activation x (fp32) is split, by the kernel that produces it, into four e4m3 numbers
//     p0 = rn(x / 16),  p1 = rn(x - 16 p0),  p2 = rn(16 (x - 16 p0 - p1)),  p3 = rn(256 (x - 16 p0 - p1 - p2 / 16))
// (rn = round to nearest e4m3, saturating; every residual is exact in fp32), so that
//     x = 16 p0 + p1 + p2 / 16 + p3 / 256
// up to half a step of the last plane: 2^-17 relative for |x| >= 2^-2 or so, 2^-18 absolute below (an e4m3 number
// carries 4 significant bits; its steps stop shrinking at 2^-9).  That is what the bf16 hi + lo pair of the 16-bit
// path carries.  |x| may reach 16 * 448 = 7168 before the first plane saturates; the later planes then absorb
// what they can.  A NaN becomes the format's NaN code in plane 0 and so reaches the logits.  The projection
// multiplies the four planes by the same weight slice in one instruction and recombines the four sums with the
// same powers of two.
//
// Layout in memory: [4 planes][rows][K] bytes, plane-major, so that one 3-D copy brings [4][n_pad][128] into a stage.
#pragma once
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace w8 {
// Two values at a time: the conversions are packed instructions.
__device__ __forceinline__ uint32_t enc2(float lo, float hi) { // code(lo) in byte 0, code(hi) in byte 1
    uint16_t d;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(d) : "f"(hi), "f"(lo));
    return d;
}
__device__ __forceinline__ float2 dec2(uint32_t codes) {
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)codes));
    return __half22float2(*reinterpret_cast<const __half2 *>(&h2));
}
// The four codes of x and of y: plane p of x in byte p of .x, of y in byte p of .y.
__device__ __forceinline__ uint2 split4x2(float x, float y) {
    const uint32_t c0 = enc2(x * 0.0625f, y * 0.0625f);
    const float2 v0 = dec2(c0);
    const float rx1 = x - 16.f * v0.x, ry1 = y - 16.f * v0.y;
    const uint32_t c1 = enc2(rx1, ry1);
    const float2 v1 = dec2(c1);
    const float rx2 = rx1 - v1.x, ry2 = ry1 - v1.y;
    const uint32_t c2 = enc2(rx2 * 16.f, ry2 * 16.f);
    const float2 v2 = dec2(c2);
    const float rx3 = rx2 - 0.0625f * v2.x, ry3 = ry2 - 0.0625f * v2.y;
    const uint32_t c3 = enc2(rx3 * 256.f, ry3 * 256.f);
    // c_k = [code_k(x), code_k(y)] in bytes 0, 1
    const uint32_t lo = __byte_perm(c0, c1, 0x5140), hi = __byte_perm(c2, c3, 0x5140); // [c0x, c1x, c0y, c1y], [c2x, c3x, c2y, c3y]
    return make_uint2(__byte_perm(lo, hi, 0x5410), __byte_perm(lo, hi, 0x7632));
}
// Four consecutive values of a row -> one 32-bit store per plane.  `at` = row * K + k (k a multiple of 4).
__device__ __forceinline__ void store4(uint8_t *planes, size_t plane_stride, size_t at, float a, float b, float c, float d) {
    const uint2 ab = split4x2(a, b), cd = split4x2(c, d);
    const uint32_t w0 = ab.x, w1 = ab.y, w2 = cd.x, w3 = cd.y;
    const uint32_t A = __byte_perm(w0, w1, 0x5140), B = __byte_perm(w2, w3, 0x5140);   // planes 0 and 1 of (a, b) / of (c, d)
    const uint32_t C = __byte_perm(w0, w1, 0x7362), D = __byte_perm(w2, w3, 0x7362);   // planes 2 and 3
    *reinterpret_cast<uint32_t *>(planes + at) = __byte_perm(A, B, 0x5410);
    *reinterpret_cast<uint32_t *>(planes + plane_stride + at) = __byte_perm(A, B, 0x7632);
    *reinterpret_cast<uint32_t *>(planes + 2 * plane_stride + at) = __byte_perm(C, D, 0x5410);
    *reinterpret_cast<uint32_t *>(planes + 3 * plane_stride + at) = __byte_perm(C, D, 0x7632);
}
} // namespace w8
