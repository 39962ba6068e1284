// Element-wise kernels of the bf16 path: they turn the fp32 residual stream into the bf16
// operands the tensor-core projections read (LayerNorm, bias + GELU), and zero the fp32
// buffers those projections accumulate into.
//
// A value v is handed to the tensor cores as two bf16 planes, hi = bf16(v) and
// lo = bf16(v - hi); the projection multiplies both by the same weight tile, which keeps the
// activations to ~16 mantissa bits at no cost in HBM traffic.
//
// With 8-bit weights the projections run on the 8-bit tensor-core kind and read their activations as four e4m3 planes
// instead (the P8 instantiations; see w8_planes.cuh).
#include "sm100_ptx.cuh"
#include "ssd_internal.h"
#include "w8_planes.cuh"
#include "act_math.cuh"

namespace {
__device__ __forceinline__ float block_sum_256(float v, float *red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) t += red[w];
    return t;
}

// Row i: a = LayerNorm(x[i, :]) -> bf16 hi/lo planes; also zero[i, 0:zero_cols] = 0.
// The row is read once, as 16-byte vectors held in registers (d a multiple of 4, at most 4 * PER4 * 256: PER4 = 2 serves d <= 2048, PER4 = 8 the rest up to 8192), so the
// kernel is one L2 round trip plus two block reductions; the code is kept small on purpose (these kernels run once
// per layer between other kernels, and what they mostly wait for is their own instructions).
using act::pack4_bf16;
using act::gelu_tanh_fast;
template <int PER4, bool P8>
__global__ void __launch_bounds__(256) ln_prep_kernel(const float *__restrict__ x, const float *__restrict__ g, const float *__restrict__ b,
                                                      int d, float eps, __nv_bfloat16 *__restrict__ a_hi, __nv_bfloat16 *__restrict__ a_lo,
                                                      float *__restrict__ zero, int zero_cols, const StepInfo *__restrict__ info,
                                                      int zero_from_info, unsigned long long *trace, uint8_t *__restrict__ planes8,
                                                      size_t plane_stride) {
    __shared__ float red[8];
    if (threadIdx.x == 0) ptx::trace_mark(trace, 0);
    ptx::pdl_launch_dependents();
    const int i = blockIdx.x, d4 = d >> 2;
    const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
    float4 gv[PER4], bv[PER4], v[PER4];
#pragma unroll
    for (int q = 0; q < PER4; ++q) { // gain and bias do not depend on the previous kernel: fetch them before waiting for it
        const int k4 = threadIdx.x + q * 256;
        gv[q] = k4 < d4 ? __ldg(reinterpret_cast<const float4 *>(g) + k4) : zero4;
        bv[q] = k4 < d4 ? __ldg(reinterpret_cast<const float4 *>(b) + k4) : zero4;
    }
    ptx::pdl_grid_wait();
    if (threadIdx.x == 0) ptx::trace_mark(trace, 1);
    if (zero_from_info) zero = info->logits;
    const float4 *xr = reinterpret_cast<const float4 *>(x + (size_t)i * d);
    float s = 0.f;
#pragma unroll
    for (int q = 0; q < PER4; ++q) {
        const int k4 = threadIdx.x + q * 256;
        v[q] = k4 < d4 ? xr[k4] : zero4;
        s += (v[q].x + v[q].y) + (v[q].z + v[q].w);
    }
    const float mean = block_sum_256(s, red) / d;
    float sq = 0.f;
#pragma unroll
    for (int q = 0; q < PER4; ++q) {
        const int k4 = threadIdx.x + q * 256;
        if (k4 < d4) {
            v[q].x -= mean; v[q].y -= mean; v[q].z -= mean; v[q].w -= mean;
            sq += (v[q].x * v[q].x + v[q].y * v[q].y) + (v[q].z * v[q].z + v[q].w * v[q].w);
        }
    }
    const float rstd = 1.0f / sqrtf(block_sum_256(sq, red) / d + eps);
#pragma unroll
    for (int q = 0; q < PER4; ++q) {
        const int k4 = threadIdx.x + q * 256;
        if (k4 < d4) {
            const float o0 = v[q].x * rstd * gv[q].x + bv[q].x, o1 = v[q].y * rstd * gv[q].y + bv[q].y;
            const float o2 = v[q].z * rstd * gv[q].z + bv[q].z, o3 = v[q].w * rstd * gv[q].w + bv[q].w;
            const size_t at = (size_t)i * d + 4 * (size_t)k4;
            if (P8) { w8::store4(planes8, plane_stride, at, o0, o1, o2, o3); continue; }
            const uint2 hi = pack4_bf16(o0, o1, o2, o3);
            *reinterpret_cast<uint2 *>(a_hi + at) = hi;
            if (a_lo) {
                const float h0 = __uint_as_float(hi.x << 16), h1 = __uint_as_float(hi.x & 0xffff0000u);
                const float h2 = __uint_as_float(hi.y << 16), h3 = __uint_as_float(hi.y & 0xffff0000u);
                *reinterpret_cast<uint2 *>(a_lo + at) = pack4_bf16(o0 - h0, o1 - h1, o2 - h2, o3 - h3);
            }
        }
    }
    if (zero) {
        float *zr = zero + (size_t)i * zero_cols;
        if ((zero_cols & 3) == 0) { // rows are then 16-byte aligned
            float4 *z4 = reinterpret_cast<float4 *>(zr);
            for (int k = threadIdx.x; k < zero_cols / 4; k += 256) z4[k] = zero4;
        } else {
            for (int k = threadIdx.x; k < zero_cols; k += 256) zr[k] = 0.f;
        }
    }
    if (trace) { __syncthreads(); if (threadIdx.x == 0) ptx::trace_mark(trace, 2); }
}

// h = gelu(acc) -> bf16 hi/lo planes (acc already holds the bias); eight consecutive values per thread (count is a
// multiple of 8: the feed-forward width is a multiple of 64)
template <bool P8>
__global__ void __launch_bounds__(256) gelu_prep_kernel(const float *__restrict__ acc, size_t count, __nv_bfloat16 *__restrict__ h_hi,
                                                        __nv_bfloat16 *__restrict__ h_lo, unsigned long long *trace, uint8_t *__restrict__ planes8,
                                                        size_t plane_stride) {
    if (threadIdx.x == 0) ptx::trace_mark(trace, 0);
    ptx::pdl_launch_dependents();
    ptx::pdl_grid_wait();
    if (threadIdx.x == 0) ptx::trace_mark(trace, 1);
    for (size_t e = ((size_t)blockIdx.x * 256 + threadIdx.x) * 8; e < count; e += (size_t)gridDim.x * 256 * 8) {
        const float4 a = __ldcg(reinterpret_cast<const float4 *>(acc + e)), b = __ldcg(reinterpret_cast<const float4 *>(acc + e + 4));
        float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
        for (int q = 0; q < 8; ++q) v[q] = gelu_tanh_fast(v[q]);
        if (P8) { // (the flat index is row * F + k: the planes have the same shape)
            w8::store4(planes8, plane_stride, e, v[0], v[1], v[2], v[3]);
            w8::store4(planes8, plane_stride, e + 4, v[4], v[5], v[6], v[7]);
            continue;
        }
        const uint2 h0 = pack4_bf16(v[0], v[1], v[2], v[3]), h1 = pack4_bf16(v[4], v[5], v[6], v[7]);
        *reinterpret_cast<uint4 *>(h_hi + e) = make_uint4(h0.x, h0.y, h1.x, h1.y);
        if (h_lo) {
            const uint32_t hw[4] = {h0.x, h0.y, h1.x, h1.y};
            float r[8];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                r[2 * q] = v[2 * q] - __uint_as_float(hw[q] << 16);
                r[2 * q + 1] = v[2 * q + 1] - __uint_as_float(hw[q] & 0xffff0000u);
            }
            const uint2 l0 = pack4_bf16(r[0], r[1], r[2], r[3]), l1 = pack4_bf16(r[4], r[5], r[6], r[7]);
            *reinterpret_cast<uint4 *>(h_lo + e) = make_uint4(l0.x, l0.y, l1.x, l1.y);
        }
    }
    if (trace) { __syncthreads(); if (threadIdx.x == 0) ptx::trace_mark(trace, 2); }
}

// c1[o] = sum_k g[k] W[o,k] ; c2[o] = sum_k beta[k] W[o,k] + bias[o]   (one warp per output feature; load time only)
__global__ void ln_fold_kernel(const __nv_bfloat16 *__restrict__ W, const float *__restrict__ g, const float *__restrict__ beta,
                               const float *__restrict__ bias, int out, int K, float *__restrict__ c1, float *__restrict__ c2) {
    const int o = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (o >= out) return;
    const __nv_bfloat16 *w = W + (size_t)o * K;
    float a = 0.f, b = 0.f;
    for (int k = lane; k < K; k += 32) {
        const float wv = __bfloat162float(w[k]);
        a = fmaf(g[k], wv, a);
        b = fmaf(beta[k], wv, b);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) { a += __shfl_xor_sync(0xffffffffu, a, off); b += __shfl_xor_sync(0xffffffffu, b, off); }
    if (lane == 0) { c1[o] = a; c2[o] = b + (bias ? bias[o] : 0.f); }
}

template <typename... Args>
cudaError_t launch_pdl(void (*kernel)(Args...), dim3 grid, dim3 block, cudaStream_t s, bool pdl, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}
} // namespace

// All kernels of the forward ask for the same (maximum) shared-memory carve-out: an SM that has
// to switch its L1/shared split between two kernels cannot overlap them.
cudaError_t prep_kernels_prepare() {
    cudaError_t e = cudaSuccess;
    const void *kernels[] = {(const void *)ln_prep_kernel<2, false>, (const void *)ln_prep_kernel<8, false>, (const void *)ln_prep_kernel<2, true>,
                             (const void *)ln_prep_kernel<8, true>, (const void *)gelu_prep_kernel<false>, (const void *)gelu_prep_kernel<true>};
    for (const void *k : kernels)
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    return e;
}

cudaError_t launch_ln_fold(const void *W, const float *g, const float *beta, const float *bias, int out, int K, float *c1, float *c2, cudaStream_t s) {
    const int threads = 256, warps_per_block = threads / 32;
    ln_fold_kernel<<<(out + warps_per_block - 1) / warps_per_block, threads, 0, s>>>((const __nv_bfloat16 *)W, g, beta, bias, out, K, c1, c2);
    return cudaGetLastError();
}

cudaError_t launch_ln_prep(const float *x, const float *g, const float *b, int n, int d, float eps, __nv_bfloat16 *a_hi, __nv_bfloat16 *a_lo,
                           float *zero, int zero_cols, const StepInfo *info, int zero_from_info, bool pdl, cudaStream_t s,
                           unsigned long long *trace, uint8_t *planes8, size_t plane_stride) {
    if ((d & 3) || d > 8192) return cudaErrorInvalidValue;
    auto kernel = planes8 ? (d <= 2048 ? ln_prep_kernel<2, true> : ln_prep_kernel<8, true>) : (d <= 2048 ? ln_prep_kernel<2, false> : ln_prep_kernel<8, false>);
    return launch_pdl(kernel, dim3(n), dim3(256), s, pdl, x, g, b, d, eps, a_hi, a_lo, zero, zero_cols, info, zero_from_info, trace, planes8, plane_stride);
}

cudaError_t launch_gelu_prep(const float *acc, int n, int F, __nv_bfloat16 *h_hi, __nv_bfloat16 *h_lo, bool pdl, cudaStream_t s,
                             unsigned long long *trace, uint8_t *planes8, size_t plane_stride) {
    const size_t count = (size_t)n * F;
    int grid = (int)((count + 256 * 8 - 1) / (256 * 8));
    if (grid > 148 * 4) grid = 148 * 4;
    return launch_pdl(planes8 ? gelu_prep_kernel<true> : gelu_prep_kernel<false>, dim3(grid), dim3(256), s, pdl, acc, count, h_hi, h_lo, trace, planes8,
                      plane_stride);
}

// ---- 8-bit weights: per-row power-of-two scale and e4m3 codes (run once, when the model is loaded) ----
namespace {
__global__ void __launch_bounds__(256) quantise_rows_e4m3_kernel(const __nv_bfloat16 *__restrict__ w, size_t cols, uint8_t *__restrict__ codes,
                                                                 float *__restrict__ scales) {
    const size_t row = blockIdx.x;
    const __nv_bfloat16 *src = w + row * cols;
    __shared__ float part[8];
    __shared__ float scale_sh;
    float amax = 0.f;
    for (size_t k = threadIdx.x; k < cols; k += blockDim.x) amax = fmaxf(amax, fabsf(__bfloat162float(src[k])));
    for (int o = 16; o; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = amax;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < 8; ++i) amax = fmaxf(amax, part[i]);
        // amax = f * 2^x with f in [0.5, 1); 448 = 0.875 * 2^9: the smallest e with amax <= 448 * 2^e
        float sc = 1.f;
        if (amax > 0.f && isfinite(amax)) {
            int x;
            const float f = frexpf(amax, &x);
            int e = (f <= 0.875f) ? x - 9 : x - 8;
            e = e < -100 ? -100 : (e > 100 ? 100 : e);
            sc = ldexpf(1.f, e);
        }
        scale_sh = sc;
        scales[row] = sc;
    }
    __syncthreads();
    const float inv = 1.f / scale_sh; // (a power of two: exact)
    for (size_t k = threadIdx.x; k < cols; k += blockDim.x)
        codes[row * cols + k] = (uint8_t)__nv_cvt_float_to_fp8(__bfloat162float(src[k]) * inv, __NV_SATFINITE, __NV_E4M3);
}
} // namespace

cudaError_t launch_quantise_rows_e4m3(const void *w_bf16, size_t rows, size_t cols, uint8_t *codes, float *scales, cudaStream_t s) {
    quantise_rows_e4m3_kernel<<<(unsigned)rows, 256, 0, s>>>((const __nv_bfloat16 *)w_bf16, cols, codes, scales);
    return cudaGetLastError();
}
