// Tree preparation, embedding and LayerNorm kernels.
//
// Section 3.1 of the paper realises the tree batch through two controls: the position given to
// each node and a mask on the in-batch attention that follows the tree.  The preparation
// kernel turns parent_idx into exactly those two things (a position per node and an
// ancestor-or-self bit mask per node) plus the children lists the acceptance walk follows.
#include "ssd_internal.h"

// One CTA, one thread per node.  parent[i] < i is guaranteed by the host check, so walking up
// from a node terminates after depth(i) steps.
__global__ void __launch_bounds__(SSD_MAX_NODES) tree_prep_kernel(NodeList tokens, NodeList parent, StepInfo step, TreeMeta m, StepInfo *info_out) {
    const int n = step.n, kv_len = step.kv_len;
    if (threadIdx.x == 0) *info_out = step;
    __shared__ int s_parent[SSD_MAX_NODES];
    __shared__ int s_count[SSD_MAX_NODES + 1];
    const int i = threadIdx.x;
    if (i < n) s_parent[i] = parent.v[i];
    s_count[i] = 0;
    if (i == 0) s_count[SSD_MAX_NODES] = 0;
    __syncthreads();
    if (i < n) {
        uint64_t mask[SSD_ANC_WORDS] = {0, 0, 0, 0};
        int depth = 0;
        for (int j = i; j >= 0; j = s_parent[j]) {
            mask[j >> 6] |= 1ull << (j & 63);
            if (j != i) ++depth;
        }
        m.tokens[i] = tokens.v[i];
        m.parent[i] = s_parent[i];
        m.depth[i] = depth;
        m.pos[i] = kv_len + depth;
#pragma unroll
        for (int w = 0; w < SSD_ANC_WORDS; ++w) m.anc[i * SSD_ANC_WORDS + w] = mask[w];
        // children of node i, ascending index; count first
        int c = 0;
        for (int j = i + 1; j < n; ++j) c += (s_parent[j] == i);
        s_count[i] = c;
    }
    __syncthreads();
    if (i == 0) { // n <= 256: a serial exclusive scan is a few hundred cycles
        int run = 0;
        for (int j = 0; j < n; ++j) {
            int c = s_count[j];
            s_count[j] = run;
            run += c;
        }
        s_count[n] = run;
    }
    __syncthreads();
    if (i < n) {
        int at = s_count[i];
        m.child_off[i] = at;
        for (int j = i + 1; j < n; ++j)
            if (s_parent[j] == i) m.child[at++] = j;
        if (i == 0) m.child_off[n] = s_count[n];
    }
}

cudaError_t launch_tree_prep(const NodeList &tokens, const NodeList &parent, const StepInfo &step, TreeMeta m, StepInfo *info_out,
                             cudaStream_t s) {
    tree_prep_kernel<<<1, SSD_MAX_NODES, 0, s>>>(tokens, parent, step, m, info_out);
    return cudaGetLastError();
}
const void *tree_prep_kernel_address() { return (const void *)tree_prep_kernel; }

__device__ __forceinline__ float block_sum_256(float v, float *red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads(); // protects `red` between two calls
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) t += red[w];
    return t;
}

// x[i, :] = wte[token_i, :] + wpe[pos_i, :]
template <typename WT>
__global__ void embed_kernel(const WT *__restrict__ wte, const WT *__restrict__ wpe, TreeMeta m, int d, float *__restrict__ x) {
    const int i = blockIdx.x;
    const WT *te = wte + (size_t)m.tokens[i] * d;
    const WT *pe = wpe + (size_t)m.pos[i] * d;
    for (int k = threadIdx.x; k < d; k += blockDim.x) x[(size_t)i * d + k] = (float)te[k] + (float)pe[k];
}

// Embedding for the cluster-reduced tensor-core path: x, the bf16 hi/lo planes of x * gain (operand of the first
// QKV projection, whose LayerNorm is folded into its epilogue) and the row's (sum, sum of squares) as part 0 of the
// statistics.  One CTA per row.
__global__ void __launch_bounds__(256) embed_planes_kernel(const __nv_bfloat16 *__restrict__ wte, const __nv_bfloat16 *__restrict__ wpe, TreeMeta m,
                                                           int d, const float *__restrict__ gain, float *__restrict__ x,
                                                           __nv_bfloat16 *__restrict__ plane_hi, __nv_bfloat16 *__restrict__ plane_lo,
                                                           float *__restrict__ stats) {
    __shared__ float red[8];
    const int i = blockIdx.x;
    const __nv_bfloat16 *te = wte + (size_t)m.tokens[i] * d;
    const __nv_bfloat16 *pe = wpe + (size_t)m.pos[i] * d;
    float s1 = 0.f, s2 = 0.f;
    for (int k = threadIdx.x; k < d; k += 256) {
        const float v = __bfloat162float(te[k]) + __bfloat162float(pe[k]);
        x[(size_t)i * d + k] = v;
        s1 += v;
        s2 += v * v;
        const float a = v * gain[k];
        const __nv_bfloat16 h = __float2bfloat16_rn(a);
        plane_hi[(size_t)i * d + k] = h;
        if (plane_lo) plane_lo[(size_t)i * d + k] = __float2bfloat16_rn(a - __bfloat162float(h));
    }
    s1 = block_sum_256(s1, red);
    s2 = block_sum_256(s2, red);
    if (threadIdx.x == 0) { stats[2 * i] = s1; stats[2 * i + 1] = s2; }
}

cudaError_t launch_embed_planes(const void *wte, const void *wpe, const TreeMeta &m, int n, int d, const float *gain, float *x, void *plane_hi,
                                void *plane_lo, float *stats, cudaStream_t s) {
    embed_planes_kernel<<<n, 256, 0, s>>>((const __nv_bfloat16 *)wte, (const __nv_bfloat16 *)wpe, m, d, gain, x, (__nv_bfloat16 *)plane_hi,
                                          (__nv_bfloat16 *)plane_lo, stats);
    return cudaGetLastError();
}

// logits[n, V] = 0 (the LM-head projection adds its stream-K partial sums into them).  Launched at the start of a
// forward, as wide as the GPU, so that the clearing is off the path between the last layer and the LM head.
__global__ void __launch_bounds__(256) zero_logits_kernel(const StepInfo *__restrict__ info, size_t count) {
    float *dst = info->logits; // (written by the tree-preparation kernel, which precedes this one in the stream)
    const size_t stride = (size_t)gridDim.x * blockDim.x, count4 = (reinterpret_cast<uintptr_t>(dst) & 15) == 0 ? count / 4 : 0;
    float4 *d4 = reinterpret_cast<float4 *>(dst);
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < count4; e += stride) d4[e] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (size_t e = 4 * count4 + (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < count; e += stride) dst[e] = 0.f;
}
cudaError_t launch_zero_logits(const StepInfo *info, int n, int vocab, cudaStream_t s) {
    zero_logits_kernel<<<148 * 4, 256, 0, s>>>(info, (size_t)n * vocab);
    return cudaGetLastError();
}

cudaError_t launch_embed(const void *wte, const void *wpe, int dtype, const TreeMeta &m, int n, int d, float *x, cudaStream_t s) {
    if (dtype == SSD_DTYPE_F32)
        embed_kernel<float><<<n, 256, 0, s>>>((const float *)wte, (const float *)wpe, m, d, x);
    else
        embed_kernel<__nv_bfloat16><<<n, 256, 0, s>>>((const __nv_bfloat16 *)wte, (const __nv_bfloat16 *)wpe, m, d, x);
    return cudaGetLastError();
}

// out[i, :] = (x[i, :] - mean) * rsqrt(var + eps) * g + b ; one CTA of 256 threads per row,
// mean first, then the variance of the centred values.
__global__ void __launch_bounds__(256) layernorm_kernel(const float *__restrict__ x, const float *__restrict__ g,
                                                        const float *__restrict__ b, int d, float eps, float *__restrict__ out) {
    __shared__ float red[8];
    const float *xr = x + (size_t)blockIdx.x * d;
    float s = 0.f;
    for (int k = threadIdx.x; k < d; k += 256) s += xr[k];
    const float mean = block_sum_256(s, red) / d;
    float v = 0.f;
    for (int k = threadIdx.x; k < d; k += 256) {
        float c = xr[k] - mean;
        v += c * c;
    }
    const float rstd = 1.0f / sqrtf(block_sum_256(v, red) / d + eps);
    for (int k = threadIdx.x; k < d; k += 256) out[(size_t)blockIdx.x * d + k] = (xr[k] - mean) * rstd * g[k] + b[k];
}

cudaError_t launch_layernorm(const float *x, const float *g, const float *b, int n, int d, float eps, float *out, cudaStream_t s) {
    layernorm_kernel<<<n, 256, 0, s>>>(x, g, b, d, eps, out);
    return cudaGetLastError();
}
