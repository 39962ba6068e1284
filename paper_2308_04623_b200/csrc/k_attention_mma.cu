// Stand-alone launch of the tree-masked attention work items (bf16 path): grid (heads, node tiles).
#include "attention_mma.cuh"

namespace {
// The tree's own K / V rows, fp32 in the QKV projection's output, as bf16 in the cache's scratch slots kv_len + j: K rows [cap, 64],
// V transposed [64, cap]; the slots from kv_len + n up to the next multiple of 16 are zeroed (the attention reads whole 16-key
// blocks and multiplies masked keys' V by zero weights).  One CTA of 128 threads per (head, 16 slots).
// V is written as 16-byte groups of eight consecutive slots of one dimension, aligned in the cache row: a group that begins below
// kv_len keeps the committed values it holds (read, merged, written back by the one thread that owns the group).
constexpr int NW_STAGED = 4; // warps of an attention CTA that reads every block from the cache: three such CTAs share an SM ...
// (six warps at 112 registers per thread, still three CTAs per SM, were measured much slower: 3210 against 2547 us per verify of 256 nodes)
constexpr int NW_STAGED_WIDE = 8; // ... or eight, two CTAs per SM, when that many slots hold all (head, node tile) items at once
__global__ void __launch_bounds__(128)
kv_stage_kernel(const float *__restrict__ qkv, const StepInfo *__restrict__ info, size_t layer_offset, int n, int d, int cap, unsigned long long *trace) {
    if (threadIdx.x == 0) ptx::trace_mark(trace, 0);
    ptx::pdl_launch_dependents();
    ptx::pdl_grid_wait();
    if (threadIdx.x == 0) ptx::trace_mark(trace, 1);
    const int h = blockIdx.x, P = info->kv_len, end = (P + n + 15) & ~15; // slots [P, end): tree rows, then zero padding
    __nv_bfloat16 *kc = reinterpret_cast<__nv_bfloat16 *>(info->kbase) + layer_offset + (size_t)h * cap * attn::DH;
    __nv_bfloat16 *vc = reinterpret_cast<__nv_bfloat16 *>(info->vbase) + layer_offset + (size_t)h * cap * attn::DH;
    { // K: thread -> (slot P + 16 y + t / 8, dims 8 (t % 8) .. + 7), one 16-byte store
        const int slot = P + blockIdx.y * 16 + (threadIdx.x >> 3), c = (threadIdx.x & 7) * 8, j = slot - P;
        if (slot < end) {
            uint4 kq = make_uint4(0u, 0u, 0u, 0u);
            if (j < n) {
                const float *kf = qkv + (size_t)j * 3 * d + d + h * attn::DH + c;
                const float4 k0 = __ldcg(reinterpret_cast<const float4 *>(kf)), k1 = __ldcg(reinterpret_cast<const float4 *>(kf + 4));
                kq.x = attn::pack_bf16(k0.x, k0.y); kq.y = attn::pack_bf16(k0.z, k0.w); kq.z = attn::pack_bf16(k1.x, k1.y); kq.w = attn::pack_bf16(k1.z, k1.w);
            }
            *reinterpret_cast<uint4 *>(kc + (size_t)slot * attn::DH + c) = kq;
        }
    }
    { // V: thread -> (dimension t % 64, the aligned group of eight slots number 2 y + t / 64 counted from kv_len rounded down to 8)
        const int c = threadIdx.x & 63, s0 = (P & ~7) + 8 * (2 * blockIdx.y + (threadIdx.x >> 6));
        if (s0 < end) {
            __nv_bfloat16 *dst = vc + (size_t)c * cap + s0;
            union { uint4 q; __nv_bfloat16 e[8]; } grp;
            grp.q = make_uint4(0u, 0u, 0u, 0u);
            if (s0 < P) grp.q = *reinterpret_cast<const uint4 *>(dst); // committed slots of the group stay as they are
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int j = s0 + i - P;
                if (j >= 0) grp.e[i] = __float2bfloat16_rn(j < n ? __ldcg(qkv + (size_t)j * 3 * d + 2 * d + h * attn::DH + c) : 0.f);
            }
            *reinterpret_cast<uint4 *>(dst) = grp.q;
        }
    }
    if (trace) { __syncthreads(); if (threadIdx.x == 0) ptx::trace_mark(trace, 2); }
}

// STAGED: 0 = the CTA converts and stages the tree's keys itself (NW_MAX warps); otherwise the warps of a CTA that reads them from the cache
template <bool LO, int STAGED>
__global__ void __maxnreg__((STAGED == NW_STAGED_WIDE ? 128 : 144))
tree_attention_mma_kernel(const float *__restrict__ qkv, const StepInfo *__restrict__ info, size_t layer_offset, TreeMeta meta, int n, int d,
                          int cap, __nv_bfloat16 *__restrict__ o_hi, __nv_bfloat16 *__restrict__ o_lo, unsigned long long *trace,
                          uint8_t *__restrict__ planes8, size_t plane_stride) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    if (threadIdx.x == 0) ptx::trace_mark(trace, 0);
    ptx::pdl_launch_dependents();
    // Long prefixes: gridDim.z CTAs - one thread-block cluster - share a (head, node tile), each with a contiguous part of the key
    // blocks; the last one holds the tree's own keys (and, for tile 0, writes them to the cache's scratch slots).
    const int splits = gridDim.z, split = blockIdx.z;
    attn::Output out = {o_hi, o_lo, nullptr, nullptr, 0, 0, splits > 1 ? 1 : 0, planes8, plane_stride};
    // (the step's tree metadata and the committed cache rows were complete before the first dependent launch of the
    //  forward began, so the item reads them before it waits for the QKV projection)
    attn::work_item<(STAGED ? STAGED : attn::NW_MAX), true, true, LO, (STAGED != 0)>(threadIdx.x, 0, smem_raw, blockIdx.x, blockIdx.y * 16, split, splits,
                                                                                 blockIdx.y == 0 && split == splits - 1, qkv, info, layer_offset, meta, n, d, cap, out, trace);
    if (trace) { __syncthreads(); if (threadIdx.x == 0) ptx::trace_mark(trace, 2); }
}
} // namespace

size_t tree_attention_mma_smem(int n) { return attn::smem_bytes(n); }

cudaError_t tree_attention_mma_prepare() {
    cudaError_t e = cudaSuccess;
    const void *kernels[] = {(const void *)tree_attention_mma_kernel<true, 0>, (const void *)tree_attention_mma_kernel<false, 0>,
                             (const void *)tree_attention_mma_kernel<true, NW_STAGED>, (const void *)tree_attention_mma_kernel<false, NW_STAGED>,
                             (const void *)tree_attention_mma_kernel<true, NW_STAGED_WIDE>, (const void *)tree_attention_mma_kernel<false, NW_STAGED_WIDE>};
    for (const void *k : kernels) {
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)attn::smem_bytes(SSD_MAX_NODES, attn::NW_MAX, false, 8));
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    }
    if (e == cudaSuccess) e = cudaFuncSetAttribute(kv_stage_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    return e;
}

cudaError_t launch_kv_stage(const float *qkv, const StepInfo *info, size_t layer_offset_elems, int n, int n_head, int cap, bool pdl, cudaStream_t s,
                            unsigned long long *trace) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_head, (n + 15 + 15) / 16 + 1); // (up to 15 slots of padding behind the tree and 7 committed ones in front of it)
    cfg.blockDim = dim3(128);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kv_stage_kernel, qkv, info, layer_offset_elems, n, n_head * attn::DH, cap, trace);
}

cudaError_t launch_tree_attention_mma(const float *qkv, const StepInfo *info, size_t layer_offset_elems, const TreeMeta &m, int n, int n_head,
                                      int cap, __nv_bfloat16 *o_hi, __nv_bfloat16 *o_lo, bool pdl, cudaStream_t s, unsigned long long *trace, bool lo_pairs,
                                      uint8_t *planes8, size_t plane_stride, int staged_warps, int splits) {
    const bool staged = staged_warps != 0;
    if (splits < 1 || splits > 8 || (staged && splits != 1)) return cudaErrorInvalidValue;
    if (staged && staged_warps != NW_STAGED && staged_warps != NW_STAGED_WIDE) return cudaErrorInvalidValue;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_head, (n + 15) / 16, splits);
    const int nw = staged ? staged_warps : attn::NW_MAX;
    cfg.blockDim = dim3(nw * 32);
    cfg.dynamicSmemBytes = attn::smem_bytes(n, nw, staged, splits);
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (pdl) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    if (splits > 1) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = 1; attr[na].val.clusterDim.y = 1; attr[na].val.clusterDim.z = (unsigned)splits;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    auto kernel = nw == NW_STAGED_WIDE ? (lo_pairs ? tree_attention_mma_kernel<true, NW_STAGED_WIDE> : tree_attention_mma_kernel<false, NW_STAGED_WIDE>)
                  : staged         ? (lo_pairs ? tree_attention_mma_kernel<true, NW_STAGED> : tree_attention_mma_kernel<false, NW_STAGED>)
                                   : (lo_pairs ? tree_attention_mma_kernel<true, 0> : tree_attention_mma_kernel<false, 0>);
    return cudaLaunchKernelEx(&cfg, kernel, qkv, info, layer_offset_elems, m, n, n_head * attn::DH, cap, o_hi, o_lo, trace, planes8, plane_stride);
}
