// Stand-alone launch of the tree-masked attention work items (bf16 path): grid (heads, node tiles).
#include "attention_mma.cuh"

namespace {
template <bool LO>
__global__ void __maxnreg__(144)
tree_attention_mma_kernel(const float *__restrict__ qkv, const StepInfo *__restrict__ info, size_t layer_offset, TreeMeta meta, int n, int d,
                          int cap, __nv_bfloat16 *__restrict__ o_hi, __nv_bfloat16 *__restrict__ o_lo, unsigned long long *trace,
                          uint8_t *__restrict__ planes8, size_t plane_stride) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    if (threadIdx.x == 0) ptx::trace_mark(trace, 0);
    ptx::pdl_launch_dependents();
    attn::Output out = {o_hi, o_lo, nullptr, nullptr, 0, 0, planes8, plane_stride};
    // (the step's tree metadata and the committed cache rows were complete before the first dependent launch of the
    //  forward began, so the item reads them before it waits for the QKV projection)
    attn::work_item<attn::NW_MAX, true, true, LO>(threadIdx.x, 0, smem_raw, blockIdx.x, blockIdx.y * 16, 0, 1, blockIdx.y == 0, qkv, info, layer_offset, meta, n, d, cap, out, trace);
    if (trace) { __syncthreads(); if (threadIdx.x == 0) ptx::trace_mark(trace, 2); }
}
} // namespace

size_t tree_attention_mma_smem(int n) { return attn::smem_bytes(n); }

cudaError_t tree_attention_mma_prepare() {
    cudaError_t e = cudaFuncSetAttribute(tree_attention_mma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tree_attention_mma_smem(SSD_MAX_NODES));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(tree_attention_mma_kernel<true>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(tree_attention_mma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tree_attention_mma_smem(SSD_MAX_NODES));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(tree_attention_mma_kernel<false>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    return e;
}

cudaError_t launch_tree_attention_mma(const float *qkv, const StepInfo *info, size_t layer_offset_elems, const TreeMeta &m, int n, int n_head,
                                      int cap, __nv_bfloat16 *o_hi, __nv_bfloat16 *o_lo, bool pdl, cudaStream_t s, unsigned long long *trace, bool lo_pairs,
                                      uint8_t *planes8, size_t plane_stride) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_head, (n + 15) / 16);
    cfg.blockDim = dim3(attn::NW_MAX * 32);
    cfg.dynamicSmemBytes = tree_attention_mma_smem(n);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, lo_pairs ? tree_attention_mma_kernel<true> : tree_attention_mma_kernel<false>, qkv, info, layer_offset_elems, m, n, n_head * attn::DH, cap, o_hi, o_lo, trace, planes8, plane_stride);
}
