// Tree-masked attention for one layer (Section 3.1 of the paper).
//
// A node's keys are the kv_len committed cache rows, taken without a mask (the part the
// paper calls cross-attention with the cache), and the tree nodes that are its ancestors or
// itself (the in-batch self-attention, masked by the tree); both parts go through ONE softmax.
// The nodes' own K/V rows are written to scratch slots kv_len + i of the cache, apart from
// the committed rows; the tree part of the attention reads the fp32 projections directly.
//
// Layout: qkv [n, 3d] fp32, row i = q | k | v of node i, each head-major (64 per head).
//         cache K and V of this layer: [H, cap, 64], float or bf16.
// Grid (H, node groups); one warp per node at a time.  Pass 1: lanes over keys (each lane one
// whole key row), scores to shared memory, warp max/sum.  Pass 2: lanes over the 64 output
// dimensions (2 each), loop over keys reading V rows coalesced.
#include "sm100_ptx.cuh"
#include "ssd_internal.h"

namespace {
constexpr int WARPS = 4;
constexpr int DH = 64;

__device__ __forceinline__ void load_row64(const float *p, float (&r)[DH]) {
    const float4 *p4 = reinterpret_cast<const float4 *>(p);
#pragma unroll
    for (int t = 0; t < DH / 4; ++t) {
        float4 v = p4[t];
        r[4 * t] = v.x; r[4 * t + 1] = v.y; r[4 * t + 2] = v.z; r[4 * t + 3] = v.w;
    }
}
__device__ __forceinline__ void load_row64(const __nv_bfloat16 *p, float (&r)[DH]) {
    const uint4 *p4 = reinterpret_cast<const uint4 *>(p);
#pragma unroll
    for (int t = 0; t < DH / 8; ++t) {
        uint4 v = p4[t];
        const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&v);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            float2 f = __bfloat1622float2(h[u]);
            r[8 * t + 2 * u] = f.x; r[8 * t + 2 * u + 1] = f.y;
        }
    }
}
__device__ __forceinline__ float2 load_pair(const float *p) { return *reinterpret_cast<const float2 *>(p); }
__device__ __forceinline__ float2 load_pair(const __nv_bfloat16 *p) {
    return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(p));
}
__device__ __forceinline__ void store_elem(float *p, float v) { *p = v; }
__device__ __forceinline__ void store_elem(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

template <typename KVT>
__global__ void __launch_bounds__(WARPS * 32) tree_attention_kernel(const float *__restrict__ qkv, const StepInfo *__restrict__ info,
                                                                   size_t layer_offset, TreeMeta m, int n, int d,
                                                                   int cap, int nodes_per_cta, float *__restrict__ o,
                                                                   __nv_bfloat16 *__restrict__ o_hi, __nv_bfloat16 *__restrict__ o_lo) {
    extern __shared__ float smem[];
    ptx::pdl_launch_dependents();
    ptx::pdl_grid_wait();
    const int h = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kv_len = info->kv_len;
    KVT *kcache = reinterpret_cast<KVT *>(info->kbase) + layer_offset;
    KVT *vcache = reinterpret_cast<KVT *>(info->vbase) + layer_offset;
    const int n_keys = kv_len + n;
    float *s_q = smem + warp * DH;                    // [WARPS][64]
    float *s_sc = smem + WARPS * DH + warp * n_keys;  // [WARPS][n_keys]
    KVT *kh = kcache + (size_t)h * cap * DH;
    KVT *vh = vcache + (size_t)h * cap * DH;

    // The first node group of each head also stores the batch's K/V rows in the scratch slots.
    if (blockIdx.y == 0) {
        for (int e = threadIdx.x; e < n * DH; e += WARPS * 32) {
            const int i = e / DH, t = e % DH;
            store_elem(kh + (size_t)(kv_len + i) * DH + t, qkv[(size_t)i * 3 * d + d + h * DH + t]);
            store_elem(vh + (size_t)(kv_len + i) * DH + t, qkv[(size_t)i * 3 * d + 2 * d + h * DH + t]);
        }
    }

    const int i_begin = blockIdx.y * nodes_per_cta;
    const int i_end = min(n, i_begin + nodes_per_cta);
    for (int i = i_begin + warp; i < i_end; i += WARPS) {
        // query row to shared memory (every lane needs all 64 values)
        s_q[lane] = qkv[(size_t)i * 3 * d + h * DH + lane];
        s_q[lane + 32] = qkv[(size_t)i * 3 * d + h * DH + lane + 32];
        __syncwarp();
        uint64_t anc[SSD_ANC_WORDS];
#pragma unroll
        for (int w = 0; w < SSD_ANC_WORDS; ++w) anc[w] = m.anc[i * SSD_ANC_WORDS + w];

        // pass 1: scores
        float mx = -INFINITY;
        for (int j = lane; j < n_keys; j += 32) {
            float sc = -INFINITY;
            bool live = true;
            float kr[DH];
            if (j < kv_len) {
                load_row64(kh + (size_t)j * DH, kr);
            } else {
                const int t = j - kv_len;
                live = (anc[t >> 6] >> (t & 63)) & 1ull;
                if (live) load_row64(qkv + (size_t)t * 3 * d + d + h * DH, kr);
            }
            if (live) {
                float acc = 0.f;
#pragma unroll
                for (int t = 0; t < DH; ++t) acc = fmaf(s_q[t], kr[t], acc);
                sc = acc * 0.125f; // 1/sqrt(64)
            }
            s_sc[j] = sc;
            mx = fmaxf(mx, sc);
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
        float den = 0.f;
        for (int j = lane; j < n_keys; j += 32) {
            const float e = (s_sc[j] == -INFINITY) ? 0.f : expf(s_sc[j] - mx);
            s_sc[j] = e;
            den += e;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) den += __shfl_xor_sync(0xffffffffu, den, off);
        __syncwarp();

        // pass 2: weighted sum of values; lane owns dimensions 2*lane, 2*lane+1
        float2 acc = make_float2(0.f, 0.f);
        for (int j = 0; j < kv_len; ++j) {
            const float p = s_sc[j];
            const float2 v = load_pair(vh + (size_t)j * DH + 2 * lane);
            acc.x = fmaf(p, v.x, acc.x);
            acc.y = fmaf(p, v.y, acc.y);
        }
        for (int t = 0; t < n; ++t) {
            const float p = s_sc[kv_len + t];
            if (p != 0.f) {
                const float2 v = load_pair(qkv + (size_t)t * 3 * d + 2 * d + h * DH + 2 * lane);
                acc.x = fmaf(p, v.x, acc.x);
                acc.y = fmaf(p, v.y, acc.y);
            }
        }
        const float inv = 1.0f / den;
        const float ox = acc.x * inv, oy = acc.y * inv;
        const size_t at = (size_t)i * d + h * DH + 2 * lane;
        if (o_hi) { // bf16 operand planes for the tensor-core output projection
            const __nv_bfloat162 hi = __floats2bfloat162_rn(ox, oy);
            *reinterpret_cast<__nv_bfloat162 *>(o_hi + at) = hi;
            if (o_lo) *reinterpret_cast<__nv_bfloat162 *>(o_lo + at) = __floats2bfloat162_rn(ox - __low2float(hi), oy - __high2float(hi));
        } else {
            *reinterpret_cast<float2 *>(o + at) = make_float2(ox, oy);
        }
        __syncwarp();
    }
}
} // namespace

// Shared memory of one CTA for key lists of up to max_keys entries (it must fit the 48 KB a kernel gets without opting in to more).
size_t tree_attention_smem(int max_keys) { return sizeof(float) * (WARPS * DH + (size_t)WARPS * max_keys); }

cudaError_t launch_tree_attention(const float *qkv, const StepInfo *info, size_t layer_offset_elems, int dtype, const TreeMeta &m, int n,
                                  int max_keys, int n_head, int cap, float *o, __nv_bfloat16 *o_hi, __nv_bfloat16 *o_lo, bool pdl,
                                  cudaStream_t s) {
    const int d = n_head * DH;
    // enough node groups to fill the machine, at least one node per warp
    int groups = (n + WARPS - 1) / WARPS;
    const int want = (148 * 4 + n_head - 1) / n_head;
    if (groups > want) groups = want;
    const int per = (n + groups - 1) / groups;
    groups = (n + per - 1) / per;
    // shared memory is sized for the longest key list the cache allows, so that one captured
    // launch serves every prefix length
    const size_t smem = tree_attention_smem(max_keys);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_head, groups);
    cfg.blockDim = dim3(WARPS * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    if (dtype == SSD_DTYPE_F32)
        return cudaLaunchKernelEx(&cfg, tree_attention_kernel<float>, qkv, info, layer_offset_elems, m, n, d, cap, per, o, o_hi, o_lo);
    return cudaLaunchKernelEx(&cfg, tree_attention_kernel<__nv_bfloat16>, qkv, info, layer_offset_elems, m, n, d, cap, per, o, o_hi, o_lo);
}
