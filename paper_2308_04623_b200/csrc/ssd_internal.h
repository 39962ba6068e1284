// Internal declarations shared by the translation units of libssd (not installed).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ssd.h"

#define SSD_MAX_NODES 256
#define SSD_ANC_WORDS 4 /* 256 nodes / 64 bits */
#define SSD_TRACE_SLOTS 4096 /* timeline buffer: eight 64-bit stamps per launch */

// Small host arrays travel to the device as kernel arguments: no staging buffer, no copy to
// wait for, and the call may return before the kernel runs.
struct NodeList {
    int32_t v[SSD_MAX_NODES];
};

// Per-tree device metadata written by the tree-preparation kernel.
struct TreeMeta {
    int32_t *tokens;    // [max_nodes]
    int32_t *parent;    // [max_nodes]
    int32_t *depth;     // [max_nodes]
    int32_t *pos;       // [max_nodes] kv_len + depth
    uint64_t *anc;      // [max_nodes, SSD_ANC_WORDS] ancestor-or-self bit masks
    int32_t *child_off; // [max_nodes + 1] CSR offsets
    int32_t *child;     // [max_nodes] children in ascending node index
};

// Per-step values every kernel of a forward reads from device memory, so that one captured
// CUDA graph serves every step: only the tree-preparation node's arguments change.
struct StepInfo {
    int32_t n, kv_len;
    void *kbase, *vbase; // cache of the sequence being verified: [n_layer, n_head, cap, 64]
    float *logits;       // caller's [n, vocab] output
};

struct LayerWeights {
    const float *ln1_g, *ln1_b, *b_qkv, *b_o, *ln2_g, *ln2_b, *b_fc, *b_proj; // fp32 on device
    const void *w_qkv, *w_o, *w_fc, *w_proj;                                  // float or bf16; e4m3 codes when the weights are 8-bit
    const float *s_qkv, *s_o, *s_fc, *s_proj;                                 // 8-bit weights: one scale per output row
};

enum GemmEpilogue { EPI_STORE = 0, EPI_GELU = 1, EPI_RESIDUAL = 2 };

// ---- launchers (each enqueues on `s` and returns the launch status) ----------------------
cudaError_t launch_tree_prep(const NodeList &tokens, const NodeList &parent, const StepInfo &step, TreeMeta m, StepInfo *info_out,
                             cudaStream_t s);
// Address of the tree-preparation kernel (to find its node in a captured graph) and a helper that
// fills the argument array of that node.
const void *tree_prep_kernel_address();
cudaError_t launch_embed(const void *wte, const void *wpe, int dtype, const TreeMeta &m, int n, int d, float *x, cudaStream_t s);
cudaError_t launch_zero_logits(const StepInfo *info, int n, int vocab, cudaStream_t s);
cudaError_t launch_layernorm(const float *x, const float *g, const float *b, int n, int d, float eps, float *out, cudaStream_t s);
// y[n, out] (+)= epilogue(a[n, K] . W[out, K]^T + bias)
cudaError_t launch_gemm_simple(const float *a, const void *W, int dtype, const float *bias, int n, int K, int out, int epilogue,
                               float *y, cudaStream_t s);
// Tree attention for one layer.  qkv: [n, 3d] fp32 (bias included).  kcache/vcache: this layer's
// [H, cap, 64] rows (float or bf16).  Writes the nodes' K/V to slots kv_len + i and o[n, d].
size_t tree_attention_smem(int max_keys);
cudaError_t launch_tree_attention(const float *qkv, const StepInfo *info, size_t layer_offset_elems, int dtype, const TreeMeta &m, int n,
                                  int max_keys, int n_head, int cap, float *o, __nv_bfloat16 *o_hi, __nv_bfloat16 *o_lo, bool pdl,
                                  cudaStream_t s);

// ---- bf16 tensor-core path --------------------------------------------------------------
// LayerNorm of n rows into bf16 hi/lo planes [n, d]; optionally zeroes zero[n, zero_cols].
// `zero` may be null; if zero_from_info is set the zeroed buffer is info->logits instead.
cudaError_t launch_ln_prep(const float *x, const float *g, const float *b, int n, int d, float eps, __nv_bfloat16 *a_hi, __nv_bfloat16 *a_lo,
                           float *zero, int zero_cols, const StepInfo *info, int zero_from_info, bool pdl, cudaStream_t s,
                           unsigned long long *trace = nullptr, uint8_t *planes8 = nullptr, size_t plane_stride = 0);
cudaError_t launch_gelu_prep(const float *acc, int n, int F, __nv_bfloat16 *h_hi, __nv_bfloat16 *h_lo, bool pdl, cudaStream_t s,
                             unsigned long long *trace = nullptr, uint8_t *planes8 = nullptr, size_t plane_stride = 0);
// (planes8, where a launcher takes it: instead of the bf16 planes write the four e4m3 planes [4][rows][K] the 8-bit projections
//  read, plane_stride = rows * K bytes apart; see w8_planes.cuh)
// (`trace`, where a launcher takes it: eight timestamp slots of this launch, see ptx::trace_mark; null = off)
// Tensor maps are opaque 128-byte objects (CUtensorMap) built on the host.
struct alignas(64) TensorMap { unsigned char bytes[128]; };
int make_tensor_map_bf16(void *map_out, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows);
int make_tensor_map_bf16_pair(void *map_out, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows);
int make_tensor_map_u8(void *map_out, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows);
int make_tensor_map_f32(void *map_out, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows); // boxes of [box_rows, 64], not swizzled
int make_tensor_map_u8_planes(void *map_out, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows, uint32_t box_planes);
// 8-bit weights: W[rows, cols] bf16 -> e4m3 codes [rows, cols] and one power-of-two scale per row, the smallest that brings the
// row's largest magnitude within the format's range (448); code = round-to-nearest-even(W / scale).  A row of zeros gets scale 1.
cudaError_t launch_quantise_rows_e4m3(const void *w_bf16, size_t rows, size_t cols, uint8_t *codes, float *scales, cudaStream_t s);
cudaError_t gemm_ws_prepare();
cudaError_t prep_kernels_prepare();
// y[n, ldy] += X[n, K] . W[out, K]^T (+ bias once).  map_w: weights [out, K], boxes of 128 rows; map_hi: the activations' hi plane
// [rows >= n_pad, K], ONE box of n_pad rows; map_lo: with use_lo, the hi AND lo planes as one 3-D map (make_tensor_map_bf16_pair:
// the lo plane follows the hi plane in memory), one box of [2][n_pad][64]; may be null when use_lo = 0.
// If y is null the destination is info->logits.  `grid` CTAs share the units; with grid > sm_count each takes at most
// half an SM's shared memory.
// With `head` set the projection runs one CTA per output tile over the whole K (complete sums): plain stores, no clearing of Y
// needed, and per (row, tile) the maximum, its lowest feature index and a non-finite flag at [row * n_tiles + tile].
// With `w_scale` set the weights are 8-bit codes (map_w from make_tensor_map_u8, w_scale[out] their per-row scales) and the
// activations e4m3 planes, the first w8_planes of the four (map_hi from make_tensor_map_u8_planes with that many planes per box;
// map_lo unused); n <= 128 rows per launch, the rows
// row0 .. row0 + n - 1 of the planes and of y; K need not be a multiple of 128; `head` is not supported.
// With group_rows > 0 (a multiple of 16) and less than n, the nodes are cut into groups of that many and the grid is one copy of
// the CTA arrangement per group (`grid` is the whole launch's CTA count); the maps' boxes then hold group_rows rows.  bf16 only.
// With act_gelu the activations are X = gelu(S), S the fp32 matrix [rows, K] behind map_hi (make_tensor_map_f32; map_lo unused):
// the kernel makes the hi / lo planes itself, with the arithmetic of launch_gelu_prep.  Needs use_lo, at most 64 rows (per
// group) and at least as many CTAs as output tiles; bf16 weights only.
struct GemmHeadStats { float *val; int32_t *arg, *bad; };
cudaError_t launch_gemm_ws(const void *map_w, const void *map_hi, const void *map_lo, float *y, const StepInfo *info, int ldy,
                           const float *bias, int n, int K, int out, int use_lo, int grid, int sm_count, int32_t *status, bool pdl,
                           cudaStream_t s, unsigned long long *trace = nullptr, const GemmHeadStats *head = nullptr,
                           const float *w_scale = nullptr, int row0 = 0, int w8_planes = 4, int group_rows = 0, int act_gelu = 0);
// ---- projection with the split-K sums reduced inside a thread-block cluster (trees of up to 64 nodes) ----
// What the epilogue does with the finished sums acc[i, o] (see k_gemm_cl.cu):
enum { MODE_FOLD_STORE = 0, MODE_FOLD_GELU = 1, MODE_RESIDUAL = 2 };
struct GemmClEpilogue {
    int mode;
    // MODE_FOLD_*: statistics of the LayerNorm in front of the projection as `stats_parts` partial
    // (sum, sum of squares) pairs per row, [part][SSD_MAX_NODES][2]; c1 = W gain, c2 = W beta + bias
    const float *stats_in;
    int stats_parts;
    const float *c1, *c2;
    float inv_d, eps;
    float *y;               // MODE_FOLD_STORE: output [n, ldy]; MODE_RESIDUAL: the residual stream, updated in place
    int ldy;
    const float *bias;      // MODE_RESIDUAL
    const float *gain;      // MODE_RESIDUAL: gain of the next LayerNorm, planes = x * gain (null: no planes)
    __nv_bfloat16 *plane_hi, *plane_lo; // MODE_FOLD_GELU / MODE_RESIDUAL: bf16 operand planes [rows, plane_ld] of the next projection
    int plane_ld;
    float *stats_out;       // MODE_RESIDUAL: [output tile][SSD_MAX_NODES][2]
};
cudaError_t gemm_cl_prepare();
bool gemm_cl_supports(int n, int d_model);
int gemm_cl_n_pad(int n);
int gemm_cl_cluster_size(int n, int K, int out, int slots, int max_cluster);
cudaError_t launch_gemm_cl(const void *map_w, const void *map_hi, const void *map_lo, int n, int K, int out, int use_lo, int cluster,
                           bool two_per_sm, const GemmClEpilogue &ep, int32_t *status, bool pdl, cudaStream_t s,
                           unsigned long long *trace = nullptr);
// x = wte[token] + wpe[pos] with the bf16 hi/lo planes of x * gain and the rows' (sum, sum of squares) as statistics part 0
cudaError_t launch_embed_planes(const void *wte, const void *wpe, const TreeMeta &m, int n, int d, const float *gain, float *x, void *plane_hi,
                                void *plane_lo, float *stats, cudaStream_t s);
// c1[o] = sum_k g[k] W[o, k], c2[o] = sum_k beta[k] W[o, k] + bias[o] (bias may be null): the vectors that fold a LayerNorm into
// the projection behind it
cudaError_t launch_ln_fold(const void *W, const float *g, const float *beta, const float *bias, int out, int K, float *c1, float *c2, cudaStream_t s);

// Moves slot kv_len + path[j] -> kv_len + j for every layer, K and V, head.
// (bf16 caches keep V transposed, [H, 64, cap]; fp32 caches keep V like K, [H, cap, 64].)
cudaError_t launch_kv_commit(void *kbase, void *vbase, int dtype, int n_layer, int n_head, int cap, int kv_len, const NodeList &path,
                             int n_path, cudaStream_t s, int *launches);
cudaError_t launch_kv_read(const void *cache_layer, int dtype, int n_head, int cap, int slot0, int rows, int transposed, float *out,
                           cudaStream_t s);
// (splits > 1: that many CTAs - one thread-block cluster - share a (head, node tile), each taking a part of the key blocks; their
//  partial softmaxes are merged in the first one's shared memory.  Worth it for long prefixes.)
// bf16 path attention on mma.sync tiles; K cache [H, cap, 64], V cache transposed [H, 64, cap]; cap a multiple of 16.
size_t tree_attention_mma_smem(int n);
cudaError_t tree_attention_mma_prepare();
cudaError_t launch_tree_attention_mma(const float *qkv, const StepInfo *info, size_t layer_offset_elems, const TreeMeta &m, int n, int n_head,
                                      int cap, __nv_bfloat16 *o_hi, __nv_bfloat16 *o_lo, bool pdl, cudaStream_t s,
                                      unsigned long long *trace = nullptr, bool lo_pairs = true, uint8_t *planes8 = nullptr,
                                      size_t plane_stride = 0, int staged_warps = 0, int splits = 1); // staged_warps: 0, or 4 / 8 warps per CTA reading the tree's rows from the cache
// Writes the tree's K / V rows (bf16) to the cache's scratch slots and zeroes the rest of the last 16-key block; an attention launched
// with `staged` then reads every block from the cache and stages nothing itself (worth its launch for large trees).
cudaError_t launch_kv_stage(const float *qkv, const StepInfo *info, size_t layer_offset_elems, int n, int n_head, int cap, bool pdl, cudaStream_t s,
                            unsigned long long *trace = nullptr);

#define SSD_ACC_SUPPORT 1024
struct AcceptScratch {
    double *rows;       // [rows_cap, vocab] target distribution of every node, computed by one CTA per row before the walk
                        // (null or too small: the walk computes the visited rows itself, one after the other)
    int rows_cap;
    double *rows_alt;   // [rows_cap, vocab] a second row per node (a refusal writes the residual there in one pass), or null
    double *row_total;  // [rows_cap][8] the rows are unnormalised: the sums of the (up to eight) slices they were computed in
    int32_t *sup_idx;   // [rows_cap, SSD_ACC_SUPPORT] with a top-k cut: the indices a row's law is positive at, ascending
    int32_t *sup_cnt;   // [rows_cap] how many (-1: more than SSD_ACC_SUPPORT, the walk then scans the whole vocabulary)
    double *r;          // [vocab] residual distribution
    int arg_parts;      // parts a row's arg-max is computed in (greedy); 0 = 1
    float *row_val;     // [max_nodes * parts] per-part row maximum (greedy)
    int32_t *row_arg;   // [max_nodes * parts] per-part arg-max (greedy)
    int32_t *row_bad;   // [max_nodes * parts] 1 if the part holds a non-finite value (sampling: [max_nodes], per row)
    int32_t *result;    // [max_nodes + 4]: n_path, next_token, status, device error word, path[...]
    const int32_t *dev_status; // the forward's device error word (copied into result[3] by the walk) or null
    // sampling with the per-node scratch: proposal rows as index / value lists [n][sp_entries] (device) instead of dense rows; null = dense
    const int32_t *sp_idx;
    const float *sp_val;
    int sp_entries;
    // greedy: per (row, part) statistics already written by the LM head (parts = head_parts > 0): the arg-max pass is skipped
    int head_parts;
    const float *head_val;
    const int32_t *head_arg, *head_bad;
};
cudaError_t launch_propose_children(const float *logits, const NodeList &nodes, int m, int vocab, int mode, float temperature, int top_k, int picks,
                                    uint64_t seed, uint64_t step, double *scratch, double *row_total, int32_t *row_bad, float *rows_out,
                                    int32_t *tokens_out, int32_t *bad_out, cudaStream_t s);
cudaError_t launch_expand_sparse_rows(const int32_t *idx, const float *val, int n, int entries, int vocab, float *rows, cudaStream_t s);
cudaError_t launch_expired_wait(int32_t *status, long long limit_cycles, cudaStream_t s);
cudaError_t launch_accept(const float *logits, const float *draft_probs, const NodeList &tokens, const NodeList &parent, int n,
                          int vocab, int mode, float temperature, int top_k, uint64_t seed, uint64_t step,
                          const AcceptScratch &sc, cudaStream_t s, int *launches);
