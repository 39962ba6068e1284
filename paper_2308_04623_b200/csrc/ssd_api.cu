// C ABI of libssd: contexts, weights, caches and the three hot-path calls.
// Host code here only validates arguments and enqueues kernels; every step of the path runs
// on the device.
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "ssd_internal.h"

struct ssd_kv {
    ssd_ctx *ctx;
    void *k, *v;        // [n_layer, n_head, cap, 64] each, float or bf16
    int32_t cap, len;
    int32_t last_n;     // nodes of the last verified tree (0 = none pending)
    int32_t last_parent[SSD_MAX_NODES];
};

struct ssd_ctx {
    ssd_config cfg;
    int device;
    cudaStream_t stream;
    bool loaded;
    int last_cuda, last_cuda_line;
    int64_t launches;
    size_t elt; // bytes per weight / cache element
    // weights
    void *wte, *wpe;
    float *lnf_g, *lnf_b;
    std::vector<LayerWeights> layers;
    std::vector<void *> owned; // every device allocation of the context
    // workspaces
    TreeMeta meta;
    float *x, *a, *qkv, *o, *h;
    // bf16 tensor-core path: activation operand planes (hi / lo) and their tensor maps
    __nv_bfloat16 *a_hi, *a_lo, *o_hi, *o_lo, *h_hi, *h_lo;
    // activation planes as tensor maps whose box is the whole padded batch [n_pad rows x 64]: one TMA operation per
    // plane and k tile (index n_pad / 16 - 1; built on first use)
    struct ActMaps { TensorMap a_hi, a_lo, o_hi, o_lo, h_hi, h_lo, a_pair, o_pair, h_pair, h_src; bool built; }; // (_pair: hi and lo planes as one box)
    ActMaps act_maps[SSD_MAX_NODES / 16];
    size_t plane_rows;
    TensorMap map_wte;
    std::vector<TensorMap> map_layers; // 4 per layer: qkv, o, fc, proj
    bool tensor_path;                  // bf16 model: projections on tcgen05
    bool w8;                           // bf16 model whose five matrix families are held as e4m3 codes + per-row scales
    uint8_t *wte8;                     // w8: the output head's codes [vocab, d_model] (the embedding look-up keeps the bf16 table)
    float *wte_scale;
    int stage_kv_from;                 // trees of at least this many nodes write their K / V rows to the cache in a kernel of its own (0 = never)
    int w8_planes;                     // w8: how many of the four planes the projections use (the rest of a value is dropped)
    uint8_t *a8, *o8, *h8;             // w8: activation operands as four e4m3 planes [4][plane_rows][d_model or d_ff] (ActMaps then holds their
                                       // maps in a_hi / o_hi / h_hi)
    int use_lo, pdl, gemm_grid, head_grid, trace_kernels, trace_count, use_graph, use_cluster, cl_max, cl_size[4], attn_lo;
    // cluster-reduced path: per-layer vectors that fold a LayerNorm into the projection behind it (c1 = W gain,
    // c2 = W beta + bias), and the two row-statistics buffers [tile][SSD_MAX_NODES][2] (in front of QKV / of FC)
    struct LayerFold { float *c1_qkv, *c2_qkv, *c1_fc, *c2_fc; };
    std::vector<LayerFold> folds;
    float *d_stats1, *d_stats2;
    unsigned long long *d_trace;
    int sm_count;
    StepInfo *d_info;                  // device copy of the current step's values
    // One captured forward per tree size: the kernels read everything that changes from step to
    // step (prefix length, cache and output addresses) from d_info, and the tree itself travels
    // in the arguments of the first node, which are patched before each launch.
    struct ForwardGraph { cudaGraph_t graph; cudaGraphExec_t exec; cudaGraphNode_t prep_node; int kernels; };
    ForwardGraph graphs[SSD_MAX_NODES + 1][3]; // (second index: the attention's key splits, 1 / 2 / 4 - chosen from the prefix length at each call)
    int attn_splits;                           // 0 = choose; 1, 2, 4 = always that many
    int attn_staged_warps;                     // 0 = choose; 4 or 8: warps of the attention CTAs that read the tree's rows from the cache
    int fused_gelu;                            // the back-projection makes its gelu(.) operand planes itself (no separate kernel)
    int node_groups;                           // trees of more than 64 nodes: the layers' projections run on node groups of 64
    cudaStream_t capture_stream;
    AcceptScratch acc;
    int32_t *h_result; // pinned host copy of acc.result
    int32_t *h_propose; // pinned: picks of ssd_propose_children [SSD_MAX_NODES * 8] then one non-finite flag per listed node
    // proposal rows given as index / value lists: device copies of the lists and the dense rows they expand to (grown on demand)
    int32_t *d_sparse_idx;
    float *d_sparse_val, *d_sparse_rows;
    size_t sparse_entries_cap, sparse_rows_cap;
    int32_t *d_status;
    // per (row, output tile) statistics of the logits, written by the LM head (bf16 path), and which logits buffer they describe
    float *head_val;
    int32_t *head_arg, *head_bad;
    int head_tiles, use_head_stats;
    const float *head_logits;
    int head_n;
};

namespace {
struct DeviceGuard {
    int prev;
    bool ok;
    explicit DeviceGuard(int dev) : prev(-1), ok(false) {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = (prev == dev) || cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

int fail_cuda_at(ssd_ctx *ctx, cudaError_t e, int line) {
    if (ctx) { ctx->last_cuda = (int)e; ctx->last_cuda_line = line; }
    cudaGetLastError(); // clear the sticky-free error state so later calls are not blamed for it
    return e == cudaErrorMemoryAllocation ? SSD_ERR_NOMEM : SSD_ERR_CUDA;
}
#define fail_cuda(ctx, e) fail_cuda_at(ctx, e, __LINE__)
#define CU(call)                                           \
    do {                                                   \
        cudaError_t e__ = (call);                          \
        if (e__ != cudaSuccess) return fail_cuda(ctx, e__); \
    } while (0)

template <typename T>
int dev_alloc(ssd_ctx *ctx, T **p, size_t count) {
    void *q = nullptr;
    cudaError_t e = cudaMalloc(&q, count * sizeof(T) + 256);
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    ctx->owned.push_back(q);
    *p = (T *)q;
    return SSD_OK;
}

// Validate a tree on the host: structure, token range, and compute depths.
int check_tree(const ssd_config &c, const int32_t *tokens, const int32_t *parent, int n, int32_t *depth, int *max_depth) {
    if (n < 1 || n > c.max_nodes) return SSD_ERR_INVALID_TREE;
    if (parent[0] != -1) return SSD_ERR_INVALID_TREE;
    depth[0] = 0;
    int md = 0;
    for (int i = 1; i < n; ++i) {
        if (parent[i] < 0 || parent[i] >= i) return SSD_ERR_INVALID_TREE;
        depth[i] = depth[parent[i]] + 1;
        if (depth[i] > md) md = depth[i];
    }
    for (int i = 0; i < n; ++i)
        if (tokens[i] < 0 || tokens[i] >= c.vocab) return SSD_ERR_BAD_ARG;
    *max_depth = md;
    return SSD_OK;
}

// Copy a host tensor to a new device buffer; small vectors are widened to fp32.
int upload_matrix(ssd_ctx *ctx, const void *src, size_t count, void **dst) {
    if (!src) return SSD_ERR_BAD_ARG;
    unsigned char *p = nullptr;
    int rc = dev_alloc(ctx, &p, count * ctx->elt);
    if (rc != SSD_OK) return rc;
    CU(cudaMemcpyAsync(p, src, count * ctx->elt, cudaMemcpyHostToDevice, ctx->stream));
    *dst = p;
    return SSD_OK;
}
int upload_vector_f32(ssd_ctx *ctx, const void *src, size_t count, const float **dst, std::vector<float> &tmp) {
    if (!src) return SSD_ERR_BAD_ARG;
    float *p = nullptr;
    int rc = dev_alloc(ctx, &p, count);
    if (rc != SSD_OK) return rc;
    const float *host = (const float *)src;
    if (ctx->cfg.dtype == SSD_DTYPE_BF16) {
        tmp.resize(count);
        const uint16_t *b = (const uint16_t *)src;
        for (size_t i = 0; i < count; ++i) {
            uint32_t u = (uint32_t)b[i] << 16;
            memcpy(&tmp[i], &u, 4);
        }
        host = tmp.data();
        // tmp is reused by the next call: finish this copy first
        CU(cudaMemcpyAsync(p, host, count * sizeof(float), cudaMemcpyHostToDevice, ctx->stream));
        CU(cudaStreamSynchronize(ctx->stream));
    } else {
        CU(cudaMemcpyAsync(p, host, count * sizeof(float), cudaMemcpyHostToDevice, ctx->stream));
    }
    *dst = p;
    return SSD_OK;
}

static const ssd_ctx::ActMaps *act_maps_pad(ssd_ctx *ctx, int n_pad) {
    ssd_ctx::ActMaps &am = ctx->act_maps[n_pad / 16 - 1];
    if (!am.built) {
        const size_t d = ctx->cfg.d_model, F = ctx->cfg.d_ff, rows = ctx->plane_rows;
        if (ctx->w8) {
            int m8 = make_tensor_map_u8_planes(&am.a_hi, ctx->a8, rows, d, n_pad, ctx->w8_planes);
            if (m8 == SSD_OK) m8 = make_tensor_map_u8_planes(&am.o_hi, ctx->o8, rows, d, n_pad, ctx->w8_planes);
            if (m8 == SSD_OK) m8 = make_tensor_map_u8_planes(&am.h_hi, ctx->h8, rows, F, n_pad, ctx->w8_planes);
            if (m8 != SSD_OK) return nullptr;
            am.built = true;
            return &am;
        }
        int m = make_tensor_map_bf16(&am.a_hi, ctx->a_hi, rows, d, n_pad);
        if (m == SSD_OK) m = make_tensor_map_bf16(&am.a_lo, ctx->a_lo, rows, d, n_pad);
        if (m == SSD_OK) m = make_tensor_map_bf16(&am.o_hi, ctx->o_hi, rows, d, n_pad);
        if (m == SSD_OK) m = make_tensor_map_bf16(&am.o_lo, ctx->o_lo, rows, d, n_pad);
        if (m == SSD_OK) m = make_tensor_map_bf16(&am.h_hi, ctx->h_hi, rows, F, n_pad);
        if (m == SSD_OK) m = make_tensor_map_bf16(&am.h_lo, ctx->h_lo, rows, F, n_pad);
        if (m == SSD_OK) m = make_tensor_map_bf16_pair(&am.a_pair, ctx->a_hi, rows, d, n_pad);
        if (m == SSD_OK) m = make_tensor_map_bf16_pair(&am.o_pair, ctx->o_hi, rows, d, n_pad);
        if (m == SSD_OK) m = make_tensor_map_bf16_pair(&am.h_pair, ctx->h_hi, rows, F, n_pad);
        if (m == SSD_OK) m = make_tensor_map_f32(&am.h_src, ctx->h, ctx->cfg.max_nodes, F, n_pad); // (the feed-forward sums themselves)
        if (m != SSD_OK) return nullptr;
        am.built = true;
    }
    return &am;
}

static const ssd_ctx::ActMaps *act_maps_for(ssd_ctx *ctx, int n) { return act_maps_pad(ctx, (n + 15) & ~15); }

// CTAs per projection kernel.  Unless set by hand: two per SM while the tree is small enough for two CTAs' pipelines
// and accumulators to share an SM (measured: 1.63 ms against 1.88 ms per GPT-2-large verification of 32 nodes), else one.
static int gemm_grid_for(const ssd_ctx *ctx, int n) {
    if (ctx->gemm_grid > 0) return ctx->gemm_grid;
    return ((n + 15) & ~15) <= 64 ? 2 * ctx->sm_count : ctx->sm_count;
}
// (8-bit weights: four accumulator column groups per node; two CTAs' double-buffered accumulators fit an SM up to 32 nodes)
static int head_grid_for(const ssd_ctx *ctx, int n) {
    return ctx->head_grid > 0 ? ctx->head_grid : (ctx->w8 && n > 32) ? ctx->sm_count : gemm_grid_for(ctx, n);
}

// Timeline slots of the next launch (profiling aid, off by default).
static unsigned long long *trace_slot(ssd_ctx *ctx, int kernels) {
    return (ctx->trace_kernels && 8 * (kernels + 1) <= SSD_TRACE_SLOTS) ? ctx->d_trace + 8 * (size_t)kernels : nullptr;
}

// Enqueue every kernel of one tree-batched forward on `s`.
// Key splits of the attention for a step: a warp should have about two 16-key blocks; more CTAs per (head, node tile) only while
// they all fit the GPU at once, and not on the large-tree path.  Measured (verify, us): GPT-2-small shape, prefix 512, 8 nodes:
// 322 / 309 / 302 with 1 / 2 / 4 splits; GPT-2-XL shape, prefix 960, 8 nodes: 1993 / 1864 / 1705; prefix 512, 32 nodes: 1799 / 1763 /
// 1979 (200 CTAs: two waves); GPT-2-large shape, prefix 256, 32 nodes (18 key blocks): 1057 / 1096.
// Whether a tree's K / V rows go to the cache in a kernel of their own and the attention reads them from there: from
// SSD_TUNE_STAGE_KV_FROM nodes on, and - with 64 nodes or more - as soon as there are more (head, node tile) items than SMs
// (a CTA that stages the tree's rows itself has an SM to itself, so those items would run in two waves; measured at the
// GPT-2-XL shape, 96 nodes = 150 items: 2875 against 2990 us per verify).
static bool attn_staged(const ssd_ctx *ctx, int n) {
    if (ctx->stage_kv_from <= 0) return false;
    return n >= ctx->stage_kv_from || (n >= 64 && ctx->cfg.n_head * ((n + 15) / 16) > ctx->sm_count);
}
static int attn_splits_for(const ssd_ctx *ctx, int kv_len, int n) {
    const int tiles = (n + 15) / 16, ctas = ctx->cfg.n_head * tiles;
    const bool staged = attn_staged(ctx, n);
    int s = ctx->attn_splits;
    if (s == 0) {
        const int blocks = (kv_len + n + 15) / 16;
        s = blocks > 27 ? 4 : blocks > 19 ? 2 : 1;
    }
    while (s > 1 && (staged || ctas * s > ctx->sm_count)) s >>= 1; // (an attention CTA has an SM to itself: more CTAs than SMs run in waves)
    return s;
}

cudaError_t enqueue_forward(ssd_ctx *ctx, int n, int cap, const NodeList &tk, const NodeList &pr, const StepInfo &step, cudaStream_t s,
                            int *kernels, int attn_splits = 1) {
    const ssd_config &c = ctx->cfg;
    const int d = c.d_model, F = c.d_ff, max_keys = c.n_ctx + n;
    const size_t layer_elems = (size_t)c.n_head * cap * 64;
    const StepInfo *info = ctx->d_info;
    const ssd_ctx::ActMaps *am = ctx->tensor_path ? act_maps_for(ctx, n) : nullptr;
    if (ctx->tensor_path && !am) return cudaErrorUnknown;
    cudaError_t e;
#define Q(call) do { if ((e = (call)) != cudaSuccess) return e; ++*kernels; } while (0)
    Q(launch_tree_prep(tk, pr, step, ctx->meta, ctx->d_info, s));
    // The LM head either holds complete sums per CTA (plain stores, row statistics per tile) or adds stream-K partial sums
    // into logits cleared here, at the start of the forward.
    const GemmHeadStats head_stats = {ctx->head_val, ctx->head_arg, ctx->head_bad};
    const GemmHeadStats *head = (ctx->tensor_path && ctx->use_head_stats && !ctx->w8) ? &head_stats : nullptr;
    if (ctx->tensor_path && !head) Q(launch_zero_logits(info, n, c.vocab, s));
    if (ctx->tensor_path && ctx->use_cluster && !ctx->w8 && gemm_cl_supports(n, c.d_model)) {
        // bf16 model, trees of up to 64 nodes: five launches per layer.  Every projection reduces its split-K partial sums
        // inside a thread-block cluster, so its epilogue holds finished sums and does the work that would otherwise be
        // kernels of their own: the LayerNorms are folded (the projection runs on x * gain; mean, rstd and the precomputed
        // c1 = W gain, c2 = W beta + bias are applied to the sums), GELU is applied where the FC sums are complete, and the
        // residual additions write the next operand planes and the next LayerNorm's row statistics.
        const bool pdl = ctx->pdl != 0;
        const int lo = ctx->use_lo, sms = ctx->sm_count, L = c.n_layer, n_pad = gemm_cl_n_pad(n);
        const bool two = n_pad <= 32; // two CTAs' pipelines and reduction buffers fit one SM
        const ssd_ctx::ActMaps *amh = am; // (the LM head's operand box is the tree's own padded size)
        am = act_maps_pad(ctx, n_pad);
        if (!am) return cudaErrorUnknown;
        // (one SM's worth of CTAs per projection: the next projection's CTAs are resident beside them and prefetch their weights)
        const int slots = ctx->gemm_grid > 0 ? ctx->gemm_grid : sms, cmax = ctx->cl_max;
        const int tiles_d = (d + 127) / 128;
        auto pick = [&](int which, int K, int out) { // a cluster size set by hand is still cut down to one the kernel can run
            return ctx->cl_size[which] > 0 ? gemm_cl_cluster_size(n, K, out, 1 << 20, ctx->cl_size[which]) : gemm_cl_cluster_size(n, K, out, slots, cmax);
        };
        const int s_qkv = pick(0, d, 3 * d), s_o = pick(1, d, d), s_fc = pick(2, d, F), s_proj = pick(3, F, d);
        __nv_bfloat16 *a_lo = lo ? ctx->a_lo : nullptr, *o_lo = lo ? ctx->o_lo : nullptr, *h_lo = lo ? ctx->h_lo : nullptr;
        Q(launch_embed_planes(ctx->wte, ctx->wpe, ctx->meta, n, d, ctx->layers[0].ln1_g, ctx->x, ctx->a_hi, a_lo, ctx->d_stats1, s));
        for (int l = 0; l < L; ++l) {
            const LayerWeights &Lw = ctx->layers[l];
            const ssd_ctx::LayerFold &v = ctx->folds[l];
            const TensorMap *t = &ctx->map_layers[(size_t)4 * l];
            GemmClEpilogue eq = {};
            eq.mode = MODE_FOLD_STORE; eq.stats_in = ctx->d_stats1; eq.stats_parts = l == 0 ? 1 : tiles_d; eq.c1 = v.c1_qkv; eq.c2 = v.c2_qkv;
            eq.inv_d = 1.0f / d; eq.eps = c.ln_eps; eq.y = ctx->qkv; eq.ldy = 3 * d;
            Q(launch_gemm_cl(&t[0], &am->a_hi, &am->a_lo, n, d, 3 * d, lo, s_qkv, two, eq, ctx->d_status, pdl, s, trace_slot(ctx, *kernels)));
            Q(launch_tree_attention_mma(ctx->qkv, info, l * layer_elems, ctx->meta, n, c.n_head, cap, ctx->o_hi, o_lo, pdl, s, trace_slot(ctx, *kernels), ctx->attn_lo != 0));
            GemmClEpilogue eo = {};
            eo.mode = MODE_RESIDUAL; eo.y = ctx->x; eo.ldy = d; eo.bias = Lw.b_o; eo.gain = Lw.ln2_g; eo.plane_hi = ctx->a_hi; eo.plane_lo = a_lo;
            eo.plane_ld = d; eo.stats_out = ctx->d_stats2;
            Q(launch_gemm_cl(&t[1], &am->o_hi, &am->o_lo, n, d, d, lo, s_o, two, eo, ctx->d_status, pdl, s, trace_slot(ctx, *kernels)));
            GemmClEpilogue ef = {};
            ef.mode = MODE_FOLD_GELU; ef.stats_in = ctx->d_stats2; ef.stats_parts = tiles_d; ef.c1 = v.c1_fc; ef.c2 = v.c2_fc; ef.inv_d = 1.0f / d;
            ef.eps = c.ln_eps; ef.plane_hi = ctx->h_hi; ef.plane_lo = h_lo; ef.plane_ld = F;
            Q(launch_gemm_cl(&t[2], &am->a_hi, &am->a_lo, n, d, F, lo, s_fc, two, ef, ctx->d_status, pdl, s, trace_slot(ctx, *kernels)));
            GemmClEpilogue ep = {};
            ep.mode = MODE_RESIDUAL; ep.y = ctx->x; ep.ldy = d; ep.bias = Lw.b_proj; ep.gain = l + 1 < L ? ctx->layers[l + 1].ln1_g : nullptr;
            ep.plane_hi = ctx->a_hi; ep.plane_lo = a_lo; ep.plane_ld = d; ep.stats_out = ctx->d_stats1;
            Q(launch_gemm_cl(&t[3], &am->h_hi, &am->h_lo, n, F, d, lo, s_proj, two, ep, ctx->d_status, pdl, s, trace_slot(ctx, *kernels)));
        }
        const int hgrid = head_grid_for(ctx, n);
        Q(launch_ln_prep(ctx->x, ctx->lnf_g, ctx->lnf_b, n, d, c.ln_eps, ctx->a_hi, a_lo, nullptr, 0, info, 0, pdl, s, trace_slot(ctx, *kernels)));
        Q(launch_gemm_ws(&ctx->map_wte, &amh->a_hi, &amh->a_pair, nullptr, info, c.vocab, nullptr, n, d, c.vocab, lo, hgrid, sms, ctx->d_status, pdl, s, trace_slot(ctx, *kernels), head));
        ctx->trace_count = ctx->trace_kernels ? 8 * *kernels : 0;
        return cudaSuccess;
    }
    Q(launch_embed(ctx->wte, ctx->wpe, c.dtype, ctx->meta, n, d, ctx->x, s));
    if (ctx->tensor_path) {
        // bf16 model, the default path: LayerNorm / GELU kernels feed bf16 operand planes, projections
        // accumulate their stream-K partial sums into fp32 buffers; every kernel is a programmatic dependent launch.
        const bool pdl = ctx->pdl != 0;
        const int lo = ctx->use_lo, grid = gemm_grid_for(ctx, n), hgrid = head_grid_for(ctx, n), sms = ctx->sm_count;
        __nv_bfloat16 *a_lo = lo ? ctx->a_lo : nullptr, *o_lo = lo ? ctx->o_lo : nullptr, *h_lo = lo ? ctx->h_lo : nullptr;
        // Large trees: one small kernel per layer writes the tree's K / V rows to the cache's scratch slots and the attention reads
        // every key block from there, instead of each of a head's node tiles converting and staging the whole tree's keys itself.
        const bool staged = attn_staged(ctx, n);
        // (reading from the cache: eight warps per CTA - half as many key blocks per warp - if two such CTAs per SM hold every
        //  (head, node tile) item at once, else four, three CTAs per SM)
        const int attn_warps = !staged ? 0 : ctx->attn_staged_warps ? ctx->attn_staged_warps : c.n_head * ((n + 15) / 16) <= 2 * sms ? 8 : 4;
        if (ctx->w8) {
            // 8-bit weights: the same eight launches per layer; the element-wise kernels and the attention write four e4m3 planes,
            // the projections run on the 8-bit tensor-core kind.  A CTA takes at most 128 nodes (512 accumulator columns); trees of
            // more than 64 nodes run on node groups of 64 (256 columns: two CTAs per SM), like the bf16 model's large trees.
            const size_t rows = ctx->plane_rows, sa = rows * (size_t)d, sh = rows * (size_t)F;
            const int g8 = n > 64 ? 64 : 0;
            const ssd_ctx::ActMaps *m1 = g8 ? act_maps_pad(ctx, g8) : am;
            if (!m1) return cudaErrorUnknown;
            const int grid8 = g8 ? (ctx->gemm_grid > 0 ? ctx->gemm_grid : 2 * sms) : grid;
            auto gemm8 = [&](const TensorMap *w, const TensorMap ssd_ctx::ActMaps::*act, float *y, int ldy, const float *bias, int K, int out, int g,
                             const float *scale) -> cudaError_t {
                return launch_gemm_ws(w, &(m1->*act), nullptr, y, info, ldy, bias, n, K, out, 0, g, sms, ctx->d_status, pdl, s, trace_slot(ctx, *kernels), nullptr, scale, 0,
                                      ctx->w8_planes, g8);
            };
            for (int l = 0; l < c.n_layer; ++l) {
                const LayerWeights &L = ctx->layers[l];
                const TensorMap *t = &ctx->map_layers[(size_t)4 * l];
                Q(launch_ln_prep(ctx->x, L.ln1_g, L.ln1_b, n, d, c.ln_eps, nullptr, nullptr, ctx->qkv, 3 * d, info, 0, pdl, s, trace_slot(ctx, *kernels), ctx->a8, sa));
                Q(gemm8(&t[0], &ssd_ctx::ActMaps::a_hi, ctx->qkv, 3 * d, L.b_qkv, d, 3 * d, grid8, L.s_qkv));
                if (staged) Q(launch_kv_stage(ctx->qkv, info, l * layer_elems, n, c.n_head, cap, pdl, s, trace_slot(ctx, *kernels)));
                Q(launch_tree_attention_mma(ctx->qkv, info, l * layer_elems, ctx->meta, n, c.n_head, cap, nullptr, nullptr, pdl, s, trace_slot(ctx, *kernels), ctx->attn_lo != 0, ctx->o8, sa, attn_warps, attn_splits));
                Q(gemm8(&t[1], &ssd_ctx::ActMaps::o_hi, ctx->x, d, L.b_o, d, d, grid8, L.s_o));
                Q(launch_ln_prep(ctx->x, L.ln2_g, L.ln2_b, n, d, c.ln_eps, nullptr, nullptr, ctx->h, F, info, 0, pdl, s, trace_slot(ctx, *kernels), ctx->a8, sa));
                Q(gemm8(&t[2], &ssd_ctx::ActMaps::a_hi, ctx->h, F, L.b_fc, d, F, grid8, L.s_fc));
                Q(launch_gelu_prep(ctx->h, n, F, nullptr, nullptr, pdl, s, trace_slot(ctx, *kernels), ctx->h8, sh));
                Q(gemm8(&t[3], &ssd_ctx::ActMaps::h_hi, ctx->x, d, L.b_proj, F, d, grid8, L.s_proj));
            }
            Q(launch_ln_prep(ctx->x, ctx->lnf_g, ctx->lnf_b, n, d, c.ln_eps, nullptr, nullptr, nullptr, 0, info, 0, pdl, s, trace_slot(ctx, *kernels), ctx->a8, sa));
            Q(gemm8(&ctx->map_wte, &ssd_ctx::ActMaps::a_hi, nullptr, c.vocab, nullptr, d, c.vocab, hgrid, ctx->wte_scale));
            ctx->trace_count = ctx->trace_kernels ? 8 * *kernels : 0;
            return cudaSuccess;
        }
        // Trees of more than 128 nodes: the layers' projections work on node groups of 64 (the grid is one 64-node arrangement per
        // group, two CTAs per SM), with activation boxes of 64 rows.  Measured at the GPT-2-large shape (verify, us, without / with):
        // 96 nodes 1565 / 1562, 128 nodes 1903 / 1917, 192 nodes 2563 / 2206, 256 nodes 3180 / 2640.
        const int gr = (ctx->node_groups && n > 128) ? 64 : 0;
        const ssd_ctx::ActMaps *ag = gr ? act_maps_pad(ctx, gr) : am;
        if (!ag) return cudaErrorUnknown;
        const int lgrid = gr ? (ctx->gemm_grid > 0 ? ctx->gemm_grid : 2 * sms) : grid;
        // (the widest projection has so many output tiles that, times the groups of 64, every CTA would be left a tile's whole K -
        //  a long chain of dependent units: it takes groups of 128 instead; measured 2640 -> 2548 us per verify at 256 nodes)
        const int gr_fc = (gr && ((F + 127) / 128) * ((n + 63) / 64) > sms) ? 128 : gr;
        const ssd_ctx::ActMaps *af = gr_fc == gr ? ag : act_maps_pad(ctx, gr_fc);
        if (!af) return cudaErrorUnknown;
        // Opt-in: the back-projection reads the feed-forward sums and applies the GELU itself (the ACT instantiation of the kernel),
        // when it runs with both planes, on at most 64 rows per CTA and with at least one CTA per output tile.  Measured slower
        // (GPT-2-large shape, 32 nodes: 1166 against 1075 us per verify; 64 nodes 1459 / 1339; 256 nodes 2877 / 2541): every CTA of
        // the ten output tiles converts the same slice again - two special-function operations per value, 0.35-0.7 us per k tile on
        // one warp per scheduler, 3.9 us from dependencies to accumulator against 1.9 - and with no kernel between the two
        // feed-forward projections the second one's CTAs find room, and start their weight loads, only as the first one's leave.
        const int rows_cta = gr ? gr : (n + 15) & ~15;
        const bool fuse_gelu = ctx->fused_gelu && lo && rows_cta <= 64 && lgrid / (gr ? (n + gr - 1) / gr : 1) >= (d + 127) / 128;
        for (int l = 0; l < c.n_layer; ++l) {
            const LayerWeights &L = ctx->layers[l];
            const TensorMap *t = &ctx->map_layers[(size_t)4 * l];
            Q(launch_ln_prep(ctx->x, L.ln1_g, L.ln1_b, n, d, c.ln_eps, ctx->a_hi, a_lo, ctx->qkv, 3 * d, info, 0, pdl, s, trace_slot(ctx, *kernels)));
            Q(launch_gemm_ws(&t[0], &ag->a_hi, &ag->a_pair, ctx->qkv, info, 3 * d, L.b_qkv, n, d, 3 * d, lo, lgrid, sms, ctx->d_status, pdl, s, trace_slot(ctx, *kernels), nullptr, nullptr, 0, 4, gr));
            if (staged) Q(launch_kv_stage(ctx->qkv, info, l * layer_elems, n, c.n_head, cap, pdl, s, trace_slot(ctx, *kernels)));
            Q(launch_tree_attention_mma(ctx->qkv, info, l * layer_elems, ctx->meta, n, c.n_head, cap, ctx->o_hi, o_lo, pdl, s, trace_slot(ctx, *kernels), ctx->attn_lo != 0, nullptr, 0, attn_warps, attn_splits));
            Q(launch_gemm_ws(&t[1], &ag->o_hi, &ag->o_pair, ctx->x, info, d, L.b_o, n, d, d, lo, lgrid, sms, ctx->d_status, pdl, s, trace_slot(ctx, *kernels), nullptr, nullptr, 0, 4, gr));
            Q(launch_ln_prep(ctx->x, L.ln2_g, L.ln2_b, n, d, c.ln_eps, ctx->a_hi, a_lo, ctx->h, F, info, 0, pdl, s, trace_slot(ctx, *kernels)));
            Q(launch_gemm_ws(&t[2], &af->a_hi, &af->a_pair, ctx->h, info, F, L.b_fc, n, d, F, lo, lgrid, sms, ctx->d_status, pdl, s, trace_slot(ctx, *kernels), nullptr, nullptr, 0, 4, gr_fc));
            if (fuse_gelu) {
                Q(launch_gemm_ws(&t[3], &ag->h_src, nullptr, ctx->x, info, d, L.b_proj, n, F, d, lo, lgrid, sms, ctx->d_status, pdl, s, trace_slot(ctx, *kernels), nullptr, nullptr, 0, 4, gr, 1));
            } else {
                Q(launch_gelu_prep(ctx->h, n, F, ctx->h_hi, h_lo, pdl, s, trace_slot(ctx, *kernels)));
                Q(launch_gemm_ws(&t[3], &ag->h_hi, &ag->h_pair, ctx->x, info, d, L.b_proj, n, F, d, lo, lgrid, sms, ctx->d_status, pdl, s, trace_slot(ctx, *kernels), nullptr, nullptr, 0, 4, gr));
            }
        }
        Q(launch_ln_prep(ctx->x, ctx->lnf_g, ctx->lnf_b, n, d, c.ln_eps, ctx->a_hi, a_lo, nullptr, 0, info, 0, pdl, s, trace_slot(ctx, *kernels)));
        Q(launch_gemm_ws(&ctx->map_wte, &am->a_hi, &am->a_pair, nullptr, info, c.vocab, nullptr, n, d, c.vocab, lo, hgrid, sms, ctx->d_status, pdl, s, trace_slot(ctx, *kernels), head));
        ctx->trace_count = ctx->trace_kernels ? 8 * *kernels : 0;
    } else {
        for (int l = 0; l < c.n_layer; ++l) {
            const LayerWeights &L = ctx->layers[l];
            Q(launch_layernorm(ctx->x, L.ln1_g, L.ln1_b, n, d, c.ln_eps, ctx->a, s));
            Q(launch_gemm_simple(ctx->a, L.w_qkv, c.dtype, L.b_qkv, n, d, 3 * d, EPI_STORE, ctx->qkv, s));
            Q(launch_tree_attention(ctx->qkv, info, l * layer_elems, c.dtype, ctx->meta, n, max_keys, c.n_head, cap, ctx->o, nullptr, nullptr, false, s));
            Q(launch_gemm_simple(ctx->o, L.w_o, c.dtype, L.b_o, n, d, d, EPI_RESIDUAL, ctx->x, s));
            Q(launch_layernorm(ctx->x, L.ln2_g, L.ln2_b, n, d, c.ln_eps, ctx->a, s));
            Q(launch_gemm_simple(ctx->a, L.w_fc, c.dtype, L.b_fc, n, d, F, EPI_GELU, ctx->h, s));
            Q(launch_gemm_simple(ctx->h, L.w_proj, c.dtype, L.b_proj, n, F, d, EPI_RESIDUAL, ctx->x, s));
        }
        Q(launch_layernorm(ctx->x, ctx->lnf_g, ctx->lnf_b, n, d, c.ln_eps, ctx->a, s));
        Q(launch_gemm_simple(ctx->a, ctx->wte, c.dtype, nullptr, n, d, c.vocab, EPI_STORE, step.logits, s));
    }
#undef Q
    return cudaSuccess;
}

// Capture the forward for tree size n into an executable graph and remember its first node.
int capture_forward(ssd_ctx *ctx, int n, int cap, const NodeList &tk, const NodeList &pr, const StepInfo &step, int attn_splits) {
    ssd_ctx::ForwardGraph &fg = ctx->graphs[n][attn_splits >> 1];
    cudaGraph_t graph = nullptr;
    int kernels = 0;
    CU(cudaStreamBeginCapture(ctx->capture_stream, cudaStreamCaptureModeThreadLocal));
    cudaError_t e = enqueue_forward(ctx, n, cap, tk, pr, step, ctx->capture_stream, &kernels, attn_splits);
    cudaError_t e2 = cudaStreamEndCapture(ctx->capture_stream, &graph);
    if (e != cudaSuccess || e2 != cudaSuccess) {
        if (graph) cudaGraphDestroy(graph);
        return fail_cuda(ctx, e != cudaSuccess ? e : e2);
    }
    size_t count = 0;
    e = cudaGraphGetNodes(graph, nullptr, &count);
    std::vector<cudaGraphNode_t> nodes(count);
    if (e == cudaSuccess) e = cudaGraphGetNodes(graph, nodes.data(), &count);
    cudaGraphNode_t prep = nullptr;
    for (size_t i = 0; i < count && e == cudaSuccess && !prep; ++i) {
        cudaGraphNodeType ty;
        if (cudaGraphNodeGetType(nodes[i], &ty) != cudaSuccess || ty != cudaGraphNodeTypeKernel) continue;
        cudaKernelNodeParams kp;
        if (cudaGraphKernelNodeGetParams(nodes[i], &kp) == cudaSuccess && kp.func == tree_prep_kernel_address()) prep = nodes[i];
    }
    cudaGraphExec_t exec = nullptr;
    if (e == cudaSuccess && !prep) e = cudaErrorUnknown;
    if (e == cudaSuccess) e = cudaGraphInstantiate(&exec, graph, 0);
    if (e != cudaSuccess) { cudaGraphDestroy(graph); return fail_cuda(ctx, e); }
    fg.graph = graph; // kept alive: prep_node is a handle into it
    fg.exec = exec;
    fg.prep_node = prep;
    fg.kernels = kernels;
    return SSD_OK;
}
// Per-row fp64 scratch of the sampling rule and of the proposal laws, [rows, vocab], with the support lists of the top-k
// cut behind it; grown on first use and when a larger tree arrives (a failed allocation only means that the acceptance
// walk computes the visited rows itself).
int ensure_law_rows(ssd_ctx *ctx, int n) {
    if (ctx->acc.rows_cap >= n) return SSD_OK;
    CU(cudaStreamSynchronize(ctx->stream));
    if (ctx->acc.rows) { cudaFree(ctx->acc.rows); ctx->acc.rows = nullptr; ctx->acc.rows_cap = 0; ctx->acc.sup_idx = ctx->acc.sup_cnt = nullptr; }
    if (ctx->acc.rows_alt) { cudaFree(ctx->acc.rows_alt); ctx->acc.rows_alt = nullptr; }
    const int rows = (n + 31) & ~31;
    const size_t law_bytes = (size_t)rows * ctx->cfg.vocab * sizeof(double), idx_bytes = (size_t)rows * SSD_ACC_SUPPORT * sizeof(int32_t);
    void *q = nullptr;
    if (cudaMalloc(&q, law_bytes + idx_bytes + (size_t)rows * sizeof(int32_t) + (size_t)rows * 8 * sizeof(double) + 8) == cudaSuccess) {
        ctx->acc.rows = (double *)q; ctx->acc.rows_cap = rows;
        ctx->acc.row_total = (double *)(((uintptr_t)q + law_bytes + idx_bytes + (size_t)rows * sizeof(int32_t) + 7) & ~(uintptr_t)7);
        ctx->acc.sup_idx = (int32_t *)((char *)q + law_bytes);
        ctx->acc.sup_cnt = (int32_t *)((char *)q + law_bytes + idx_bytes);
        void *alt = nullptr; // (optional: without it a refusal takes two passes)
        if (cudaMalloc(&alt, law_bytes) == cudaSuccess) ctx->acc.rows_alt = (double *)alt;
        else (void)cudaGetLastError();
    } else {
        (void)cudaGetLastError();
    }
    return SSD_OK;
}
} // namespace

extern "C" {

const char *ssd_strerror(int status) {
    switch (status) {
    case SSD_OK: return "ok";
    case SSD_ERR_BAD_ARG: return "bad argument";
    case SSD_ERR_NOT_LOADED: return "weights not loaded";
    case SSD_ERR_INVALID_TREE: return "invalid tree";
    case SSD_ERR_CTX_OVERFLOW: return "context overflow";
    case SSD_ERR_BAD_PATH: return "path is not a root-to-node path of the last verified tree";
    case SSD_ERR_CUDA: return "CUDA error";
    case SSD_ERR_TIMEOUT: return "device-side wait timed out";
    case SSD_ERR_NOMEM: return "out of memory";
    case SSD_ERR_UNSUPPORTED: return "unsupported shape";
    default: return "unknown status";
    }
}

int ssd_create(const ssd_config *cfg, int device, void *cuda_stream, ssd_ctx **out) {
    if (out) *out = nullptr;
    if (!cfg || !out) return SSD_ERR_BAD_ARG;
    if (cfg->n_layer < 1 || cfg->d_model < 1 || cfg->n_head < 1 || cfg->d_ff < 1 || cfg->vocab < 1 || cfg->n_ctx < 2 ||
        cfg->max_nodes < 1 || !(cfg->ln_eps > 0.f) || (cfg->dtype != SSD_DTYPE_F32 && cfg->dtype != SSD_DTYPE_BF16 && cfg->dtype != SSD_DTYPE_BF16_W8))
        return SSD_ERR_BAD_ARG;
    if (cfg->d_head != 64 || cfg->n_head * cfg->d_head != cfg->d_model || cfg->d_model % 64 || cfg->d_ff % 64 ||
        cfg->max_nodes > SSD_MAX_NODES || cfg->d_model > 8192)
        return SSD_ERR_UNSUPPORTED;
    // (the fp32 model's attention keeps one score per key and warp in shared memory)
    if (cfg->dtype == SSD_DTYPE_F32 && tree_attention_smem(cfg->n_ctx + cfg->max_nodes) > 48 * 1024) return SSD_ERR_UNSUPPORTED;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return SSD_ERR_CUDA;
    ssd_ctx *ctx = new (std::nothrow) ssd_ctx();
    if (!ctx) return SSD_ERR_NOMEM;
    ctx->cfg = *cfg;
    // 8-bit weights change how the matrices are stored and streamed, nothing else: the cache, the activations and every
    // other kernel are those of the bf16 model
    ctx->w8 = cfg->dtype == SSD_DTYPE_BF16_W8;
    if (ctx->w8) ctx->cfg.dtype = SSD_DTYPE_BF16;
    ctx->wte8 = nullptr; ctx->wte_scale = nullptr;
    ctx->w8_planes = 4;
    ctx->attn_splits = 0;
    ctx->node_groups = 1;
    ctx->fused_gelu = 0;
    ctx->attn_staged_warps = 0;
    ctx->stage_kv_from = 128; // (measured at the GPT-2-large shape: 2 % faster at 128 nodes, 14 % at 256, slower below)
    ctx->device = device;
    ctx->stream = (cudaStream_t)cuda_stream;
    ctx->loaded = false;
    ctx->last_cuda = 0;
    ctx->last_cuda_line = 0;
    ctx->launches = 0;
    ctx->elt = cfg->dtype == SSD_DTYPE_F32 ? 4 : 2;
    cfg = &ctx->cfg; // (dtype normalised)
    ctx->h_result = nullptr;
    ctx->h_propose = nullptr;
    ctx->d_sparse_idx = nullptr; ctx->d_sparse_val = nullptr; ctx->d_sparse_rows = nullptr;
    ctx->sparse_entries_cap = ctx->sparse_rows_cap = 0;
    DeviceGuard g(device);
    int rc = g.ok ? SSD_OK : SSD_ERR_CUDA;
    const size_t n = cfg->max_nodes, d = cfg->d_model;
    auto A = [&](auto **p, size_t cnt) { if (rc == SSD_OK) rc = dev_alloc(ctx, p, cnt); };
    A(&ctx->meta.tokens, n); A(&ctx->meta.parent, n); A(&ctx->meta.depth, n); A(&ctx->meta.pos, n);
    A(&ctx->meta.anc, n * SSD_ANC_WORDS); A(&ctx->meta.child_off, n + 1); A(&ctx->meta.child, n);
    A(&ctx->x, n * d); A(&ctx->a, n * d); A(&ctx->qkv, n * 3 * d); A(&ctx->o, n * d); A(&ctx->h, n * (size_t)cfg->d_ff);
    ctx->acc.arg_parts = 4;
    ctx->acc.dev_status = nullptr;
    ctx->acc.head_parts = 0;
    ctx->acc.sp_idx = nullptr; ctx->acc.sp_val = nullptr; ctx->acc.sp_entries = 0;
    ctx->head_val = nullptr; ctx->head_arg = ctx->head_bad = nullptr; ctx->head_tiles = 0; ctx->use_head_stats = 0;
    ctx->head_logits = nullptr; ctx->head_n = 0;
    A(&ctx->acc.r, (size_t)cfg->vocab); A(&ctx->acc.row_val, 4 * n); A(&ctx->acc.row_arg, 4 * n); A(&ctx->acc.row_bad, 4 * n); A(&ctx->acc.result, n + 4);
    A(&ctx->d_status, 1);
    A(&ctx->d_info, 1);
    memset(ctx->graphs, 0, sizeof(ctx->graphs));
    ctx->capture_stream = nullptr;
    ctx->use_graph = 1;
    ctx->use_cluster = 0;
    ctx->attn_lo = 0;
    ctx->cl_max = 8;
    for (int &v : ctx->cl_size) v = 0;
    ctx->d_stats1 = ctx->d_stats2 = nullptr;
    ctx->d_trace = nullptr;
    ctx->sm_count = 148;
    ctx->tensor_path = cfg->dtype == SSD_DTYPE_BF16;
    ctx->use_lo = 1;
    ctx->pdl = 1;
    ctx->gemm_grid = 0;
    ctx->trace_kernels = 0;
    ctx->trace_count = 0;
    ctx->head_grid = 0;
    ctx->a_hi = ctx->a_lo = ctx->o_hi = ctx->o_lo = ctx->h_hi = ctx->h_lo = nullptr;
    if (ctx->tensor_path) {
        const size_t rows = n <= 32 ? 32 : ((n + 15) & ~size_t(15)); // operand planes hold whole 16-row boxes, at least two
        // (a buffer's lo plane follows its hi plane, so that one 3-D copy fetches both)
        A(&ctx->a_hi, 2 * rows * d); A(&ctx->o_hi, 2 * rows * d); A(&ctx->h_hi, 2 * rows * (size_t)cfg->d_ff);
        if (rc == SSD_OK) { ctx->a_lo = ctx->a_hi + rows * d; ctx->o_lo = ctx->o_hi + rows * d; ctx->h_lo = ctx->h_hi + rows * (size_t)cfg->d_ff; }
        ctx->a8 = ctx->o8 = ctx->h8 = nullptr;
        if (ctx->w8) { A(&ctx->a8, 4 * rows * d); A(&ctx->o8, 4 * rows * d); A(&ctx->h8, 4 * rows * (size_t)cfg->d_ff); }
        ctx->head_tiles = (cfg->vocab + 127) / 128;
        A(&ctx->head_val, n * (size_t)ctx->head_tiles); A(&ctx->head_arg, n * (size_t)ctx->head_tiles); A(&ctx->head_bad, n * (size_t)ctx->head_tiles);
        if (rc == SSD_OK) {
            cudaError_t e = cudaSuccess;
            __nv_bfloat16 *planes[6] = {ctx->a_hi, ctx->a_lo, ctx->o_hi, ctx->o_lo, ctx->h_hi, ctx->h_lo};
            for (int q = 0; q < 6 && e == cudaSuccess; ++q)
                e = cudaMemsetAsync(planes[q], 0, rows * (q < 4 ? d : (size_t)cfg->d_ff) * sizeof(__nv_bfloat16), ctx->stream);
            uint8_t *planes8[3] = {ctx->a8, ctx->o8, ctx->h8}; // (rows past the tree are read by the projections' boxes: zero codes)
            for (int q = 0; q < 3 && e == cudaSuccess && ctx->w8; ++q)
                e = cudaMemsetAsync(planes8[q], 0, 4 * rows * (q < 2 ? d : (size_t)cfg->d_ff), ctx->stream);
            int dev_sms = 0;
            if (e == cudaSuccess) e = cudaDeviceGetAttribute(&dev_sms, cudaDevAttrMultiProcessorCount, device);
            if (e == cudaSuccess) e = gemm_ws_prepare();
            if (e == cudaSuccess) e = tree_attention_mma_prepare();
            if (e == cudaSuccess) e = prep_kernels_prepare();
            if (e == cudaSuccess) e = gemm_cl_prepare();
            if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->capture_stream, cudaStreamNonBlocking);
            if (e != cudaSuccess) rc = fail_cuda(ctx, e);
            if (dev_sms > 0) ctx->sm_count = dev_sms;
        }
        if (rc == SSD_OK) {
            int m = SSD_OK;
            ctx->plane_rows = rows;
            for (auto &am : ctx->act_maps) am.built = false;
            if (!act_maps_for(ctx, 1)) m = SSD_ERR_CUDA; // (also checks that the driver entry point exists)
            rc = m;
        }
    }
    if (rc == SSD_OK) {
        cudaError_t e = cudaMallocHost((void **)&ctx->h_result, sizeof(int32_t) * (n + 4));
        if (e == cudaSuccess) e = cudaMallocHost((void **)&ctx->h_propose, sizeof(int32_t) * SSD_MAX_NODES * 9);
        if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_status, 0, sizeof(int32_t), ctx->stream);
        if (e != cudaSuccess) rc = fail_cuda(ctx, e);
    }
    if (rc != SSD_OK) { ssd_destroy(ctx); return rc; }
    *out = ctx;
    return SSD_OK;
}

void ssd_destroy(ssd_ctx *ctx) {
    if (!ctx) return;
    DeviceGuard g(ctx->device);
    cudaStreamSynchronize(ctx->stream);
    for (auto &row : ctx->graphs)
        for (auto &g : row)
            if (g.exec) { cudaGraphExecDestroy(g.exec); cudaGraphDestroy(g.graph); }
    if (ctx->capture_stream) cudaStreamDestroy(ctx->capture_stream);
    for (void *p : ctx->owned) cudaFree(p);
    if (ctx->acc.rows) cudaFree(ctx->acc.rows);
    if (ctx->acc.rows_alt) cudaFree(ctx->acc.rows_alt);
    if (ctx->h_result) cudaFreeHost(ctx->h_result);
    if (ctx->h_propose) cudaFreeHost(ctx->h_propose);
    cudaFree(ctx->d_sparse_idx); cudaFree(ctx->d_sparse_val); cudaFree(ctx->d_sparse_rows);
    delete ctx;
}

int ssd_load_weights(ssd_ctx *ctx, const ssd_weights *w) {
    if (!ctx || !w) return SSD_ERR_BAD_ARG;
    if (ctx->loaded) return SSD_ERR_BAD_ARG; // one model per context
    const ssd_config &c = ctx->cfg;
    const void *const *tables[] = {w->ln1_g, w->ln1_b, w->w_qkv, w->b_qkv, w->w_o, w->b_o, w->ln2_g, w->ln2_b, w->w_fc, w->b_fc, w->w_proj, w->b_proj};
    for (auto t : tables) {
        if (!t) return SSD_ERR_BAD_ARG;
        for (int l = 0; l < c.n_layer; ++l)
            if (!t[l]) return SSD_ERR_BAD_ARG;
    }
    if (!w->wte || !w->wpe || !w->lnf_g || !w->lnf_b) return SSD_ERR_BAD_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return SSD_ERR_CUDA;
    const size_t d = c.d_model, F = c.d_ff;
    std::vector<float> tmp;
    int rc;
#define UP_M(src, cnt, dst) if ((rc = upload_matrix(ctx, src, cnt, (void **)(dst))) != SSD_OK) return rc
#define UP_V(src, cnt, dst) if ((rc = upload_vector_f32(ctx, src, cnt, dst, tmp)) != SSD_OK) return rc
    UP_M(w->wte, (size_t)c.vocab * d, &ctx->wte);
    UP_M(w->wpe, (size_t)c.n_ctx * d, &ctx->wpe);
    UP_V(w->lnf_g, d, (const float **)&ctx->lnf_g);
    UP_V(w->lnf_b, d, (const float **)&ctx->lnf_b);
    ctx->layers.assign(c.n_layer, LayerWeights());
    for (int l = 0; l < c.n_layer; ++l) {
        LayerWeights &L = ctx->layers[l];
        UP_V(w->ln1_g[l], d, &L.ln1_g); UP_V(w->ln1_b[l], d, &L.ln1_b);
        UP_M(w->w_qkv[l], 3 * d * d, &L.w_qkv); UP_V(w->b_qkv[l], 3 * d, &L.b_qkv);
        UP_M(w->w_o[l], d * d, &L.w_o); UP_V(w->b_o[l], d, &L.b_o);
        UP_V(w->ln2_g[l], d, &L.ln2_g); UP_V(w->ln2_b[l], d, &L.ln2_b);
        UP_M(w->w_fc[l], F * d, &L.w_fc); UP_V(w->b_fc[l], F, &L.b_fc);
        UP_M(w->w_proj[l], d * F, &L.w_proj); UP_V(w->b_proj[l], d, &L.b_proj);
    }
#undef UP_M
#undef UP_V
    if (ctx->w8) {
        // Quantise on the device: codes and scales in new buffers; a layer's bf16 matrices are released once quantised
        // (the embedding table stays: the look-up reads it).
        int rc3;
        auto quantise = [&](const void *src, size_t rows, size_t cols, const void **codes_out, const float **scales_out) -> int {
            uint8_t *q = nullptr;
            float *sc = nullptr;
            int r = dev_alloc(ctx, &q, rows * cols);
            if (r == SSD_OK) r = dev_alloc(ctx, &sc, rows);
            if (r != SSD_OK) return r;
            CU(launch_quantise_rows_e4m3(src, rows, cols, q, sc, ctx->stream));
            *codes_out = q; *scales_out = sc;
            return SSD_OK;
        };
        auto release = [&](const void *p) {
            for (size_t i = ctx->owned.size(); i-- > 0;)
                if (ctx->owned[i] == p) { ctx->owned.erase(ctx->owned.begin() + (long)i); break; }
            cudaFree(const_cast<void *>(p));
        };
        const void *q8 = nullptr;
        const float *s8 = nullptr;
        if ((rc3 = quantise(ctx->wte, c.vocab, d, &q8, &s8)) != SSD_OK) return rc3;
        ctx->wte8 = (uint8_t *)q8; ctx->wte_scale = (float *)s8;
        for (int l = 0; l < c.n_layer; ++l) {
            LayerWeights &L = ctx->layers[l];
            const void *bf[4] = {L.w_qkv, L.w_o, L.w_fc, L.w_proj};
            if ((rc3 = quantise(bf[0], 3 * d, d, &L.w_qkv, &L.s_qkv)) != SSD_OK || (rc3 = quantise(bf[1], d, d, &L.w_o, &L.s_o)) != SSD_OK ||
                (rc3 = quantise(bf[2], F, d, &L.w_fc, &L.s_fc)) != SSD_OK || (rc3 = quantise(bf[3], d, F, &L.w_proj, &L.s_proj)) != SSD_OK)
                return rc3;
            CU(cudaStreamSynchronize(ctx->stream));
            for (const void *p : bf) release(p);
        }
    }
    if (ctx->tensor_path) {
        ctx->map_layers.assign((size_t)4 * c.n_layer, TensorMap());
        auto make_map = ctx->w8 ? make_tensor_map_u8 : make_tensor_map_bf16;
        int m = make_map(&ctx->map_wte, ctx->w8 ? (const void *)ctx->wte8 : ctx->wte, c.vocab, d, 128);
        for (int l = 0; l < c.n_layer && m == SSD_OK; ++l) {
            const LayerWeights &L = ctx->layers[l];
            TensorMap *t = &ctx->map_layers[(size_t)4 * l];
            m = make_map(&t[0], L.w_qkv, 3 * d, d, 128);
            if (m == SSD_OK) m = make_map(&t[1], L.w_o, d, d, 128);
            if (m == SSD_OK) m = make_map(&t[2], L.w_fc, F, d, 128);
            if (m == SSD_OK) m = make_map(&t[3], L.w_proj, d, F, 128);
        }
        if (m != SSD_OK) return m;
        // LayerNorm-fold vectors of the cluster-reduced path, its statistics buffers, the timeline buffer
        int rc2;
        ctx->folds.assign(c.n_layer, ssd_ctx::LayerFold());
        for (int l = 0; l < c.n_layer && !ctx->w8; ++l) { // (the cluster-reduced path does not take 8-bit weights)
            const LayerWeights &L = ctx->layers[l];
            ssd_ctx::LayerFold &f = ctx->folds[l];
            if ((rc2 = dev_alloc(ctx, &f.c1_qkv, 3 * d)) != SSD_OK || (rc2 = dev_alloc(ctx, &f.c2_qkv, 3 * d)) != SSD_OK ||
                (rc2 = dev_alloc(ctx, &f.c1_fc, F)) != SSD_OK || (rc2 = dev_alloc(ctx, &f.c2_fc, F)) != SSD_OK)
                return rc2;
            CU(launch_ln_fold(L.w_qkv, L.ln1_g, L.ln1_b, L.b_qkv, (int)(3 * d), (int)d, f.c1_qkv, f.c2_qkv, ctx->stream));
            CU(launch_ln_fold(L.w_fc, L.ln2_g, L.ln2_b, L.b_fc, (int)F, (int)d, f.c1_fc, f.c2_fc, ctx->stream));
        }
        const size_t stats_parts_max = (d + 127) / 128 > 16 ? (d + 127) / 128 : 16; // output tiles (cluster path) / CTAs per tile (self-staged path)
        const size_t stats_floats = stats_parts_max * SSD_MAX_NODES * 2;
        if ((rc2 = dev_alloc(ctx, &ctx->d_stats1, stats_floats)) != SSD_OK || (rc2 = dev_alloc(ctx, &ctx->d_stats2, stats_floats)) != SSD_OK) return rc2;
        if ((rc2 = dev_alloc(ctx, &ctx->d_trace, (size_t)SSD_TRACE_SLOTS)) != SSD_OK) return rc2;
        CU(cudaMemsetAsync(ctx->d_trace, 0, sizeof(unsigned long long) * SSD_TRACE_SLOTS, ctx->stream));
    }
    CU(cudaStreamSynchronize(ctx->stream));
    ctx->loaded = true;
    return SSD_OK;
}

int ssd_w8_read(ssd_ctx *ctx, int32_t which, int32_t layer, uint8_t *codes_out, float *scales_out) {
    if (!ctx || !codes_out || !scales_out || !ctx->w8 || which < 0 || which > 4) return SSD_ERR_BAD_ARG;
    if (!ctx->loaded) return SSD_ERR_NOT_LOADED;
    if (which < 4 && (layer < 0 || layer >= ctx->cfg.n_layer)) return SSD_ERR_BAD_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return SSD_ERR_CUDA;
    const size_t d = ctx->cfg.d_model, F = ctx->cfg.d_ff;
    const void *codes = ctx->wte8;
    const float *scales = ctx->wte_scale;
    size_t rows = ctx->cfg.vocab, cols = d;
    if (which < 4) {
        const LayerWeights &L = ctx->layers[layer];
        const void *cw[4] = {L.w_qkv, L.w_o, L.w_fc, L.w_proj};
        const float *sw[4] = {L.s_qkv, L.s_o, L.s_fc, L.s_proj};
        const size_t rw[4] = {3 * d, d, F, d}, kw[4] = {d, d, d, F};
        codes = cw[which]; scales = sw[which]; rows = rw[which]; cols = kw[which];
    }
    CU(cudaMemcpyAsync(codes_out, codes, rows * cols, cudaMemcpyDeviceToHost, ctx->stream));
    CU(cudaMemcpyAsync(scales_out, scales, rows * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream));
    CU(cudaStreamSynchronize(ctx->stream));
    return SSD_OK;
}

int ssd_kv_create(ssd_ctx *ctx, ssd_kv **out) {
    if (out) *out = nullptr;
    if (!ctx || !out) return SSD_ERR_BAD_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return SSD_ERR_CUDA;
    ssd_kv *kv = new (std::nothrow) ssd_kv();
    if (!kv) return SSD_ERR_NOMEM;
    kv->ctx = ctx;
    kv->cap = (ctx->cfg.n_ctx + ctx->cfg.max_nodes + 15) & ~15; // whole 16-key blocks
    kv->len = 0;
    kv->last_n = 0;
    kv->k = kv->v = nullptr;
    const size_t bytes = (size_t)ctx->cfg.n_layer * ctx->cfg.d_model * kv->cap * ctx->elt;
    cudaError_t e = cudaMalloc(&kv->k, bytes);
    if (e == cudaSuccess) e = cudaMalloc(&kv->v, bytes);
    if (e == cudaSuccess) e = cudaMemsetAsync(kv->k, 0, bytes, ctx->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(kv->v, 0, bytes, ctx->stream);
    if (e != cudaSuccess) {
        cudaFree(kv->k); cudaFree(kv->v);
        delete kv;
        return fail_cuda(ctx, e);
    }
    *out = kv;
    return SSD_OK;
}

void ssd_kv_destroy(ssd_kv *kv) {
    if (!kv) return;
    DeviceGuard g(kv->ctx->device);
    cudaStreamSynchronize(kv->ctx->stream);
    cudaFree(kv->k);
    cudaFree(kv->v);
    delete kv;
}

int ssd_kv_reset(ssd_kv *kv) {
    if (!kv) return SSD_ERR_BAD_ARG;
    kv->len = 0;
    kv->last_n = 0;
    return SSD_OK;
}
int ssd_kv_len(const ssd_kv *kv, int32_t *len) {
    if (!kv || !len) return SSD_ERR_BAD_ARG;
    *len = kv->len;
    return SSD_OK;
}
int ssd_kv_rollback(ssd_kv *kv, int32_t len) {
    if (!kv || len < 0 || len > kv->len) return SSD_ERR_BAD_ARG;
    kv->len = len;
    kv->last_n = 0;
    return SSD_OK;
}

int ssd_verify_tree(ssd_ctx *ctx, const int32_t *tokens, const int32_t *parent_idx, int32_t n_nodes, ssd_kv *kv, float *logits_out) {
    if (!ctx || !tokens || !parent_idx || !kv || !logits_out || kv->ctx != ctx) return SSD_ERR_BAD_ARG;
    if (!ctx->loaded) return SSD_ERR_NOT_LOADED;
    const ssd_config &c = ctx->cfg;
    int32_t depth[SSD_MAX_NODES];
    int max_depth = 0;
    int rc = check_tree(c, tokens, parent_idx, n_nodes, depth, &max_depth);
    if (rc != SSD_OK) return rc;
    if (kv->len + max_depth >= c.n_ctx) return SSD_ERR_CTX_OVERFLOW;
    DeviceGuard g(ctx->device);
    if (!g.ok) return SSD_ERR_CUDA;

    NodeList tk, pr;
    memcpy(tk.v, tokens, sizeof(int32_t) * n_nodes);
    memcpy(pr.v, parent_idx, sizeof(int32_t) * n_nodes);
    StepInfo step;
    step.n = n_nodes; step.kv_len = kv->len; step.kbase = kv->k; step.vbase = kv->v; step.logits = logits_out;
    int kernels = 0;
    const int splits = ctx->tensor_path ? attn_splits_for(ctx, kv->len, n_nodes) : 1;
    if (ctx->tensor_path && ctx->use_graph) {
        ssd_ctx::ForwardGraph &fg = ctx->graphs[n_nodes][splits >> 1];
        if (!fg.exec) {
            rc = capture_forward(ctx, n_nodes, kv->cap, tk, pr, step, splits);
            if (rc != SSD_OK) return rc;
        }
        // patch the tree, prefix length and addresses into the first node, then replay
        TreeMeta meta = ctx->meta;
        StepInfo *info_out = ctx->d_info;
        void *args[5] = {&tk, &pr, &step, &meta, &info_out};
        cudaKernelNodeParams kp = {};
        kp.func = const_cast<void *>(tree_prep_kernel_address());
        kp.gridDim = dim3(1); kp.blockDim = dim3(SSD_MAX_NODES); kp.sharedMemBytes = 0; kp.kernelParams = args; kp.extra = nullptr;
        CU(cudaGraphExecKernelNodeSetParams(fg.exec, fg.prep_node, &kp));
        CU(cudaGraphLaunch(fg.exec, ctx->stream));
        kernels = fg.kernels;
    } else {
        CU(enqueue_forward(ctx, n_nodes, kv->cap, tk, pr, step, ctx->stream, &kernels, splits));
    }
    ctx->launches += kernels;
    ctx->head_logits = (ctx->tensor_path && ctx->use_head_stats) ? logits_out : nullptr;
    ctx->head_n = n_nodes;
    kv->last_n = n_nodes;
    memcpy(kv->last_parent, parent_idx, sizeof(int32_t) * n_nodes);
    return SSD_OK;
}

namespace {
// ssd_accept_tree, with the proposal rows dense (draft_probs) or as device lists (sp_idx / sp_val, [n][sp_entries]).
int accept_impl(ssd_ctx *ctx, const float *logits, const float *draft_probs, const int32_t *sp_idx, const float *sp_val, int sp_entries,
                const int32_t *tokens, const int32_t *parent_idx, int32_t n_nodes, const ssd_sampling *sampling, ssd_rng *rng_state,
                int32_t *path_out, int32_t *n_path_out, int32_t *next_token_out) {
    if (!ctx || !logits || !tokens || !parent_idx || !sampling || !rng_state || !path_out || !n_path_out || !next_token_out)
        return SSD_ERR_BAD_ARG;
    if (sampling->mode != SSD_GREEDY && sampling->mode != SSD_SAMPLING) return SSD_ERR_BAD_ARG;
    if (sampling->mode == SSD_SAMPLING && ((!draft_probs && !sp_idx) || !(sampling->temperature > 0.f) || sampling->top_k < 0)) return SSD_ERR_BAD_ARG;
    const ssd_config &c = ctx->cfg;
    int32_t depth[SSD_MAX_NODES];
    int max_depth = 0;
    int rc = check_tree(c, tokens, parent_idx, n_nodes, depth, &max_depth);
    if (rc != SSD_OK) return rc;
    DeviceGuard g(ctx->device);
    if (!g.ok) return SSD_ERR_CUDA;
    const int n = n_nodes;
    NodeList tk, pr;
    memcpy(tk.v, tokens, sizeof(int32_t) * n);
    memcpy(pr.v, parent_idx, sizeof(int32_t) * n);
    if (sampling->mode == SSD_SAMPLING && n > 1) {
        rc = ensure_law_rows(ctx, n);
        if (rc != SSD_OK) return rc;
    }
    int launched = 0;
    AcceptScratch sc = ctx->acc;
    sc.sp_idx = sp_idx; sc.sp_val = sp_val; sc.sp_entries = sp_entries;
    sc.result = ctx->h_result; // the walk writes its few words straight into the pinned host buffer: no copy to enqueue and wait for
    sc.dev_status = ctx->d_status;
    // greedy on the very logits the last forward of this context wrote: the LM head's per-tile row statistics stand in for them
    if (sampling->mode == SSD_GREEDY && ctx->head_logits && ctx->head_logits == logits && ctx->head_n == n) {
        sc.head_parts = ctx->head_tiles; sc.head_val = ctx->head_val; sc.head_arg = ctx->head_arg; sc.head_bad = ctx->head_bad;
    }
    ctx->h_result[0] = 0;
    CU(launch_accept(logits, draft_probs, tk, pr, n, c.vocab, sampling->mode, sampling->temperature, sampling->top_k, rng_state->seed,
                     rng_state->step, sc, ctx->stream, &launched));
    ctx->launches += launched;
    CU(cudaStreamSynchronize(ctx->stream));
    rng_state->step += 1;
    const int np = ctx->h_result[0];
    if (np < 1 || np > n) return SSD_ERR_CUDA; // cannot happen with a healthy device
    *n_path_out = np;
    *next_token_out = ctx->h_result[1];
    memcpy(path_out, ctx->h_result + 4, sizeof(int32_t) * np);
    // A bounded wait of one of the forward's kernels expired (the word stays set, and later forwards are no-ops, until
    // ssd_reset_device_status): the logits this walk read are not to be trusted.
    if (ctx->h_result[3] != 0) return SSD_ERR_TIMEOUT;
    return ctx->h_result[2];
}
} // namespace

int ssd_accept_tree(ssd_ctx *ctx, const float *logits, const float *draft_probs, const int32_t *tokens, const int32_t *parent_idx,
                    int32_t n_nodes, const ssd_sampling *sampling, ssd_rng *rng_state, int32_t *path_out, int32_t *n_path_out,
                    int32_t *next_token_out) {
    return accept_impl(ctx, logits, draft_probs, nullptr, nullptr, 0, tokens, parent_idx, n_nodes, sampling, rng_state, path_out, n_path_out, next_token_out);
}

int ssd_accept_tree_sparse(ssd_ctx *ctx, const float *logits, const int32_t *row_idx, const float *row_val, int32_t entries,
                           const int32_t *tokens, const int32_t *parent_idx, int32_t n_nodes, const ssd_sampling *sampling, ssd_rng *rng_state,
                           int32_t *path_out, int32_t *n_path_out, int32_t *next_token_out) {
    if (!ctx || !row_idx || !row_val || entries < 1 || entries > SSD_ACC_SUPPORT || n_nodes < 1 || n_nodes > SSD_MAX_NODES) return SSD_ERR_BAD_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return SSD_ERR_CUDA;
    if (!sampling) return SSD_ERR_BAD_ARG;
    const size_t need_e = (size_t)n_nodes * entries, need_r = (size_t)n_nodes * ctx->cfg.vocab;
    if (ctx->sparse_entries_cap < need_e) {
        CU(cudaStreamSynchronize(ctx->stream));
        cudaFree(ctx->d_sparse_idx); cudaFree(ctx->d_sparse_val);
        ctx->d_sparse_idx = nullptr; ctx->d_sparse_val = nullptr; ctx->sparse_entries_cap = 0;
        CU(cudaMalloc((void **)&ctx->d_sparse_idx, need_e * sizeof(int32_t)));
        CU(cudaMalloc((void **)&ctx->d_sparse_val, need_e * sizeof(float)));
        ctx->sparse_entries_cap = need_e;
    }
    // (the lists are pageable host memory: the copies have read them by the time the calls return)
    CU(cudaMemcpyAsync(ctx->d_sparse_idx, row_idx, need_e * sizeof(int32_t), cudaMemcpyHostToDevice, ctx->stream));
    CU(cudaMemcpyAsync(ctx->d_sparse_val, row_val, need_e * sizeof(float), cudaMemcpyHostToDevice, ctx->stream));
    // The decision kernels read the lists directly (a refusal then costs O(entries), not two passes over the vocabulary) whenever
    // every node has a scratch row for its law - the normal case; a greedy walk reads no rows at all.
    bool lists = sampling->mode == SSD_GREEDY;
    if (sampling->mode == SSD_SAMPLING && n_nodes > 1) lists = ensure_law_rows(ctx, n_nodes) == SSD_OK && ctx->acc.rows_cap >= n_nodes;
    if (lists || n_nodes == 1)
        return accept_impl(ctx, logits, nullptr, ctx->d_sparse_idx, ctx->d_sparse_val, entries, tokens, parent_idx, n_nodes, sampling, rng_state, path_out,
                           n_path_out, next_token_out);
    // otherwise: expand to dense rows and take the one-CTA walk
    if (ctx->sparse_rows_cap < need_r) {
        CU(cudaStreamSynchronize(ctx->stream));
        cudaFree(ctx->d_sparse_rows);
        ctx->d_sparse_rows = nullptr; ctx->sparse_rows_cap = 0;
        CU(cudaMalloc((void **)&ctx->d_sparse_rows, need_r * sizeof(float)));
        ctx->sparse_rows_cap = need_r;
    }
    CU(launch_expand_sparse_rows(ctx->d_sparse_idx, ctx->d_sparse_val, n_nodes, entries, ctx->cfg.vocab, ctx->d_sparse_rows, ctx->stream));
    ctx->launches += 1;
    return ssd_accept_tree(ctx, logits, ctx->d_sparse_rows, tokens, parent_idx, n_nodes, sampling, rng_state, path_out, n_path_out, next_token_out);
}

int ssd_propose_children(ssd_ctx *ctx, const float *logits, const int32_t *nodes, int32_t m, int32_t picks, const ssd_sampling *sampling,
                         ssd_rng *rng_state, float *rows_out, int32_t *tokens_out) {
    if (!ctx || !logits || !nodes || !sampling || !rng_state || !tokens_out || m < 1 || m > SSD_MAX_NODES || picks < 0 || picks > 8) return SSD_ERR_BAD_ARG;
    if (sampling->mode != SSD_GREEDY && sampling->mode != SSD_SAMPLING) return SSD_ERR_BAD_ARG;
    if (!(sampling->temperature > 0.f) || sampling->top_k < 0) return SSD_ERR_BAD_ARG;
    for (int j = 0; j < m; ++j)
        if (nodes[j] < 0 || nodes[j] >= SSD_MAX_NODES) return SSD_ERR_BAD_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return SSD_ERR_CUDA;
    int rc = ensure_law_rows(ctx, m);
    if (rc != SSD_OK) return rc;
    if (ctx->acc.rows_cap < m) return SSD_ERR_NOMEM;
    NodeList nl;
    memcpy(nl.v, nodes, sizeof(int32_t) * m);
    int32_t *picks_host = ctx->h_propose, *bad_host = ctx->h_propose + SSD_MAX_NODES * 8; // the kernel writes into pinned host memory
    CU(launch_propose_children(logits, nl, m, ctx->cfg.vocab, sampling->mode, sampling->temperature, sampling->top_k, picks, rng_state->seed,
                               rng_state->step, ctx->acc.rows, ctx->acc.row_total, ctx->acc.row_bad, rows_out, picks_host, bad_host, ctx->stream));
    ctx->launches += 2;
    CU(cudaStreamSynchronize(ctx->stream));
    rng_state->step += 1;
    for (int j = 0; j < m; ++j)
        if (bad_host[j]) return SSD_ERR_BAD_ARG; // a listed row holds a non-finite logit
    memcpy(tokens_out, picks_host, sizeof(int32_t) * m * picks);
    return SSD_OK;
}

int ssd_kv_commit(ssd_ctx *ctx, ssd_kv *kv, const int32_t *path, int32_t n_path) {
    if (!ctx || !kv || !path || kv->ctx != ctx) return SSD_ERR_BAD_ARG;
    if (n_path < 1 || n_path > kv->last_n || path[0] != 0) return SSD_ERR_BAD_PATH;
    for (int j = 1; j < n_path; ++j)
        if (path[j] <= 0 || path[j] >= kv->last_n || kv->last_parent[path[j]] != path[j - 1]) return SSD_ERR_BAD_PATH;
    if (kv->len + n_path > ctx->cfg.n_ctx) return SSD_ERR_CTX_OVERFLOW;
    DeviceGuard g(ctx->device);
    if (!g.ok) return SSD_ERR_CUDA;
    NodeList p;
    memcpy(p.v, path, sizeof(int32_t) * n_path);
    int launched = 0;
    CU(launch_kv_commit(kv->k, kv->v, ctx->cfg.dtype, ctx->cfg.n_layer, ctx->cfg.n_head, kv->cap, kv->len, p, n_path, ctx->stream, &launched));
    ctx->launches += launched;
    kv->len += n_path;
    kv->last_n = 0;
    return SSD_OK;
}

int ssd_kv_read(ssd_ctx *ctx, const ssd_kv *kv, int32_t layer, int32_t which, int32_t slot0, int32_t rows, float *out_host) {
    if (!ctx || !kv || !out_host || kv->ctx != ctx || layer < 0 || layer >= ctx->cfg.n_layer || (which != 0 && which != 1) || slot0 < 0 ||
        rows < 1 || slot0 + rows > kv->cap)
        return SSD_ERR_BAD_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return SSD_ERR_CUDA;
    const size_t cnt = (size_t)rows * ctx->cfg.d_model;
    float *tmp = nullptr;
    CU(cudaMalloc((void **)&tmp, cnt * sizeof(float)));
    const size_t layer_elems = (size_t)ctx->cfg.n_head * kv->cap * 64;
    const void *base = (const char *)(which ? kv->v : kv->k) + (size_t)layer * layer_elems * ctx->elt;
    const int transposed = (which == 1 && ctx->tensor_path) ? 1 : 0;
    cudaError_t e = launch_kv_read(base, ctx->cfg.dtype, ctx->cfg.n_head, kv->cap, slot0, rows, transposed, tmp, ctx->stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(out_host, tmp, cnt * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
    cudaFree(tmp);
    if (e != cudaSuccess) return fail_cuda(ctx, e);
    return SSD_OK;
}

int ssd_last_device_status(ssd_ctx *ctx, int32_t *word) {
    if (!ctx || !word) return SSD_ERR_BAD_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return SSD_ERR_CUDA;
    CU(cudaMemcpyAsync(word, ctx->d_status, sizeof(int32_t), cudaMemcpyDeviceToHost, ctx->stream));
    CU(cudaStreamSynchronize(ctx->stream));
    return SSD_OK;
}
int ssd_reset_device_status(ssd_ctx *ctx) {
    if (!ctx) return SSD_ERR_BAD_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return SSD_ERR_CUDA;
    CU(cudaMemsetAsync(ctx->d_status, 0, sizeof(int32_t), ctx->stream));
    CU(cudaStreamSynchronize(ctx->stream));
    return SSD_OK;
}
int ssd_debug_expire_wait(ssd_ctx *ctx, int32_t limit_us) {
    if (!ctx || limit_us < 1 || limit_us > 1000000) return SSD_ERR_BAD_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return SSD_ERR_CUDA;
    CU(launch_expired_wait(ctx->d_status, (long long)limit_us * 2000ll, ctx->stream)); // ~2 GHz SM clock
    ctx->launches += 1;
    return SSD_OK;
}
int ssd_set_tuning(ssd_ctx *ctx, int32_t knob, int32_t value) {
    if (!ctx) return SSD_ERR_BAD_ARG;
    switch (knob) {
    case SSD_TUNE_LOW_PLANE: if (value != 0 && value != 1) return SSD_ERR_BAD_ARG; ctx->use_lo = value; break;
    case SSD_TUNE_DEPENDENT_LAUNCH: if (value != 0 && value != 1) return SSD_ERR_BAD_ARG; ctx->pdl = value; break;
    case SSD_TUNE_GRAPH: if (value != 0 && value != 1) return SSD_ERR_BAD_ARG; ctx->use_graph = value; break;
    case SSD_TUNE_GEMM_CTAS: if (value < 0 || value > 4096) return SSD_ERR_BAD_ARG; ctx->gemm_grid = value; break;
    case SSD_TUNE_KERNEL_TRACE: if (value != 0 && value != 1) return SSD_ERR_BAD_ARG; ctx->trace_kernels = value; ctx->trace_count = 0; break;
    case SSD_TUNE_HEAD_CTAS: if (value < 0 || value > 4096) return SSD_ERR_BAD_ARG; ctx->head_grid = value; break;
    case SSD_TUNE_CLUSTER_REDUCE: if (value != 0 && value != 1) return SSD_ERR_BAD_ARG; ctx->use_cluster = value; break;
    case SSD_TUNE_ATTN_LOW_PLANE: if (value != 0 && value != 1) return SSD_ERR_BAD_ARG; ctx->attn_lo = value; break;
    case SSD_TUNE_HEAD_STATS: if (value != 0 && value != 1) return SSD_ERR_BAD_ARG; ctx->use_head_stats = value; ctx->head_logits = nullptr; break;
    case SSD_TUNE_STAGE_KV_FROM: if (value < 0 || value > SSD_MAX_NODES + 1) return SSD_ERR_BAD_ARG; ctx->stage_kv_from = value; break;
    case SSD_TUNE_NODE_GROUPS: if (value != 0 && value != 1) return SSD_ERR_BAD_ARG; ctx->node_groups = value; break;
    case SSD_TUNE_ATTN_STAGED_WARPS: if (value != 0 && value != 4 && value != 8) return SSD_ERR_BAD_ARG; ctx->attn_staged_warps = value; break;
    case SSD_TUNE_FUSED_GELU: if (value != 0 && value != 1) return SSD_ERR_BAD_ARG; ctx->fused_gelu = value; break;
    case SSD_TUNE_ATTN_SPLITS: if (value != 0 && value != 1 && value != 2 && value != 4) return SSD_ERR_BAD_ARG; ctx->attn_splits = value; break;
    case SSD_TUNE_W8_PLANES:
        if (!ctx->w8 || value < 2 || value > 4) return SSD_ERR_BAD_ARG;
        ctx->w8_planes = value;
        for (auto &am : ctx->act_maps) am.built = false; // (the maps' boxes hold that many planes)
        break;
    case SSD_TUNE_CLUSTER_MAX: if (value < 1 || value > 16) return SSD_ERR_BAD_ARG; ctx->cl_max = value; break;
    case SSD_TUNE_CLUSTER_QKV: case SSD_TUNE_CLUSTER_O: case SSD_TUNE_CLUSTER_FC: case SSD_TUNE_CLUSTER_PROJ:
        if (value < 0 || value > 16) return SSD_ERR_BAD_ARG;
        ctx->cl_size[knob - SSD_TUNE_CLUSTER_QKV] = value; break;
    default: return SSD_ERR_BAD_ARG;
    }
    DeviceGuard g(ctx->device);
    if (!g.ok) return SSD_ERR_CUDA;
    CU(cudaStreamSynchronize(ctx->stream));
    for (auto &row : ctx->graphs) // captured forwards bake the old setting in
        for (auto &fg : row)
            if (fg.exec) { cudaGraphExecDestroy(fg.exec); cudaGraphDestroy(fg.graph); fg.exec = nullptr; fg.graph = nullptr; }
    return SSD_OK;
}
int ssd_get_phase_trace(ssd_ctx *ctx, uint64_t *out_ns, int32_t capacity, int32_t *count) {
    if (!ctx || !out_ns || !count || capacity < 1) return SSD_ERR_BAD_ARG;
    *count = 0;
    if (!ctx->d_trace) return SSD_OK;
    DeviceGuard g(ctx->device);
    if (!g.ok) return SSD_ERR_CUDA;
    std::vector<unsigned long long> h(SSD_TRACE_SLOTS);
    CU(cudaMemcpyAsync(h.data(), ctx->d_trace, sizeof(unsigned long long) * SSD_TRACE_SLOTS, cudaMemcpyDeviceToHost, ctx->stream));
    CU(cudaStreamSynchronize(ctx->stream));
    int n = 0;
    for (; n < ctx->trace_count && n < SSD_TRACE_SLOTS && n < capacity; ++n) out_ns[n] = h[n]; // eight slots per kernel, unused ones zero
    *count = n;
    return SSD_OK;
}
int ssd_last_cuda_error(const ssd_ctx *ctx) { return ctx ? ctx->last_cuda : 0; }
int ssd_last_cuda_error_line(const ssd_ctx *ctx) { return ctx ? ctx->last_cuda_line : 0; }
int ssd_kernel_launches(const ssd_ctx *ctx, int64_t *count) {
    if (!ctx || !count) return SSD_ERR_BAD_ARG;
    *count = ctx->launches;
    return SSD_OK;
}

} // extern "C"
