/*
 * libssd - tree verification for staged speculative decoding on one B200 (sm_100a).
 *
 * The library runs the batch-1 hot path of staged speculative decoding
 * (arXiv 2308.04623): one forward pass of a GPT-2-style verifier over every node
 * of a speculative token tree (Section 3.1), the acceptance walk down the tree
 * (Section 2.3) and the append of the accepted K/V slices to the cache
 * (Section 3.1, last sentence).  The same calls verify the draft model's own
 * tree in the second stage (Section 3.2).  Every step runs in CUDA kernels of
 * this library; there is no CPU fallback.
 *
 * Conventions
 *  - All functions return an int status: SSD_OK (0) or a negative SSD_ERR_*.
 *    Nothing throws, aborts or exits across this boundary.  No global state.
 *  - "host" / "DEVICE" in a comment says where a pointer must live.
 *  - A tree is given by parent_idx: parent_idx[0] = -1 and 0 <= parent_idx[i] < i.
 *    Node 0, the root, is the last token already emitted whose K/V is not yet in
 *    the cache; the other nodes are speculated continuations.  Siblings are tried
 *    in ascending node index.  1 <= n_nodes <= max_nodes; every node must fit the
 *    context: kv_len + depth(node) < n_ctx.  Tokens lie in [0, vocab).
 *  - Work is enqueued on the stream given to ssd_create.  ssd_verify_tree and
 *    ssd_kv_commit return without waiting for the GPU; ssd_accept_tree waits once,
 *    to hand back its small host results.
 *  - Ownership: the context owns device weights and workspaces, an ssd_kv owns one
 *    sequence's cache, the caller owns every buffer it passes in.
 */
#ifndef SSD_H
#define SSD_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ssd_ctx ssd_ctx; /* device weights, workspaces; bound to one device and stream */
typedef struct ssd_kv ssd_kv;   /* one sequence's K/V cache: n_ctx + max_nodes slots per layer */

enum {
    SSD_OK = 0,
    SSD_ERR_BAD_ARG = -1,      /* NULL pointer, size or value out of range, non-finite logits */
    SSD_ERR_NOT_LOADED = -2,   /* ssd_load_weights has not succeeded on this context */
    SSD_ERR_INVALID_TREE = -3, /* parent_idx breaks the tree contract, or n_nodes out of range */
    SSD_ERR_CTX_OVERFLOW = -4, /* a node or the accepted path would pass n_ctx */
    SSD_ERR_BAD_PATH = -5,     /* commit path is not a root-to-node path of the last verified tree */
    SSD_ERR_CUDA = -6,         /* a CUDA call failed; ssd_last_cuda_error gives the code */
    SSD_ERR_TIMEOUT = -7,      /* a bounded device-side wait ran out (see ssd_last_device_status) */
    SSD_ERR_NOMEM = -8,        /* host or device allocation failed */
    SSD_ERR_UNSUPPORTED = -9   /* shape outside what the kernels handle (see ssd_create) */
};

typedef struct {
    int32_t n_layer, d_model, n_head, d_head, d_ff, vocab, n_ctx, max_nodes;
    int32_t dtype; /* 0: fp32 weights and cache; 1: bf16 weights and cache, fp32 accumulation; 2: as 1 with 8-bit matrices */
    float ln_eps;
} ssd_config;

/*
 * SSD_DTYPE_BF16_W8 (8-bit quantisation is the second item of the future-work list that closes Section 4): the model is
 * given and run as the bf16 model, but ssd_load_weights re-encodes the matrices the projections stream - w_qkv, w_o,
 * w_fc, w_proj and the output head (wte) - as e4m3 codes (1 sign, 4 exponent, 3 fraction bits) with one fp32 scale per
 * output row, halving the bytes a step reads.  The scale of a row is the smallest power of two s with max|w| <= 448 s
 * (1 for a row of zeros); code = round-to-nearest-even(w / s), saturating; the kernels compute with code * s exactly:
 * the codes go to the tensor cores as they are (the 8-bit kind of tcgen05.mma, fp32 accumulation) and the scale
 * multiplies the fp32 sums.  A matrix whose entries are already code * power-of-two values is therefore represented
 * without loss.  That instruction kind wants its other operand in an 8-bit format too, so the kernels that produce the
 * projections' inputs write each value as four e4m3 planes, x = 16 p0 + p1 + p2 / 16 + p3 / 256 to about 16
 * significant bits (what the bf16 model's hi + lo operand pair carries; |x| up to 7168 before the first plane
 * saturates); SSD_TUNE_W8_PLANES can drop the last ones.  The embedding look-up keeps the bf16 table; biases, LayerNorm
 * parameters, the attention and the cache are as with dtype 1.  SSD_TUNE_CLUSTER_REDUCE and SSD_TUNE_HEAD_STATS
 * have no effect on such a context.
 */
enum { SSD_DTYPE_F32 = 0, SSD_DTYPE_BF16 = 1, SSD_DTYPE_BF16_W8 = 2 };
enum { SSD_GREEDY = 0, SSD_SAMPLING = 1 };

typedef struct {
    int32_t mode;      /* SSD_GREEDY or SSD_SAMPLING */
    float temperature; /* sampling only, > 0 */
    int32_t top_k;     /* sampling only; 0 = off; k > 0 keeps every logit >= the k-th largest of its row */
} ssd_sampling;

/* Counter-based random state: Philox4x32-10 keyed by seed; the uniform for a decision is
 * a function of (seed, step, node) only.  ssd_accept_tree adds 1 to step. */
typedef struct {
    uint64_t seed, step;
} ssd_rng;

/* Host pointers to the model in its plain layout.  Every matrix is [out_features, in_features]
 * row-major; w_qkv stacks query, key and value rows (each head-major).  Elements are float when
 * dtype = 0 and bf16 bit patterns (uint16_t) when dtype = 1 or 2 - LayerNorm gains/biases and linear
 * biases included.  Per-layer members are arrays of n_layer pointers. */
typedef struct {
    const void *wte;   /* [vocab, d_model] token embedding, also the output head */
    const void *wpe;   /* [n_ctx, d_model] position embedding */
    const void *lnf_g, *lnf_b;
    const void *const *ln1_g, *const *ln1_b;
    const void *const *w_qkv /* [3*d_model, d_model] */, *const *b_qkv;
    const void *const *w_o /* [d_model, d_model] */, *const *b_o;
    const void *const *ln2_g, *const *ln2_b;
    const void *const *w_fc /* [d_ff, d_model] */, *const *b_fc;
    const void *const *w_proj /* [d_model, d_ff] */, *const *b_proj;
} ssd_weights;

/*
 * Create a context on CUDA device `device`, enqueueing on `cuda_stream` (a cudaStream_t passed
 * as void*; NULL = the legacy default stream).  Supported shapes: d_head = 64,
 * n_head * d_head = d_model, d_model and d_ff multiples of 64, 1 <= max_nodes <= 256,
 * n_ctx >= 2; an fp32 model also needs n_ctx + max_nodes <= 3008 (its attention's shared memory).  Allocates the device workspaces.  *out is NULL on failure.
 */
int ssd_create(const ssd_config *cfg, int device, void *cuda_stream, ssd_ctx **out);

/*
 * Copy the model to the device (host pointers, layout above).  The caller keeps its buffers
 * and may free them on return.  The paper's model is GPT-2 (Section 4).  Must succeed before
 * any verify call.  Synchronises the stream.
 */
int ssd_load_weights(ssd_ctx *ctx, const ssd_weights *w);

/*
 * Read back one 8-bit matrix of a SSD_DTYPE_BF16_W8 context (to check the encoding): which = 0 w_qkv, 1 w_o, 2 w_fc,
 * 3 w_proj of layer `layer`, 4 the output head (layer ignored).
 *   codes_out  : host, [rows, cols] bytes (e4m3 bit patterns), rows / cols those of the matrix
 *   scales_out : host, [rows] float
 * Errors: BAD_ARG (also for a context of another dtype), NOT_LOADED, CUDA.  Synchronises the stream.
 */
int ssd_w8_read(ssd_ctx *ctx, int32_t which, int32_t layer, uint8_t *codes_out, float *scales_out);

/* Cache objects.  A new or reset cache has length 0.  Rollback shortens the committed length
 * (len <= current length); rows above the length are scratch and may be overwritten. */
int ssd_kv_create(ssd_ctx *ctx, ssd_kv **out);
int ssd_kv_reset(ssd_kv *kv);
int ssd_kv_len(const ssd_kv *kv, int32_t *len);
int ssd_kv_rollback(ssd_kv *kv, int32_t len);
void ssd_kv_destroy(ssd_kv *kv);

/*
 * Tree-batched forward (Section 3.1).  Node i is placed at position kv_len + depth(i); it
 * attends to the kv_len cached rows without a mask (cross-attention with the cache) and to the
 * tree nodes that are its ancestors or itself (self-attention inside the batch, masked by the
 * tree), under one softmax.  The K/V rows of all nodes are written to scratch slots
 * kv_len + i of `kv`, apart from the committed rows; the committed length is not changed, and a
 * second verify without a commit overwrites the scratch.
 *   tokens, parent_idx : host, n_nodes int32 each (copied before return)
 *   logits_out         : DEVICE, caller-owned, [n_nodes, vocab] fp32 row-major, written
 *                        asynchronously on the context's stream
 * Errors: BAD_ARG, NOT_LOADED, INVALID_TREE, CTX_OVERFLOW (all before anything is launched), CUDA.
 */
int ssd_verify_tree(ssd_ctx *ctx, const int32_t *tokens, const int32_t *parent_idx, int32_t n_nodes,
                    ssd_kv *kv, float *logits_out);

/*
 * Acceptance walk (Section 2.3; top-k sampling as in Section 4).  Starts at the root.
 *  Greedy: at the current node take the lowest index attaining the row maximum of its logits;
 *   move to the first child carrying that token, else stop and emit it as next_token.
 *  Sampling: r = softmax(logits/T) (after the optional top-k cut) is the node's target law.
 *   Child c with token x is accepted iff u * q_c[x] < r[x], where q_c = row c of draft_probs is
 *   the law c's token was proposed from (given that its earlier siblings were refused) and
 *   u = uniform(seed, step, 2c).  A refusal replaces r by max(0, r - q_c) renormalised.  When no
 *   child is accepted, next_token is drawn from r by inverse CDF with uniform(seed, step,
 *   2*cur + 1).  This keeps the verifier's distribution exactly.
 *  The decisions are taken in fp64.
 *   logits      : DEVICE [n_nodes, vocab] fp32 (normally the output of ssd_verify_tree)
 *   draft_probs : DEVICE [n_nodes, vocab] fp32, row 0 unused; may be NULL when greedy
 *   tokens, parent_idx : host, n_nodes int32 each
 *   rng_state   : host; read, then step += 1 (also when greedy)
 *   path_out    : host, room for n_nodes int32; receives the accepted node indices, root first
 *   n_path_out, next_token_out : host scalars
 * The step emits tokens[path[1..]] followed by next_token, which is the next root.
 * Waits for the stream.  Errors: BAD_ARG (also: a visited logits row holds NaN/Inf, in which case
 * path = [0]), INVALID_TREE, CUDA.
 * Memory: the first sampling call, and a sampling call with more nodes than any before, allocates
 * [n_nodes rounded up to 32, vocab] fp64 (plus 4 KB per node) of device scratch owned by the context (every node's target law
 * and the decision taken at it are computed side by side, then the walk follows the decisions); if that allocation fails the call still succeeds, computing the visited
 * rows one after the other.
 * Deterministic mode on a bf16 model with SSD_TUNE_HEAD_STATS set: if `logits` is the buffer the context's last ssd_verify_tree wrote (same n_nodes), the walk
 * reads the row maxima the LM head left per vocabulary tile instead of the logits themselves; do not modify that buffer between
 * the two calls (or pass a copy: any other buffer is read in full).
 */
int ssd_accept_tree(ssd_ctx *ctx, const float *logits, const float *draft_probs, const int32_t *tokens,
                    const int32_t *parent_idx, int32_t n_nodes, const ssd_sampling *sampling, ssd_rng *rng_state,
                    int32_t *path_out, int32_t *n_path_out, int32_t *next_token_out);

/*
 * The same acceptance walk for callers that cannot allocate memory.  (The paper has no
 * counterpart: this is a deployment variant of ssd_accept_tree.)
 *
 * Who needs it: a serving loop that must never hit the device-wide synchronisation cudaMalloc
 * implies, or a process whose whole memory budget is owned by another allocator (a framework's
 * caching pool, a fixed arena handed out at start-up), where a cudaMalloc from a library would
 * either fail or take memory that allocator counts on.  This entry
 * point needs no ssd_ctx and calls no allocation routine, on the device or on the host: its
 * scratch (the fp64 residual distribution of the sampling rule, and a few small arrays) lives in
 * fixed device arrays that every GPU loading the library holds until the process exits
 * (0.5 MB).  That fixes the limits: vocab <= SSD_NOALLOC_MAX_VOCAB (65536) and
 * n_nodes <= 256; larger problems return SSD_ERR_UNSUPPORTED / SSD_ERR_INVALID_TREE and
 * nothing is launched.
 *
 * Arguments and results are those of ssd_accept_tree, plus the device ordinal, the stream
 * (cudaStream_t as void*, NULL = legacy default stream) and the vocabulary size, which the
 * context would otherwise supply.  logits / draft_probs are DEVICE pointers, everything else host.
 *
 * The first call on a device looks up the arrays' device addresses (cudaGetSymbolAddress); make
 * that first call before any stream capture begins.  `cuda_stream` itself must not be capturing: the
 * call copies its few result words back and waits for the stream.  All calls share the same arrays: they keep the
 * previous call's contents (nothing in them has to start at zero - every word a call reads it has
 * written first), and two calls whose kernels overlap on the GPU (different streams or threads)
 * race on them, so serialise such calls.  Waits for the stream before returning.
 */
#define SSD_NOALLOC_MAX_VOCAB 65536
int ssd_accept_tree_noalloc(int device, void *cuda_stream, const float *logits, const float *draft_probs, const int32_t *tokens,
                            const int32_t *parent_idx, int32_t n_nodes, int32_t vocab, const ssd_sampling *sampling, ssd_rng *rng_state,
                            int32_t *path_out, int32_t *n_path_out, int32_t *next_token_out);

/*
 * ssd_accept_tree with the proposal rows given as short index / value lists instead of dense rows: row c is zero except
 * row c[row_idx[c][e]] = row_val[c][e], e < entries (host arrays [n_nodes][entries], entries <= 1024; an index < 0 marks an
 * unused slot; the indices of a row are distinct).  A deterministic proposal ("the second or third most likely tokens",
 * Section 3.1) is a one-entry row with value 1, a trigram row has four entries.  Same rule, same results, same errors as
 * ssd_accept_tree on the dense rows; the kernels read the lists themselves, and a refusal - which changes the residual law
 * at the listed entries only - costs them O(entries) instead of two passes over the vocabulary.
 */
int ssd_accept_tree_sparse(ssd_ctx *ctx, const float *logits, const int32_t *row_idx, const float *row_val, int32_t entries,
                           const int32_t *tokens, const int32_t *parent_idx, int32_t n_nodes, const ssd_sampling *sampling, ssd_rng *rng_state,
                           int32_t *path_out, int32_t *n_path_out, int32_t *next_token_out);

/*
 * What a stage proposes to the stage above it (Section 3.1: a tree of likely continuations is built from the lower
 * model's distributions; Section 3.2: the lower model may itself be the verifier of a still lower one).  For each of the
 * `m` listed nodes of a verified tree (nodes: host [m], logits: DEVICE [*, vocab] as written by ssd_verify_tree):
 *   - the node's next-token law, exactly the target law ssd_accept_tree gives that node (fp64 softmax of logits /
 *     temperature over the entries kept by the top-k cut), written as an fp32 row to rows_out[j] (DEVICE [m, vocab];
 *     may be NULL) - the proposal row of children proposed from it;
 *   - `picks` (0..8) candidate next tokens, tokens_out (host [m][picks]): mode SSD_GREEDY, the most probable tokens in
 *     order (ties towards the lower id); mode SSD_SAMPLING, independent inverse-CDF draws from the law with the uniforms
 *     u(seed, step, 1024 + 16 node + t) of rng_state (Philox4x32-10 as in ssd_accept_tree).
 * Increments rng_state->step.  Waits for the stream.  Errors: BAD_ARG (also: a listed row holds a non-finite logit), NOMEM, CUDA.
 */
int ssd_propose_children(ssd_ctx *ctx, const float *logits, const int32_t *nodes, int32_t m, int32_t picks, const ssd_sampling *sampling,
                         ssd_rng *rng_state, float *rows_out, int32_t *tokens_out);

/*
 * Append the accepted slices (Section 3.1): for every layer, scratch row kv_len + path[j] becomes
 * committed row kv_len + j, in place; kv_len += n_path.  `path` (host) must start at the root and
 * each entry must be a child of the one before in the tree of the last ssd_verify_tree on `kv`
 * (else BAD_PATH); one commit per verify.  Errors: BAD_ARG, BAD_PATH, CTX_OVERFLOW, CUDA.
 */
int ssd_kv_commit(ssd_ctx *ctx, ssd_kv *kv, const int32_t *path, int32_t n_path);

/* Inspection helper for tests: copy rows [slot0, slot0+rows) of layer `layer` (which: 0 = K,
 * 1 = V) to host as fp32 [rows, d_model] (head-major inside a row).  Waits for the stream. */
int ssd_kv_read(ssd_ctx *ctx, const ssd_kv *kv, int32_t layer, int32_t which, int32_t slot0, int32_t rows,
                float *out_host);

/*
 * Performance knobs of the bf16 path (defaults in brackets); results stay within the stated
 * tolerances for every setting.  Waits for the stream and drops the captured graphs.
 *   SSD_TUNE_LOW_PLANE [1]        feed activations to the tensor cores as bf16 hi + lo pairs
 *   SSD_TUNE_ATTN_LOW_PLANE [0]   the same for the queries and softmax weights inside the attention kernel (off: one bf16 value each,
 *                                 which rounds them as coarsely as the bf16 cache already rounds K and V; 6.5e-3 -> 7.4e-3 maximum logit
 *                                 error at the GPT-2-large shape, 30 us per step faster)
 *   SSD_TUNE_DEPENDENT_LAUNCH [1] programmatic dependent launch between the forward's kernels
 *   SSD_TUNE_GRAPH [1]            replay one captured CUDA graph per tree size
 *   SSD_TUNE_GEMM_CTAS [0]        CTAs per projection kernel of the layers; 0 = choose (two per SM for small trees, else one)
 *   SSD_TUNE_CLUSTER_REDUCE [0]   trees of up to 64 nodes: reduce every projection's split-K partial sums inside a thread-block
 *                                 cluster and fuse LayerNorm / GELU / residual into its epilogue (5 launches per layer instead
 *                                 of 8, layers reproducible bit for bit; measured slower than the default so far)
 *   SSD_TUNE_CLUSTER_MAX [8]      largest cluster (CTAs per output tile) of that path, 1..16
 *   SSD_TUNE_CLUSTER_QKV / _O / _FC / _PROJ [0]  cluster size of one of the four projections of a layer; 0 = choose
 *   SSD_TUNE_HEAD_CTAS [0]        CTAs of the LM-head projection; 0 = as the layers'
 *   SSD_TUNE_HEAD_STATS [0]       the LM head runs one CTA per 128-word tile of the vocabulary over the whole width (complete sums,
 *                                 plain stores, no clearing of the logits) and leaves per (row, tile) the maximum, its lowest index
 *                                 and a non-finite flag; a greedy ssd_accept_tree on the buffer the last ssd_verify_tree of the
 *                                 context wrote (same n_nodes, buffer not modified in between) reads those instead of the logits.
 *                                 Measured: the forward 10 us slower (393 tiles over 296 CTA slots leave a ragged last wave), the
 *                                 acceptance 10 us faster.  0 = stream-K head adding partial sums at L2 into cleared logits
 *   SSD_TUNE_W8_PLANES [4]        SSD_DTYPE_BF16_W8 only: how many e4m3 planes of an activation the projections use, 2..4 (each carries
 *                                 4 significant bits; every plane less shortens the projections' epilogues)
 *   SSD_TUNE_STAGE_KV_FROM [128]  bf16 models: trees of at least this many nodes get one more kernel per layer, which writes the tree's
 *                                 K / V rows to the cache's scratch slots so that the attention reads every key block from the cache
 *                                 (otherwise each 16-node tile of a head converts and stages the whole tree's keys itself); 0 = never
 *                                 (whatever the value, other than 0, trees of 64 nodes or more also take that path when heads x 16-node
 *                                 tiles exceed the SM count: the self-staging CTAs, one per SM, would run in two waves)
 *   SSD_TUNE_ATTN_STAGED_WARPS [0] warps of an attention CTA on that path: 4 (three CTAs per SM), 8 (two per SM, half as many key blocks per
 *                                 warp); 0 = eight when two CTAs per SM hold every (head, 16-node tile) at once, else four
 *   SSD_TUNE_ATTN_SPLITS [0]      bf16 models: CTAs (one thread-block cluster) that share a (head, 16-node tile) of the attention, each
 *                                 with a part of the keys, merged in the first one's shared memory: 1, 2 or 4; 0 = from the prefix
 *                                 length of each call (1 up to 19 key blocks of 16, 2 up to 27, else 4)
 *   SSD_TUNE_NODE_GROUPS [1]      bf16 models, trees of more than 128 nodes: the layers' projections run on node groups of 64 (one
 *                                 copy of a 64-node tree's CTA arrangement per group) instead of on the whole batch per CTA
 *   SSD_TUNE_FUSED_GELU [0]       bf16 models, both planes, at most 64 nodes per CTA of the projections: the feed-forward block's
 *                                 back-projection reads the fp32 sums of the first projection and makes its gelu(.) operand planes
 *                                 itself (one kernel fewer per layer; same values; measured slower: every output tile's CTAs
 *                                 convert the same values again); 0 = a separate element-wise kernel writes them
 *   SSD_TUNE_KERNEL_TRACE [0]     record a timeline of every kernel of a bf16 forward (see ssd_get_phase_trace)
 */
enum { SSD_TUNE_LOW_PLANE = 0, SSD_TUNE_DEPENDENT_LAUNCH = 1, SSD_TUNE_GRAPH = 2, SSD_TUNE_GEMM_CTAS = 3, SSD_TUNE_CLUSTER_REDUCE = 4,
       SSD_TUNE_CLUSTER_MAX = 5, SSD_TUNE_ATTN_LOW_PLANE = 6, SSD_TUNE_HEAD_CTAS = 7, SSD_TUNE_KERNEL_TRACE = 8, SSD_TUNE_CLUSTER_QKV = 9, SSD_TUNE_CLUSTER_O = 10,
       SSD_TUNE_CLUSTER_FC = 11, SSD_TUNE_CLUSTER_PROJ = 12, SSD_TUNE_HEAD_STATS = 13, SSD_TUNE_W8_PLANES = 14, SSD_TUNE_STAGE_KV_FROM = 15, SSD_TUNE_ATTN_SPLITS = 16, SSD_TUNE_NODE_GROUPS = 17, SSD_TUNE_FUSED_GELU = 18, SSD_TUNE_ATTN_STAGED_WARPS = 19 };
int ssd_set_tuning(ssd_ctx *ctx, int32_t knob, int32_t value);

/*
 * Per-kernel timeline of the last bf16 forward run with SSD_TUNE_KERNEL_TRACE set: eight nanosecond device
 * timestamps per kernel, in launch order: the first CTA's time of entry, of its dependencies being met, of
 * its end and (projections) of its first complete accumulator, then the same four of the last CTA, except that
 * the seventh value is the latest end over all CTAs; unused slots are zero.  `out_ns` (host) receives up to
 * `capacity` values, `count` how many.  Waits for the stream.  A profiling aid.
 */
int ssd_get_phase_trace(ssd_ctx *ctx, uint64_t *out_ns, int32_t capacity, int32_t *count);

/* Message for a status code (static string). */
const char *ssd_strerror(int status);
/* Device-side status word of the last launches (0 = clean; non-zero: a bounded wait gave up). */
int ssd_last_device_status(ssd_ctx *ctx, int32_t *word);
/*
 * Failure handling of the device-side waits.  Every wait inside the kernels (on an mbarrier that a copy, an MMA or
 * another warp completes) is bounded; when one expires the kernel records a non-zero word, leaves its loops, frees
 * its tensor memory and returns, and every later projection kernel of the context becomes a no-op while the word is
 * set.  ssd_accept_tree - the step's one synchronisation point - reads the word with its results and returns
 * SSD_ERR_TIMEOUT when it is set.  ssd_reset_device_status clears the word (waits for the stream); the context is
 * then usable again.  ssd_debug_expire_wait is a test hook: it enqueues a tiny kernel in which one warp waits
 * `limit_us` microseconds on an mbarrier at which nothing arrives - nothing else is in flight - and records the
 * word 0xE00, so that the whole failure path can be exercised without making a production kernel time out.
 */
int ssd_reset_device_status(ssd_ctx *ctx);
int ssd_debug_expire_wait(ssd_ctx *ctx, int32_t limit_us);
/* cudaError_t value of the last failed CUDA call on this context (0 if none). */
int ssd_last_cuda_error(const ssd_ctx *ctx);
/* Line of the library's API source file where that call failed (diagnostic aid; 0 if none). */
int ssd_last_cuda_error_line(const ssd_ctx *ctx);
/* Number of kernels this library launched on the context since creation (for benchmarks). */
int ssd_kernel_launches(const ssd_ctx *ctx, int64_t *count);

void ssd_destroy(ssd_ctx *ctx);

/*
 * The lowest speculation stage: a Katz back-off trigram model (Section 4 names it as the model that proposes tokens
 * for the small draft; Section 3.2 is the staging; the closing list of Section 4 asks for such proposers to answer
 * in under 10 microseconds).  The paper gives no formula; the reading: counts over a token stream, absolute discount
 * 0.5 at the trigram and bigram levels, back-off weights that make every level sum to one, a context never seen backs
 * off entirely, and a context's proposals are its four most probable next tokens (ties towards the lower id).
 *
 * ssd_trigram_build    counts `stream_tokens` (host, n_tokens >= 3 ids in [0, vocab)) and builds the device tables (the
 *                      answers of every context the stream contains); the handle owns them.  BAD_ARG, NOMEM, CUDA.
 * ssd_trigram_lookup   contexts (host [m][2]: the two preceding tokens, m <= 4096) -> the four best next tokens and their
 *                      probabilities (host [m][4] each).  Waits for the stream.
 * ssd_trigram_propose  fills a proposal tree on the device: node 0 holds `root`, which `prev1` precedes; the children of a
 *                      node, in index order, receive the best continuations of (the token before the node, the node's
 *                      token).  parent_idx as in ssd_verify_tree, at most four children per node (else INVALID_TREE).
 *                      tokens_out / probs_out: host [n_nodes] (probs_out[0] = 0).  One warp, four dependent table
 *                      look-ups for the eight-node tree of the stage-two configuration.  Waits for the stream.
 * ssd_trigram_contexts number of distinct two-token contexts in the table.
 */
typedef struct ssd_trigram ssd_trigram;
int ssd_trigram_build(const int32_t *stream_tokens, int64_t n_tokens, int32_t vocab, int device, void *cuda_stream, ssd_trigram **out);
int ssd_trigram_lookup(ssd_trigram *t, const int32_t *contexts, int32_t m, int32_t *tokens_out, float *probs_out);
int ssd_trigram_propose(ssd_trigram *t, int32_t prev1, int32_t root, const int32_t *parent_idx, int32_t n_nodes, int32_t *tokens_out,
                        float *probs_out);
int ssd_trigram_contexts(const ssd_trigram *t, int64_t *count);
void ssd_trigram_destroy(ssd_trigram *t);

#ifdef __cplusplus
}
#endif
#endif /* SSD_H */
