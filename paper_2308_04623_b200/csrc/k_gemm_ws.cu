// Weight-streaming small-M projection on the 5th-generation tensor cores (bf16 path).
//
//   Y[i, o] += sum_k X[i, k] * W[o, k]   (+ bias[o] once),   i < n nodes (n <= 256), o < out
//
// The batch (tree size) is small and every weight is used once per step, so the kernel is
// bound by reading W from HBM (Section 2.2 of the paper: batch-1 decoding has arithmetic
// intensity ~1; a tree of n nodes raises it to ~n).  Design:
//   * roles are swapped so that the 128-wide MMA dimension runs over OUTPUT FEATURES: the
//     weight tile [128 rows x 64 k] is operand A, the activations [n_pad x 64 k] operand B,
//     the accumulator D[128 x n_pad] fp32 lives in tensor memory;
//   * weights arrive by TMA straight from their plain [out, K] row-major matrix, 128-byte
//     swizzled, into a ring of shared-memory stages; activations (bf16, optionally a second
//     "low" plane holding the rounding residual, issued as a second MMA on the same weight
//     tile) arrive by TMA, one box of the whole padded batch per plane;
//   * the work is cut into (output tile, k tile) units.  With at least as many CTAs as output tiles
//     every tile gets its own group of CTAs that share its k tiles (split-K, one epilogue per CTA:
//     the kernel ends with its slowest CTA, and one that straddles two tiles runs two epilogues);
//     otherwise the flattened unit list is cut into equal contiguous ranges, one per CTA (stream-K),
//     so every SM streams the same number of bytes whatever the matrix shape.  Partial sums are added
//     to Y with fp32 reductions at L2.  For trees of up to 64 nodes there are two CTAs per SM;
//   * warp 0 = TMA producer, warp 1 = MMA issuer (one thread), warps 2..5 = epilogue;
//   * the weight loads of a CTA are issued at its very start - before its tensor memory is
//     allocated and before the programmatic-dependent-launch wait - so the HBM stream of this
//     kernel overlaps the kernels that produce its activations;
//   * at these sizes the kernel is a chain of latencies, not a stream: the single-thread loops
//     hold no integer division and no per-unit fence or commit, and the epilogue fetches what
//     does not depend on the accumulator before it waits for it;
//   * every wait is bounded; on a time-out the CTA records an error word and unwinds;
//   * 8-bit weights (the W8 instantiation; Section 4's closing list names 8-bit quantisation as the next step): the
//     matrix is stored as e4m3 codes with one fp32 scale per output row, so half the bytes stream from HBM, and it
//     goes to the tensor cores as it is - the 8-bit kind of tcgen05.mma, 32 codes of K per instruction, a weight
//     tile of [128 rows x 128 codes] per stage.  No thread touches a weight.  The activations, which that kind wants
//     in an 8-bit format too, arrive as FOUR e4m3 planes (see w8_planes.cuh: x = 16 p0 + p1 + p2 / 16 + p3 / 256 to
//     about 16 significant bits, what the bf16 hi + lo pair carries); the planes are stacked along N, so one
//     instruction multiplies a weight slice by all four (N = 4 n_pad <= 256; two instructions for 128 rows), each
//     plane's product in accumulator columns of its own.  The epilogue adds the four with their powers of two and
//     multiplies by the row's scale.  At most 128 rows per node group (512 accumulator columns).
//   * large trees: the nodes are cut into GROUPS of 64 and the grid is `groups` copies of the CTA arrangement of a
//     64-node tree, copy g working on nodes 64 g .. 64 g + 63 (its activation boxes start at that row, its sums go
//     to those rows of Y).  The weights are not read more often for it - the copies run at the same time and the
//     tile one of them fetches is in L2 for the others - but what grows with the tree no longer lands on one CTA:
//     one instruction still covers hi and lo (N = 128), two CTAs still share an SM, the epilogue drains 64 nodes,
//     not 256, and with the CTAs spread over node groups a tile's K needs fewer splits, hence fewer partial sums.
#include <cuda.h>
#include <cstring>

#include "sm100_ptx.cuh"
#include "ssd_internal.h"
#include "act_math.cuh"

namespace {
constexpr int TILE_M = 128;                 // output features per tile (MMA M)
constexpr int TILE_K = 64;                  // bf16 elements per k tile = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;                  // k per tcgen05.mma for 16-bit inputs
constexpr int A_BYTES = TILE_M * TILE_K * 2;  // 16 KB
constexpr int MAX_STAGES = 12;
constexpr int W8_PLANES = 4;                // e4m3 planes an activation is split into
constexpr int GEMM_THREADS = 192;
constexpr int SMEM_BUDGET = 210 * 1024;   // stages of one CTA per SM (the barriers and the statistics scratch follow them)
constexpr int SMEM_BUDGET_SHARED = 106 * 1024;
#ifndef EPI_POLL_NS
#define EPI_POLL_NS 32
#endif

struct GemmParams {
    float *y;          // [n, ldy] fp32, accumulated into; null = take info->logits
    const StepInfo *info;
    const float *bias; // [out] or nullptr
    int n, n_pad;      // nodes, nodes rounded up to 16
    int out, ldy;
    int k_tiles;       // K / 64
    int n_tiles;       // ceil(out / 128)
    int stages;
    int split;         // > 0: every output tile's k tiles are shared by `split` CTAs of its own (grid = split * n_tiles); 0: stream-K ranges
    int use_lo;
    int32_t *status;   // device error word
    const float *w_scale; // W8: [out] scale of each output row's codes
    int planes;        // W8: how many of the four e4m3 planes of the activations take part (2..4)
    int row0;          // first activation row (node) of this launch (W8 with more than 128 nodes runs in two launches)
    int groups;        // node groups (1 = the whole batch); group g = CTAs [g * gridDim.x / groups, ...) on nodes g * n_pad .. (n = ALL nodes then)
    // LM head with complete sums (split == 1): plain stores instead of reductions, and per (row, output tile) the maximum,
    // its lowest index and a non-finite flag, so that greedy acceptance need not read the logits again
    int store;
    float *stat_val;   // [n, n_tiles] or null
    int32_t *stat_arg, *stat_bad;
    unsigned long long *trace; // timeline slots of this launch or null
};

struct __align__(8) Barriers {
    float stat_val[4][SSD_MAX_NODES];   // the four epilogue warps' row maxima over their 32 features (statistics epilogue)
    int32_t stat_arg[4][SSD_MAX_NODES];
    int32_t stat_bad[4];
    uint64_t full[MAX_STAGES];
    uint64_t empty[MAX_STAGES];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint64_t b_full[MAX_STAGES];        // ACT: the epilogue warps have written a stage's activation planes
    uint32_t tmem_base;
    uint32_t abort;
};

__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 2, 128;" ::: "memory"); } // the four epilogue warps

__device__ __forceinline__ void fail(const GemmParams &p, Barriers *b, int code) {
    atomicExch(p.status, code);
    atomicExch(&b->abort, 1u);
}


// (Few enough registers for three CTAs of it, or two next to the element-wise kernels' CTAs, to be resident on an SM.)
// ACT (bf16 weights, hi + lo planes, tile-aligned split, at most 64 rows per node group): the activations are not read as
// prepared planes; `map_hi` is the fp32 matrix the previous projection accumulated into, its [n_pad x 64] block of a stage
// lands where the two planes will be (the same bytes), and the epilogue warps - idle until the accumulator completes - turn
// it into gelu(.) as hi / lo planes in the swizzled layout the MMA reads.  That removes a kernel, and with it one
// hand-over between dependent kernels per layer, from the chain.
template <bool W8, bool ACT>
__global__ void __launch_bounds__(GEMM_THREADS, 3)
gemm_ws_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_hi,
               const __grid_constant__ CUtensorMap map_lo, const GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    // stage ring first (1024-byte aligned for the 128-byte swizzle), barriers after it
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int b_bytes = p.n_pad * TILE_K * 2;   // one activation plane of a stage: n_pad rows of 128 bytes (64 bf16 or 128 codes)
    const int stage_bytes = A_BYTES + b_bytes * (W8 ? p.planes : p.use_lo ? 2 : 1);
    constexpr int KT = W8 ? 2 * TILE_K : TILE_K; // elements of K per stage
    Barriers *bars = reinterpret_cast<Barriers *>(smem + (size_t)p.stages * stage_bytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // node group of this CTA, its index among the group's CTAs, the group's rows
    const int cpg = gridDim.x / p.groups, grp = blockIdx.x / cpg, bid = blockIdx.x - grp * cpg;
    const int row0 = p.row0 + grp * p.n_pad, n_rows = p.groups > 1 ? min(p.n_pad, p.n - grp * p.n_pad) : p.n;
    // this CTA's contiguous range of (tile, k tile) units
    const long long units = (long long)p.n_tiles * p.k_tiles;
    int u0, u1;
    if (p.split > 0) { // tile-aligned: no CTA straddles two output tiles, so each runs exactly one epilogue
        const int tile = bid / p.split, r = bid - tile * p.split;
        u0 = tile * p.k_tiles + (p.k_tiles * r) / p.split;
        u1 = tile * p.k_tiles + (p.k_tiles * (r + 1)) / p.split;
    } else {
        u0 = (int)((units * bid) / cpg);
        u1 = (int)((units * (bid + 1)) / cpg);
    }
    // The hi and lo planes of the activations are adjacent in a stage, so while 2 * n_pad <= 256 ONE MMA
    // covers both (N = 2 * n_pad, the lo part lands in its own accumulator columns and is added in the
    // epilogue): a tcgen05.mma costs about the same whatever N is, so this halves the tensor-pipe time.
    const bool stacked = !W8 && p.use_lo && 2 * p.n_pad <= 256;
    const int acc_cols = W8 ? p.planes * p.n_pad : stacked ? 2 * p.n_pad : p.n_pad;   // columns of one accumulator buffer
    // two accumulator buffers, so that the epilogue of one output tile overlaps the MMAs of the next - unless the CTA
    // works on a single tile (tile-aligned split): then one buffer, and more CTAs' accumulators fit the SM's tensor memory
    // (or two would not fit the 512 columns)
    const int n_acc = (p.split > 0 || 2 * acc_cols > 512) ? 1 : 2;
    const uint32_t tmem_need = (uint32_t)(n_acc * acc_cols);
    const uint32_t tmem_cols = tmem_need <= 32 ? 32u : tmem_need <= 64 ? 64u : tmem_need <= 128 ? 128u : tmem_need <= 256 ? 256u : 512u;

    ptx::pdl_launch_dependents(); // the next kernel may start: its CTAs begin their own weight prefetch as SMs have room
    if (threadIdx.x == 0) {
        ptx::trace_mark(p.trace, 0);
        for (int s = 0; s < p.stages; ++s) { ptx::mbar_init(&bars->full[s], 1); ptx::mbar_init(&bars->empty[s], 1); }
        for (int a = 0; a < 2; ++a) { ptx::mbar_init(&bars->acc_full[a], 1); ptx::mbar_init(&bars->acc_empty[a], 4); }
        if (ACT) for (int s = 0; s < p.stages; ++s) ptx::mbar_init(&bars->b_full[s], 4);
        // a device error recorded by an earlier kernel makes every later one a no-op, so that a
        // failure costs one time-out, not one per launch
        bars->abort = (*reinterpret_cast<volatile int32_t *>(p.status) != 0) ? 1u : 0u;
        ptx::fence_mbar_init();
        // Phase 1 of the producer, issued here by the same thread: weights only, for as many units as there are stages.
        // They depend neither on the previous kernel nor on this CTA's tensor memory, whose allocation (below) waits
        // while the CTAs of the previous projection still hold theirs - with more than 32 nodes two CTAs fill it.
        if (!bars->abort && u1 > u0) {
            ptx::prefetch_tensormap(&map_w);
            const uint64_t pol = ptx::policy_evict_first();
            const uint32_t tx = (uint32_t)stage_bytes;
            int tile = u0 / p.k_tiles, kt = u0 - tile * p.k_tiles;
            const int pre = min(u1 - u0, p.stages);
            for (int j = 0; j < pre; ++j) {
                ptx::mbar_arrive_expect_tx(&bars->full[j], tx);
                ptx::tma_load_2d_hint(smem + (size_t)j * stage_bytes, &map_w, kt * KT, tile * TILE_M, &bars->full[j], pol);
                if (++kt == p.k_tiles) { kt = 0; ++tile; }
            }
        }
    }
    if (warp == 1) {
        ptx::tmem_alloc(&bars->tmem_base, tmem_cols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;
    const bool skip = bars->abort != 0;

    if (skip) {
        // nothing to do
    } else if (warp == 0) {
        // ===================== TMA producer =====================
        if (lane == 0 && u1 > u0) {
            if (W8 || ACT || !p.use_lo) ptx::prefetch_tensormap(&map_hi);
            else ptx::prefetch_tensormap(&map_lo);
            const uint64_t pol = ptx::policy_evict_first();
            const uint32_t tx = (uint32_t)stage_bytes;
            // (phase 1, the weight tiles of the first `pre` units, was issued before the CTA-wide set-up barrier)
            const int pre = min(u1 - u0, p.stages);
            // (one integer division per role, none per unit: for one thread a division is ~150 cycles, and several per unit
            //  used to cost more than the unit's loads and tensor-core instructions)
            int tile = u0 / p.k_tiles, kt = u0 - tile * p.k_tiles, s = 0, round = 0;
            ptx::pdl_grid_wait(); // activations are produced by the previous kernel
            ptx::trace_mark(p.trace, 1);
            bool ok = true;
            for (int u = u0; u < u1 && ok; ++u) {
                const int j = u - u0;
                uint8_t *st = smem + (size_t)s * stage_bytes;
                if (j >= pre) {
                    if (!ptx::mbar_wait_bounded(&bars->empty[s], (round - 1) & 1)) { fail(p, bars, 0x100 + s); ok = false; break; }
                    ptx::mbar_arrive_expect_tx(&bars->full[s], tx);
                    ptx::tma_load_2d_hint(st, &map_w, kt * KT, tile * TILE_M, &bars->full[s], pol);
                }
                // (the activation maps' box is the whole padded batch: one operation per plane; W8: one for the four planes)
                if (W8) {
                    ptx::tma_load_3d(st + A_BYTES, &map_hi, kt * KT, row0, 0, &bars->full[s]);
                } else if (ACT) { // the fp32 block [n_pad x 64]: as many bytes as the two planes made from it
                    ptx::tma_load_2d(st + A_BYTES, &map_hi, kt * TILE_K, row0, &bars->full[s]);
                } else {
                    // (with the lo plane: ONE box over both planes - they are adjacent in memory as in the stage - since every copy
                    //  this one thread issues costs it some 50-100 ns ahead of the first MMA)
                    if (p.use_lo) ptx::tma_load_3d(st + A_BYTES, &map_lo, kt * TILE_K, row0, 0, &bars->full[s]);
                    else ptx::tma_load_2d(st + A_BYTES, &map_hi, kt * TILE_K, row0, &bars->full[s]);
                }
                if (bars->abort) ok = false;
                if (++kt == p.k_tiles) { kt = 0; ++tile; }
                if (++s == p.stages) { s = 0; ++round; }
            }
            if (!ok) {
                // a failed wait: let the copies already in flight land before shared memory is released
                for (int s = 0; s < p.stages; ++s) ptx::mbar_wait_bounded(&bars->full[s], 0, 20000000ll);
            }
        }
    } else if (warp == 1) {
        // ===================== MMA issuer =====================
        if (lane == 0) {
            // (W8: the stacked planes are 4 n_pad rows of B; an instruction takes at most 256 of them)
            const int n_mma = (W8 && acc_cols > 256) ? 2 : 1, mma_n = acc_cols / n_mma;
            const uint32_t idesc = W8 ? ptx::umma_idesc_e4m3(TILE_M, mma_n) : ptx::umma_idesc_bf16(TILE_M, mma_n);
            int seg = 0;
            bool ok = true;
            int kt = u0 % p.k_tiles, s = 0, round = 0; // (kept incrementally: no integer division inside the loop)
            // (no stage can be complete before the previous kernel has produced the activations: wait for that in hardware rather
            //  than by polling the first stage's barrier next to the CTAs that are still at work on this SM)
            ptx::pdl_grid_wait();
            for (int u = u0; u < u1 && ok; ++u) {
                const int j = u - u0;
                const bool seg_first = (u == u0) || (kt == 0);
                const bool seg_last = (u + 1 == u1) || (kt + 1 == p.k_tiles);
                const int ab = n_acc == 2 ? seg & 1 : 0, use = n_acc == 2 ? seg >> 1 : seg; // buffer, and how often it was used before
                if (seg_first && use >= 1) { // accumulator buffer reuse: wait until the epilogue drained it
                    if (!ptx::mbar_wait_bounded(&bars->acc_empty[ab], (use - 1) & 1)) { fail(p, bars, 0x200 + ab); ok = false; break; }
                    ptx::tc_fence_after_sync();
                }
                if (!ptx::mbar_wait_bounded(&bars->full[s], round & 1)) { fail(p, bars, 0x300 + s); ok = false; break; }
                if (ACT && !ptx::mbar_wait_bounded(&bars->b_full[s], round & 1)) { fail(p, bars, 0x500 + s); ok = false; break; }
                // (no tcgen05 fence here: the stage was filled through the asynchronous proxy and its completion observed on
                //  the mbarrier; a fence per unit made the issuing thread wait out the MMAs in flight, ~0.6 us each time)
                const uint32_t a_addr = ptx::smem_u32(smem + (size_t)s * stage_bytes);
                const uint32_t b_addr = a_addr + A_BYTES;
                const uint32_t d_addr = tmem_base + (uint32_t)(ab * acc_cols);
#pragma unroll
                for (int k = 0; k < TILE_K / UMMA_K; ++k) { // (four slices of 32 bytes of K, for either kind)
                    const uint64_t da = ptx::umma_desc_k_sw128(a_addr + k * UMMA_K * 2);
                    if (W8) {
                        for (int g = 0; g < n_mma; ++g)
                            ptx::umma_e4m3(d_addr + g * mma_n, da, ptx::umma_desc_k_sw128(b_addr + g * mma_n * 128 + k * 32), idesc, (seg_first && k == 0) ? 0u : 1u);
                    } else {
                        ptx::umma_bf16(d_addr, da, ptx::umma_desc_k_sw128(b_addr + k * UMMA_K * 2), idesc, (seg_first && k == 0) ? 0u : 1u);
                        if (p.use_lo && !stacked) ptx::umma_bf16(d_addr, da, ptx::umma_desc_k_sw128(b_addr + b_bytes + k * UMMA_K * 2), idesc, 1u);
                    }
                }
                if (j + p.stages < u1 - u0) ptx::umma_commit(&bars->empty[s]); // hand the stage back (only if a later unit of this CTA reuses it)
                if (seg_last) { ptx::umma_commit(&bars->acc_full[ab]); ++seg; }
                if (bars->abort) ok = false;
                if (++kt == p.k_tiles) kt = 0;
                if (++s == p.stages) { s = 0; ++round; }
            }
        }
    } else {
        // ===================== epilogue (warps 2..5) =====================
        const int quarter = warp & 3; // TMEM lanes a warp may touch: 32 * (warp id % 4) ...
        ptx::pdl_grid_wait();         // Y may still be read or written by the previous kernels
        float *const y = p.y ? p.y : p.info->logits;
        const int et = threadIdx.x - 64; // 0..127 among the epilogue threads
        int seg = 0;
        bool ok = true;
        if (ACT) {
            // Stage by stage: wait for the fp32 block, take it into registers (thread -> (row, 8 columns): 32 bytes), meet - the
            // planes overwrite the block - then write gelu(.) as bf16 hi and lo, 16 bytes each, where the 128-byte swizzle puts
            // chunk c of row r: at chunk c ^ (r & 7).  Rows past the tree (or the group) become zeros.
            const int iters = p.n_pad >> 4;     // 8 chunks per row, 128 threads: n_pad / 16 chunks per thread (at most 4)
            int s = 0, round = 0;
            for (int u = u0; u < u1; ++u) {
                int good = 1;
                if (lane == 0) good = ptx::mbar_wait_bounded<EPI_POLL_NS>(&bars->full[s], round & 1) ? 1 : 0;
                good = __shfl_sync(0xffffffffu, good, 0);
                if (!good && lane == 0) fail(p, bars, 0x600 + s);
                uint8_t *const blk = smem + (size_t)s * stage_bytes + A_BYTES;
                float4 v[4][2];
#pragma unroll
                for (int it = 0; it < 4; ++it)
                    if (it < iters && good) {
                        const int id = et + it * 128, r = id >> 3, c = id & 7;
                        const float4 *src = reinterpret_cast<const float4 *>(blk + r * 256 + c * 32);
                        v[it][0] = src[0]; v[it][1] = src[1];
                    }
                epi_sync();
                if (*reinterpret_cast<volatile uint32_t *>(&bars->abort)) { ok = false; break; } // (the same answer in all four warps)
#pragma unroll
                for (int it = 0; it < 4; ++it)
                    if (it < iters) {
                        const int id = et + it * 128, r = id >> 3, c = id & 7;
                        uint4 hi = make_uint4(0u, 0u, 0u, 0u), lo = hi;
                        if (r < n_rows) {
                            const float g[8] = {act::gelu_tanh_fast(v[it][0].x), act::gelu_tanh_fast(v[it][0].y), act::gelu_tanh_fast(v[it][0].z),
                                                act::gelu_tanh_fast(v[it][0].w), act::gelu_tanh_fast(v[it][1].x), act::gelu_tanh_fast(v[it][1].y),
                                                act::gelu_tanh_fast(v[it][1].z), act::gelu_tanh_fast(v[it][1].w)};
                            act::split8_bf16(g, hi, lo);
                        }
                        const int at = r * 128 + ((c ^ (r & 7)) << 4);
                        *reinterpret_cast<uint4 *>(blk + at) = hi;
                        *reinterpret_cast<uint4 *>(blk + b_bytes + at) = lo;
                    }
                ptx::fence_proxy_async_smem(); // the tensor cores read shared memory through the asynchronous proxy
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&bars->b_full[s]);
                if (++s == p.stages) { s = 0; ++round; }
            }
        }
        for (int u = u0; u < u1;) { // (no early exit: the four warps must meet at the same barriers)
            const int tile = u / p.k_tiles;
            const int seg_end = min(u1, (tile + 1) * p.k_tiles);
            const bool has_k0 = (u % p.k_tiles) == 0;
            const int ab = n_acc == 2 ? seg & 1 : 0, use = n_acc == 2 ? seg >> 1 : seg;
            // (what does not depend on the accumulator is fetched before waiting for it)
            const int o = tile * TILE_M + quarter * 32 + lane;
            const float bias = (has_k0 && p.bias && o < p.out) ? p.bias[o] : 0.f;
            const float scale = (W8 && o < p.out) ? p.w_scale[o] : 1.f;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(ab * acc_cols);
            // one lane per warp polls (spinning threads would compete with the tensor cores for shared memory)
            int good = ok ? 1 : 0;
            if (lane == 0 && good) good = ptx::mbar_wait_bounded<EPI_POLL_NS>(&bars->acc_full[ab], use & 1) ? 1 : 0;
            good = __shfl_sync(0xffffffffu, good, 0);
            if (!good) { if (lane == 0) fail(p, bars, 0x400 + ab); ok = false; }
            if (seg == 0 && et == 0) ptx::trace_mark(p.trace, 3); // first accumulator complete
            ptx::tc_fence_after_sync();
            int warp_bad = 0;
            if (W8) { // the planes' products of sixteen rows at a time: acc = 16 a0 + a1 + a2 / 16 + a3 / 256, times the row's scale
                // (draining the accumulator is what this epilogue takes its time for - tensor memory reads at a fixed rate per SM - so
                //  every plane left out shortens it)
                for (int c0 = 0; c0 < p.n_pad && good; c0 += 16) { // (the loads are warp-wide: every lane runs the loop)
                    uint32_t a0[16], a1[16], a2[16], a3[16];
                    ptx::tmem_ld_32x16(taddr + c0, a0);
                    ptx::tmem_ld_32x16(taddr + p.n_pad + c0, a1);
                    if (p.planes > 2) ptx::tmem_ld_32x16(taddr + 2 * p.n_pad + c0, a2);
                    if (p.planes > 3) ptx::tmem_ld_32x16(taddr + 3 * p.n_pad + c0, a3);
                    ptx::tmem_ld_wait();
                    if (o < p.out) {
                        float *yo = y + (size_t)(row0 + c0) * p.ldy + o;
                        const int rows = min(16, n_rows - c0);
#pragma unroll
                        for (int t = 0; t < 16; ++t, yo += p.ldy) {
                            const float hi = fmaf(16.f, __uint_as_float(a0[t]), __uint_as_float(a1[t]));
                            float lo = p.planes > 2 ? __uint_as_float(a2[t]) : 0.f;
                            if (p.planes > 3) lo = fmaf(0.0625f, __uint_as_float(a3[t]), lo);
                            if (t < rows) ptx::red_add_f32(yo, fmaf(fmaf(0.0625f, lo, hi), scale, bias));
                        }
                    }
                }
            }
            for (int c0 = 0; c0 < p.n_pad && good && !W8; c0 += 16) {
                uint32_t r[16], q[16];
                ptx::tmem_ld_32x16(taddr + c0, r);
                if (stacked) ptx::tmem_ld_32x16(taddr + p.n_pad + c0, q); // the lo plane's part of the product
                ptx::tmem_ld_wait();
                if (p.store) { // this CTA holds the complete sums of its tile: plain stores, and the rows' statistics over the tile
                    float v[16];
#pragma unroll
                    for (int t = 0; t < 16; ++t) {
                        v[t] = __uint_as_float(r[t]) + (stacked ? __uint_as_float(q[t]) : 0.f) + bias;
                        if (o < p.out && c0 + t < n_rows) y[(size_t)(row0 + c0 + t) * p.ldy + o] = v[t];
                    }
                    if (p.stat_val) {
                        // row maximum over this warp's 32 features with one warp-wide integer reduction per row: floats map to
                        // unsigned keys of the same order; the lowest lane holding the maximum is the lowest index
#pragma unroll
                        for (int t = 0; t < 16; ++t) {
                            const bool live = o < p.out;
                            warp_bad |= (live && c0 + t < n_rows && !isfinite(v[t])) ? 1 : 0;
                            const unsigned bits = __float_as_uint(v[t]);
                            unsigned key = (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
                            if (!live || v[t] != v[t]) key = 0u;       // (padding features and NaNs never win; the flag reports NaNs)
                            const unsigned top = __reduce_max_sync(0xffffffffu, key);
                            const unsigned who = __ballot_sync(0xffffffffu, key == top);
                            if (lane == 0 && c0 + t < n_rows) {
                                bars->stat_val[quarter][c0 + t] = top == 0u ? -INFINITY : __uint_as_float((top & 0x80000000u) ? (top & 0x7fffffffu) : ~top);
                                bars->stat_arg[quarter][c0 + t] = tile * TILE_M + quarter * 32 + (__ffs(who) - 1);
                            }
                        }
                    }
                } else if (o < p.out) {
                    float *yo = y + (size_t)(row0 + c0) * p.ldy + o;
                    if (stacked && c0 + 16 <= n_rows) { // the usual case, kept short: sixteen full rows, hi + lo columns
#pragma unroll
                        for (int t = 0; t < 16; ++t, yo += p.ldy) ptx::red_add_f32(yo, __uint_as_float(r[t]) + __uint_as_float(q[t]) + bias);
                    } else {
#pragma unroll
                        for (int t = 0; t < 16; ++t) {
                            const int i = c0 + t;
                            if (i < n_rows) {
                                float v = __uint_as_float(r[t]) + (stacked ? __uint_as_float(q[t]) : 0.f) + bias;
                                ptx::red_add_f32(yo + (size_t)t * p.ldy, v);
                            }
                        }
                    }
                }
            }
            if (p.store && p.stat_val) { // the four warps' 32-feature shares -> one (maximum, lowest index, flag) per row and tile
                warp_bad = __any_sync(0xffffffffu, warp_bad);
                if (lane == 0) bars->stat_bad[quarter] = warp_bad;
                epi_sync();
                for (int i = et; i < p.n; i += 128) {
                    float best = bars->stat_val[0][i];
                    int arg = bars->stat_arg[0][i];
#pragma unroll
                    for (int w = 1; w < 4; ++w)
                        if (bars->stat_val[w][i] > best || (bars->stat_val[w][i] == best && bars->stat_arg[w][i] < arg)) { best = bars->stat_val[w][i]; arg = bars->stat_arg[w][i]; }
                    const size_t at = (size_t)i * p.n_tiles + tile;
                    p.stat_val[at] = good ? best : -INFINITY;
                    p.stat_arg[at] = arg;
                    p.stat_bad[at] = (bars->stat_bad[0] | bars->stat_bad[1] | bars->stat_bad[2] | bars->stat_bad[3]) ? 1 : 0;
                }
                epi_sync();
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&bars->acc_empty[ab]);
            ++seg;
            u = seg_end;
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, tmem_cols);
    }
    if (threadIdx.x == 0) ptx::trace_mark(p.trace, 2);
}

// ---- host side ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}
} // namespace

// A bf16 row-major matrix [rows, cols] (cols a multiple of 64) as a 2-D tensor map with boxes
// of [box_rows, 64] and the 128-byte swizzle; out-of-range rows read as zero.
int make_tensor_map_bf16(void *map_out, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return SSD_ERR_CUDA;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {TILE_K, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn((CUtensorMap *)map_out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SSD_OK : SSD_ERR_CUDA;
}

// 8-bit operands.  Weights: codes [rows, cols] row-major (cols a multiple of 64), boxes of [box_rows, 128 codes], 128-byte
// swizzle; a box that reaches past the matrix reads zeros (cols need not be a multiple of 128).
int make_tensor_map_u8(void *map_out, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return SSD_ERR_CUDA;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols};
    cuuint32_t box[2] = {2 * TILE_K, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn((CUtensorMap *)map_out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SSD_OK : SSD_ERR_CUDA;
}
// Activations: four planes [4][rows][cols] of codes; ONE box takes [the first box_planes planes][box_rows][128 codes].
int make_tensor_map_u8_planes(void *map_out, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows, uint32_t box_planes) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return SSD_ERR_CUDA;
    cuuint64_t dims[3] = {cols, rows, W8_PLANES};
    cuuint64_t strides[2] = {cols, rows * cols};
    cuuint32_t box[3] = {2 * TILE_K, box_rows, box_planes};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn((CUtensorMap *)map_out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SSD_OK : SSD_ERR_CUDA;
}

// The bf16 hi and lo planes of an activation buffer, adjacent in memory ([2][rows][cols]): ONE box takes [2][box_rows][64].
int make_tensor_map_bf16_pair(void *map_out, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return SSD_ERR_CUDA;
    cuuint64_t dims[3] = {cols, rows, 2};
    cuuint64_t strides[2] = {cols * 2, rows * cols * 2};
    cuuint32_t box[3] = {TILE_K, box_rows, 2};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn((CUtensorMap *)map_out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SSD_OK : SSD_ERR_CUDA;
}

// Pipeline depth.  With `shared_sm` (more CTAs than SMs) a CTA takes at most half an SM's shared memory, so that two
// are resident and one's tensor-core and epilogue phases overlap the other's loads.
int gemm_ws_stages(int n_pad, int planes, bool shared_sm) {
    const int stage_bytes = A_BYTES + n_pad * TILE_K * 2 * planes;
    int s = (shared_sm ? SMEM_BUDGET_SHARED : SMEM_BUDGET) / stage_bytes;
    return s > MAX_STAGES ? MAX_STAGES : (s < 2 ? 2 : s);
}

cudaError_t gemm_ws_prepare() {
    cudaError_t e = cudaSuccess;
    const void *kernels[] = {(const void *)gemm_ws_kernel<false, false>, (const void *)gemm_ws_kernel<true, false>, (const void *)gemm_ws_kernel<false, true>};
    for (const void *k : kernels) {
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(k, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    }
    return e;
}

// An fp32 row-major matrix [rows, cols] (cols a multiple of 64) as a 2-D tensor map with boxes of [box_rows, 64], not
// swizzled; out-of-range rows read as zero.
int make_tensor_map_f32(void *map_out, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return SSD_ERR_CUDA;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 4};
    cuuint32_t box[2] = {TILE_K, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn((CUtensorMap *)map_out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SSD_OK : SSD_ERR_CUDA;
}

cudaError_t launch_gemm_ws(const void *map_w, const void *map_hi, const void *map_lo, float *y, const StepInfo *info, int ldy,
                           const float *bias, int n, int K, int out, int use_lo, int grid, int sm_count, int32_t *status, bool pdl,
                           cudaStream_t s, unsigned long long *trace, const GemmHeadStats *head, const float *w_scale, int row0, int w8_planes, int group_rows, int act_gelu) {
    const bool w8 = w_scale != nullptr; // map_w: the codes; map_hi: the four activation planes
    // node groups: the activation maps' boxes hold group_rows rows (a multiple of 16), fewer than the tree has nodes
    const bool grouped = group_rows > 0 && group_rows < n;
    if (grouped && (head || (group_rows & 15) || row0 != 0)) return cudaErrorInvalidValue;
    if (w8 && ((grouped ? group_rows : n) > 128 || head || w8_planes < 2 || w8_planes > W8_PLANES)) return cudaErrorInvalidValue;
    GemmParams p;
    p.trace = trace;
    p.y = y; p.info = info; p.bias = bias; p.n = n; p.n_pad = grouped ? group_rows : (n + 15) & ~15;
    p.groups = grouped ? (n + group_rows - 1) / group_rows : 1;
    if (grouped) grid = grid / p.groups > 0 ? grid / p.groups : 1; // (the CTA count asked for is the whole launch's)
    p.out = out; p.ldy = ldy; p.k_tiles = w8 ? (K + 2 * TILE_K - 1) / (2 * TILE_K) : K / TILE_K; p.n_tiles = (out + TILE_M - 1) / TILE_M;
    p.use_lo = use_lo; p.status = status; p.w_scale = w_scale; p.row0 = row0; p.planes = w8_planes;
    p.store = 0; p.stat_val = nullptr; p.stat_arg = nullptr; p.stat_bad = nullptr;
    const int planes = w8 ? w8_planes : use_lo ? 2 : 1;
    const int stage_bytes = A_BYTES + p.n_pad * TILE_K * 2 * planes;
    const long long units = (long long)p.n_tiles * p.k_tiles;
    if (grid > units) grid = (int)units;
    int per_cta = (int)((units + grid - 1) / grid);
    p.split = 0;
    if (grid >= p.n_tiles) {
        // When there are at least as many CTAs as output tiles, give every tile its own group of CTAs: a CTA whose range
        // straddles two tiles runs two epilogues, and the kernel ends with its slowest CTA.
        int most = grid / p.n_tiles;
        if (most > p.k_tiles) most = p.k_tiles;
        per_cta = (p.k_tiles + most - 1) / most;                // the fewest units per CTA this many CTAs allow ...
        // (with 64 nodes or more, CTAs of a single unit all reach their epilogue together and their reductions onto the same
        //  rows queue up at L2: two units per CTA halve the partial sums; measured on the output projection)
        if (p.n_pad >= 64 && per_cta < 2 && p.k_tiles >= 2) per_cta = 2;
        p.split = (p.k_tiles + per_cta - 1) / per_cta;          // ... and the fewest CTAs per tile that reach it
        grid = p.split * p.n_tiles;
    }
    if (head) { // complete sums: one CTA per output tile, whatever the grid asked for
        p.split = 1; grid = p.n_tiles; per_cta = p.k_tiles;
        p.store = 1; p.stat_val = head->val; p.stat_arg = head->arg; p.stat_bad = head->bad;
    }
    p.stages = gemm_ws_stages(p.n_pad, planes, grid * p.groups > sm_count);
    if (p.stages > per_cta) p.stages = per_cta < 1 ? 1 : per_cta;
    size_t smem = (size_t)p.stages * stage_bytes + sizeof(Barriers) + 1024;
    // Two CTAs per SM, not three: with a third one resident the slowest CTA of a projection ends later (measured: 1.19 ms per
    // GPT-2-large verification of 32 nodes against 1.09 ms), so a CTA asks for more than a third of an SM's shared memory.
    if (grid * p.groups > sm_count && smem < 78 * 1024) smem = 78 * 1024;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid * p.groups);
    cfg.blockDim = dim3(GEMM_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    // (fp32 source of the activations: one tile per CTA, both planes, a block a thread can hold its share of)
    if (act_gelu && (w8 || head || !use_lo || p.split == 0 || p.n_pad > 64)) return cudaErrorInvalidValue;
    return cudaLaunchKernelEx(&cfg, w8 ? gemm_ws_kernel<true, false> : act_gelu ? gemm_ws_kernel<false, true> : gemm_ws_kernel<false, false>, *(const CUtensorMap *)map_w,
                              *(const CUtensorMap *)map_hi, *(const CUtensorMap *)(map_lo ? map_lo : map_hi), p);
}
