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
//   * 8-bit weights (the W8 instantiation; Section 4's closing list names 8-bit quantisation as the next step):
//     the matrix is stored as e4m3 codes with one fp32 scale per output row, so half the bytes stream from HBM.
//     The codes are stored tile by tile - the [128 rows x 64 codes] of an (output tile, k tile) unit are 8 KB in a row,
//     rows past the matrix zero - so a unit arrives as ONE contiguous copy (rows of 64 bytes fetched one by one from a
//     row-major matrix use a fraction of every DRAM burst and of every 256-byte L2 fetch).
//     A tile is widened on chip to bf16, in the swizzled layout the tensor cores read (both MMA operands stay bf16).
//     When a CTA has no more units than stages (the projections of a layer), a tile lands in the upper half of its
//     stage's own 16 KB weight buffer and the four epilogue warps, which have nothing else to do yet, widen it in place
//     (through registers, a barrier between the reads and the writes): the CTA has the threads and the shared memory of
//     the bf16 kernel, so the next kernels' CTAs stay resident beside it.  Otherwise (the LM head) tiles land in a
//     ring of 8 KB slots behind a short ring of stages - a deep, cheap ring that covers the HBM latency -, eight more
//     warps widen them, four units at a time (the epilogue warps help with the CTA's first units), and refill a slot
//     themselves as soon as they have read it.
//     The epilogue multiplies the sums by the row's scale.  The widening needs no activations, so it too runs ahead
//     of the dependency wait.
#include <cuda.h>
#include <cstring>

#include "sm100_ptx.cuh"
#include "ssd_internal.h"

namespace {
constexpr int TILE_M = 128;                 // output features per tile (MMA M)
constexpr int TILE_K = 64;                  // bf16 elements per k tile = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;                  // k per tcgen05.mma for 16-bit inputs
constexpr int A_BYTES = TILE_M * TILE_K * 2;  // 16 KB
constexpr int MAX_STAGES = 12;
constexpr int MAX_LANDING = 16;               // W8: landing slots
constexpr int A8_BYTES = TILE_M * TILE_K;     // 8 KB: the same tile as 8-bit codes
constexpr int GEMM_THREADS = 192;
constexpr int W8_PAIRS = 4;                   // pairs of dedicated converter warps (landing-ring mode)
constexpr int GEMM_THREADS_W8 = GEMM_THREADS + 64 * W8_PAIRS;
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
    int landing;       // W8: landing slots of 8 KB behind the stages; 0 = tiles land inside their stage (units <= stages)
    int split;         // > 0: every output tile's k tiles are shared by `split` CTAs of its own (grid = split * n_tiles); 0: stream-K ranges
    int use_lo;
    int32_t *status;   // device error word
    const float *w_scale; // [out] scale of each output row's 8-bit codes (W8 only)
    const uint8_t *w_codes; // W8: [n_tiles][k_tiles][128][64] codes
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
    uint64_t wfull[MAX_LANDING];        // W8: a landing slot's 8-bit tile has arrived
    uint64_t wempty[MAX_LANDING];       // W8: the converters have read it
    uint64_t empty[MAX_STAGES];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint32_t tmem_base;
    uint32_t abort;
};

__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 2, 128;" ::: "memory"); } // the four epilogue warps

__device__ __forceinline__ void fail(const GemmParams &p, Barriers *b, int code) {
    atomicExch(p.status, code);
    atomicExch(&b->abort, 1u);
}


// Four e4m3 codes (one 32-bit word, lowest byte first) as four bf16 values in two words.  A code's seven magnitude bits
// placed at bits 4..10 of a bf16 give the same number scaled by 2^-120, sub-normal codes included (they become sub-normal
// bf16 values with the same fraction); one packed multiplication by 2^120 - exact - restores the scale.
__device__ __forceinline__ void e4m3x4_to_bf16x4(uint32_t w, uint32_t &lo, uint32_t &hi) {
    const uint32_t x01 = __byte_perm(w, 0u, 0x1404), x23 = __byte_perm(w, 0u, 0x3424); // codes in the high byte of each half
    const uint32_t b01 = (x01 & 0x80008000u) | ((x01 >> 4) & 0x07f007f0u);
    const uint32_t b23 = (x23 & 0x80008000u) | ((x23 >> 4) & 0x07f007f0u);
    const uint32_t two120 = 0x7B807B80u;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(lo) : "r"(b01), "r"(two120));
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(hi) : "r"(b23), "r"(two120));
}

// One thread's share of widening a landed 8-bit tile [128 rows][64 bytes] into the bf16 tile of a compute stage: `items`
// 16-byte groups starting at group `first + lane` and 32 apart.  Group g = 16 codes of row g / 4 (its quarter g % 4) -> the two
// 16-byte chunks 2c, 2c + 1 of the bf16 row, each stored at chunk position (chunk ^ (row & 7)): the 128-byte swizzle the weight
// tiles otherwise get from the copy engine.  Waits (bounded) for the tile and, when given, for the stage to be free.
template <int ITEMS>
__device__ __forceinline__ bool w8_convert_unit(const GemmParams &p, Barriers *bars, uint8_t *stage, const uint8_t *src, uint64_t *landed, uint32_t landed_parity,
                                                uint64_t *stage_free, uint32_t free_parity, int first, int lane, int code) {
    int good = 1;
    if (lane == 0) {
        good = ptx::mbar_wait_bounded(landed, landed_parity) ? 1 : 0;
        if (good && stage_free) good = ptx::mbar_wait_bounded(stage_free, free_parity) ? 1 : 0;
        if (!good) fail(p, bars, code);
    }
    good = __shfl_sync(0xffffffffu, good, 0);
    if (!good) return false;
    uint4 wv[ITEMS]; // (all reads first: the compiler cannot move them across the stores itself)
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) wv[it] = *reinterpret_cast<const uint4 *>(src + (first + it * 32 + lane) * 16);
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) {
        const int idx = first + it * 32 + lane, r = idx >> 2, c = idx & 3;
        const uint4 w = wv[it];
        uint4 lo4, hi4;
        e4m3x4_to_bf16x4(w.x, lo4.x, lo4.y); e4m3x4_to_bf16x4(w.y, lo4.z, lo4.w);
        e4m3x4_to_bf16x4(w.z, hi4.x, hi4.y); e4m3x4_to_bf16x4(w.w, hi4.z, hi4.w);
        uint8_t *row = stage + r * 128;
        *reinterpret_cast<uint4 *>(row + (((2 * c) ^ (r & 7)) << 4)) = lo4;
        *reinterpret_cast<uint4 *>(row + (((2 * c + 1) ^ (r & 7)) << 4)) = hi4;
    }
    ptx::fence_proxy_async_smem(); // the tensor cores read the tile through the asynchronous proxy
    __syncwarp();
    return true;
}

// The same for a tile that landed in the upper half of the stage's own bf16 buffer [128 rows][128 bytes]: the four epilogue warps
// (`t` = 0..127) first read the whole 8-bit tile into registers, meet, and then write the bf16 tile over it.
__device__ __forceinline__ bool w8_convert_in_place(const GemmParams &p, Barriers *bars, uint8_t *stage, uint64_t *landed, uint64_t *full, int t, int lane,
                                                    int code) {
    int good = 1;
    if (lane == 0) {
        good = ptx::mbar_wait_bounded(landed, 0) ? 1 : 0;
        if (!good) fail(p, bars, code);
    }
    good = __shfl_sync(0xffffffffu, good, 0);
    const uint8_t *src = stage + A8_BYTES;
    uint4 w[4];
#pragma unroll
    for (int it = 0; it < 4; ++it)
        if (good) w[it] = *reinterpret_cast<const uint4 *>(src + (t + it * 128) * 16);
    asm volatile("bar.sync 3, 128;" ::: "memory"); // (a warp whose wait failed still meets the others here; they see the abort flag below)
    if (!good || bars->abort) return false;
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const int idx = t + it * 128, r = idx >> 2, c = idx & 3;
        {
            uint4 lo4, hi4;
            e4m3x4_to_bf16x4(w[it].x, lo4.x, lo4.y); e4m3x4_to_bf16x4(w[it].y, lo4.z, lo4.w);
            e4m3x4_to_bf16x4(w[it].z, hi4.x, hi4.y); e4m3x4_to_bf16x4(w[it].w, hi4.z, hi4.w);
            uint8_t *row = stage + r * 128;
            *reinterpret_cast<uint4 *>(row + (((2 * c) ^ (r & 7)) << 4)) = lo4;
            *reinterpret_cast<uint4 *>(row + (((2 * c + 1) ^ (r & 7)) << 4)) = hi4;
        }
    }
    ptx::fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) ptx::mbar_arrive(full);
    return true;
}

// (Few enough registers for three CTAs of it, or two next to the element-wise kernels' CTAs, to be resident on an SM.)
template <bool W8>
__global__ void __launch_bounds__(W8 ? 640 : GEMM_THREADS, W8 ? 1 : 3) // (W8: bounds that cap it at 96 registers, like the bf16 instance)

gemm_ws_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_hi,
               const __grid_constant__ CUtensorMap map_lo, const GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    // stage ring first (1024-byte aligned for the 128-byte swizzle), barriers after it
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int b_bytes = p.n_pad * TILE_K * 2;
    const int stage_bytes = A_BYTES + b_bytes * (p.use_lo ? 2 : 1);
    uint8_t *landing = smem + (size_t)p.stages * stage_bytes;     // W8: p.landing slots of A8_BYTES
    Barriers *bars = reinterpret_cast<Barriers *>(landing + (W8 ? (size_t)p.landing * A8_BYTES : 0));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // this CTA's contiguous range of (tile, k tile) units
    const long long units = (long long)p.n_tiles * p.k_tiles;
    int u0, u1;
    if (p.split > 0) { // tile-aligned: no CTA straddles two output tiles, so each runs exactly one epilogue
        const int tile = blockIdx.x / p.split, r = blockIdx.x - tile * p.split;
        u0 = tile * p.k_tiles + (p.k_tiles * r) / p.split;
        u1 = tile * p.k_tiles + (p.k_tiles * (r + 1)) / p.split;
    } else {
        u0 = (int)((units * blockIdx.x) / gridDim.x);
        u1 = (int)((units * (blockIdx.x + 1)) / gridDim.x);
    }
    // The hi and lo planes of the activations are adjacent in a stage, so while 2 * n_pad <= 256 ONE MMA
    // covers both (N = 2 * n_pad, the lo part lands in its own accumulator columns and is added in the
    // epilogue): a tcgen05.mma costs about the same whatever N is, so this halves the tensor-pipe time.
    const bool stacked = p.use_lo && 2 * p.n_pad <= 256;
    const int acc_cols = stacked ? 2 * p.n_pad : p.n_pad;   // columns of one accumulator buffer
    // two accumulator buffers, so that the epilogue of one output tile overlaps the MMAs of the next - unless the CTA
    // works on a single tile (tile-aligned split): then one buffer, and more CTAs' accumulators fit the SM's tensor memory
    const uint32_t tmem_need = (p.split > 0 ? 1u : 2u) * acc_cols;
    const uint32_t tmem_cols = tmem_need <= 32 ? 32u : tmem_need <= 64 ? 64u : tmem_need <= 128 ? 128u : tmem_need <= 256 ? 256u : 512u;

    ptx::pdl_launch_dependents(); // the next kernel may start: its CTAs begin their own weight prefetch as SMs have room
    if (threadIdx.x == 0) {
        ptx::trace_mark(p.trace, 0);
        // (W8: a stage is full when its activations have landed and the converters have arrived: the four epilogue warps when
        //  tiles land inside their stages; with the landing ring six warps' worth - six warps' one each, or the two dedicated
        //  warps' three each)
        for (int s = 0; s < p.stages; ++s) { ptx::mbar_init(&bars->full[s], W8 ? (p.landing ? 7 : 5) : 1); ptx::mbar_init(&bars->empty[s], 1); }
        if (W8) for (int l = 0; l < max(p.landing, p.stages); ++l) { ptx::mbar_init(&bars->wfull[l], 1); ptx::mbar_init(&bars->wempty[l], 6); }
        for (int a = 0; a < 2; ++a) { ptx::mbar_init(&bars->acc_full[a], 1); ptx::mbar_init(&bars->acc_empty[a], 4); }
        // a device error recorded by an earlier kernel makes every later one a no-op, so that a
        // failure costs one time-out, not one per launch
        bars->abort = (*reinterpret_cast<volatile int32_t *>(p.status) != 0) ? 1u : 0u;
        ptx::fence_mbar_init();
        // Phase 1 of the producer, issued here by the same thread: weights only, for as many units as there are stages.
        // They depend neither on the previous kernel nor on this CTA's tensor memory, whose allocation (below) waits
        // while the CTAs of the previous projection still hold theirs - with more than 32 nodes two CTAs fill it.
        if (!bars->abort && u1 > u0) {
            if (!W8) ptx::prefetch_tensormap(&map_w);
            const uint64_t pol = ptx::policy_evict_first();
            const uint32_t tx = (uint32_t)stage_bytes;
            int tile = u0 / p.k_tiles, kt = u0 - tile * p.k_tiles;
            const int pre = min(u1 - u0, (W8 && p.landing) ? p.landing : p.stages);
            for (int j = 0; j < pre; ++j) {
                if (W8) {
                    uint8_t *dst = p.landing ? landing + (size_t)j * A8_BYTES : smem + (size_t)j * stage_bytes + A8_BYTES;
                    ptx::mbar_arrive_expect_tx(&bars->wfull[j], A8_BYTES);
                    ptx::bulk_load_hint(dst, p.w_codes + (size_t)(u0 + j) * A8_BYTES, A8_BYTES, &bars->wfull[j], pol);
                } else {
                    ptx::mbar_arrive_expect_tx(&bars->full[j], tx);
                    ptx::tma_load_2d_hint(smem + (size_t)j * stage_bytes, &map_w, kt * TILE_K, tile * TILE_M, &bars->full[j], pol);
                }
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
            ptx::prefetch_tensormap(&map_hi);
            if (p.use_lo) ptx::prefetch_tensormap(&map_lo);
            const uint64_t pol = ptx::policy_evict_first();
            const uint32_t tx = (uint32_t)stage_bytes;
            // (phase 1, the weight tiles of the first `pre` units, was issued before the CTA-wide set-up barrier)
            const int pre = W8 ? 0 : min(u1 - u0, p.stages); // (W8: this thread loads activations only; the converters refill the landing slots)
            // (one integer division per role, none per unit: for one thread a division is ~150 cycles, and several per unit
            //  used to cost more than the unit's loads and tensor-core instructions)
            int tile = u0 / p.k_tiles, kt = u0 - tile * p.k_tiles, s = 0, round = 0;
            ptx::pdl_grid_wait(); // activations are produced by the previous kernel
            ptx::trace_mark(p.trace, 1);
            bool ok = true;
            for (int u = u0; u < u1 && ok; ++u) {
                const int j = u - u0;
                uint8_t *st = smem + (size_t)s * stage_bytes;
                if (W8) {
                    if (round > 0 && !ptx::mbar_wait_bounded(&bars->empty[s], (round - 1) & 1)) { fail(p, bars, 0x100 + s); ok = false; break; }
                    ptx::mbar_arrive_expect_tx(&bars->full[s], (uint32_t)(stage_bytes - A_BYTES)); // the activation planes' bytes
                } else if (j >= pre) {
                    if (!ptx::mbar_wait_bounded(&bars->empty[s], (round - 1) & 1)) { fail(p, bars, 0x100 + s); ok = false; break; }
                    ptx::mbar_arrive_expect_tx(&bars->full[s], tx);
                    ptx::tma_load_2d_hint(st, &map_w, kt * TILE_K, tile * TILE_M, &bars->full[s], pol);
                }
                // (the activation maps' box is the whole padded batch: one operation per plane)
                ptx::tma_load_2d(st + A_BYTES, &map_hi, kt * TILE_K, 0, &bars->full[s]);
                if (p.use_lo) ptx::tma_load_2d(st + A_BYTES + b_bytes, &map_lo, kt * TILE_K, 0, &bars->full[s]);
                if (bars->abort) ok = false;
                if (++kt == p.k_tiles) { kt = 0; ++tile; }
                if (++s == p.stages) { s = 0; ++round; }
            }
            if (!ok) {
                // a failed wait: let the copies already in flight land before shared memory is released
                if (W8) for (int l = 0; l < max(p.landing, p.stages); ++l) ptx::mbar_wait_bounded(&bars->wfull[l], 0, 20000000ll);
                else for (int s = 0; s < p.stages; ++s) ptx::mbar_wait_bounded(&bars->full[s], 0, 20000000ll);
            }
        }
    } else if (warp == 1) {
        // ===================== MMA issuer =====================
        if (lane == 0) {
            const uint32_t idesc = ptx::umma_idesc_bf16(TILE_M, acc_cols);
            int seg = 0;
            bool ok = true;
            int kt = u0 % p.k_tiles, s = 0, round = 0; // (kept incrementally: no integer division inside the loop)
            for (int u = u0; u < u1 && ok; ++u) {
                const int j = u - u0;
                const bool seg_first = (u == u0) || (kt == 0);
                const bool seg_last = (u + 1 == u1) || (kt + 1 == p.k_tiles);
                const int ab = seg & 1;
                if (seg_first && seg >= 2) { // accumulator buffer reuse: wait until the epilogue drained it
                    if (!ptx::mbar_wait_bounded(&bars->acc_empty[ab], ((seg >> 1) - 1) & 1)) { fail(p, bars, 0x200 + ab); ok = false; break; }
                    ptx::tc_fence_after_sync();
                }
                if (!ptx::mbar_wait_bounded(&bars->full[s], round & 1)) { fail(p, bars, 0x300 + s); ok = false; break; }
                // (no tcgen05 fence here: the stage was filled through the asynchronous proxy and its completion observed on
                //  the mbarrier; a fence per unit made the issuing thread wait out the MMAs in flight, ~0.6 us each time)
                const uint32_t a_addr = ptx::smem_u32(smem + (size_t)s * stage_bytes);
                const uint32_t b_addr = a_addr + A_BYTES;
                const uint32_t d_addr = tmem_base + (uint32_t)(ab * acc_cols);
#pragma unroll
                for (int k = 0; k < TILE_K / UMMA_K; ++k) {
                    const uint64_t da = ptx::umma_desc_k_sw128(a_addr + k * UMMA_K * 2);
                    ptx::umma_bf16(d_addr, da, ptx::umma_desc_k_sw128(b_addr + k * UMMA_K * 2), idesc, (seg_first && k == 0) ? 0u : 1u);
                    if (p.use_lo && !stacked) ptx::umma_bf16(d_addr, da, ptx::umma_desc_k_sw128(b_addr + b_bytes + k * UMMA_K * 2), idesc, 1u);
                }
                if (j + p.stages < u1 - u0) ptx::umma_commit(&bars->empty[s]); // hand the stage back (only if a later unit of this CTA reuses it)
                if (seg_last) { ptx::umma_commit(&bars->acc_full[ab]); ++seg; }
                if (bars->abort) ok = false;
                if (++kt == p.k_tiles) kt = 0;
                if (++s == p.stages) { s = 0; ++round; }
            }
        }
    } else if (W8 && warp >= 6) {
        // ===================== dedicated converters (W8 with the landing ring: warps 6..13, four pairs) =====================
        // A warp alone runs the dependent bit operations of a tile at a fraction of an instruction per cycle, so the pairs work
        // on several units at once.  Pair q OWNS stage q: it widens units q, q + stages, ... one after the other, so that its
        // parity waits on the stage's barriers always concern the phase next to the one it last saw (a pair that skipped ahead
        // over a stage's phase would take an older phase of the same parity for the one it waits for).
        const int pair = (warp - 6) >> 1, half = (warp - 6) & 1, n_units = u1 - u0;
        const int helped = min(n_units, p.stages); // units the epilogue warps help with
        const uint64_t pol = ptx::policy_evict_first();
        for (int j = pair, round = 0; j < n_units && pair < p.stages; j += p.stages, ++round) {
            const int s = pair, l = j % p.landing, lround = j / p.landing;
            const bool with_help = j < helped;
            uint8_t *st = smem + (size_t)s * stage_bytes;
            const uint8_t *src = landing + (size_t)l * A8_BYTES;
            const bool done = with_help ? w8_convert_unit<2>(p, bars, st, src, &bars->wfull[l], lround & 1, nullptr, 0, half * 64, lane, 0x500 + l)
                                        : w8_convert_unit<8>(p, bars, st, src, &bars->wfull[l], lround & 1, round > 0 ? &bars->empty[s] : nullptr,
                                                             (round - 1) & 1, half * 256, lane, 0x500 + l);
            if (!done) break;
            if (lane == 0) { // (unhelped units: the pair arrives for all six)
                ptx::mbar_arrive_n(&bars->full[s], with_help ? 1u : 3u);
                ptx::mbar_arrive_n(&bars->wempty[l], with_help ? 1u : 3u);
                if (half == 0 && j + p.landing < n_units) { // the slot is read: request the unit that lands in it next
                    if (!ptx::mbar_wait_bounded(&bars->wempty[l], lround & 1)) { fail(p, bars, 0x600 + l); }
                    else {
                        ptx::mbar_arrive_expect_tx(&bars->wfull[l], A8_BYTES);
                        ptx::bulk_load_hint(landing + (size_t)l * A8_BYTES, p.w_codes + (size_t)(u0 + j + p.landing) * A8_BYTES, A8_BYTES, &bars->wfull[l], pol);
                    }
                }
            }
            __syncwarp();
            if (bars->abort) break;
        }
        if (bars->abort && warp == 6 && lane == 0) // a failed wait somewhere: let the weight copies in flight land before shared memory is released
            for (int q = 0; q < max(p.landing, p.stages); ++q) { ptx::mbar_wait_bounded(&bars->wfull[q], 0, 10000000ll); ptx::mbar_wait_bounded(&bars->wfull[q], 1, 10000000ll); }
    } else {
        // ===================== epilogue (warps 2..5) =====================
        const int quarter = warp & 3; // TMEM lanes a warp may touch: 32 * (warp id % 4) ...
        if (W8) { // help to widen the CTA's first units (rows 32..127; the dedicated warps take rows 0..31): no epilogue is due before them
            const int helped = min(u1 - u0, p.stages);
            for (int j = 0; j < helped && p.landing == 0; ++j)
                if (!w8_convert_in_place(p, bars, smem + (size_t)j * stage_bytes, &bars->wfull[j], &bars->full[j], threadIdx.x - 64, lane, 0x700 + j)) break;
            for (int j = 0; j < helped && p.landing; ++j) // (there are at least as many landing slots as stages)
                if (!w8_convert_unit<3>(p, bars, smem + (size_t)j * stage_bytes, landing + (size_t)j * A8_BYTES, &bars->wfull[j], 0, nullptr, 0,
                                        128 + (warp - 2) * 96, lane, 0x700 + j))
                    break;
                else if (lane == 0) { ptx::mbar_arrive_n(&bars->full[j], 1u); ptx::mbar_arrive_n(&bars->wempty[j], 1u); }
        }
        ptx::pdl_grid_wait();         // Y may still be read or written by the previous kernels
        float *const y = p.y ? p.y : p.info->logits;
        const int et = threadIdx.x - 64; // 0..127 among the epilogue threads
        int seg = 0;
        bool ok = true;
        for (int u = u0; u < u1;) { // (no early exit: the four warps must meet at the same barriers)
            const int tile = u / p.k_tiles;
            const int seg_end = min(u1, (tile + 1) * p.k_tiles);
            const bool has_k0 = (u % p.k_tiles) == 0;
            const int ab = seg & 1;
            // (what does not depend on the accumulator is fetched before waiting for it)
            const int o = tile * TILE_M + quarter * 32 + lane;
            const float bias = (has_k0 && p.bias && o < p.out) ? p.bias[o] : 0.f;
            const float scale = (W8 && o < p.out) ? p.w_scale[o] : 1.f;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(ab * acc_cols);
            // one lane per warp polls (spinning threads would compete with the tensor cores for shared memory)
            int good = ok ? 1 : 0;
            if (lane == 0 && good) good = ptx::mbar_wait_bounded<EPI_POLL_NS>(&bars->acc_full[ab], (seg >> 1) & 1) ? 1 : 0;
            good = __shfl_sync(0xffffffffu, good, 0);
            if (!good) { if (lane == 0) fail(p, bars, 0x400 + ab); ok = false; }
            if (seg == 0 && et == 0) ptx::trace_mark(p.trace, 3); // first accumulator complete
            ptx::tc_fence_after_sync();
            int warp_bad = 0;
            for (int c0 = 0; c0 < p.n_pad && good; c0 += 16) {
                uint32_t r[16], q[16];
                ptx::tmem_ld_32x16(taddr + c0, r);
                if (stacked) ptx::tmem_ld_32x16(taddr + p.n_pad + c0, q); // the lo plane's part of the product
                ptx::tmem_ld_wait();
                if (p.store) { // this CTA holds the complete sums of its tile: plain stores, and the rows' statistics over the tile
                    float v[16];
#pragma unroll
                    for (int t = 0; t < 16; ++t) {
                        v[t] = (__uint_as_float(r[t]) + (stacked ? __uint_as_float(q[t]) : 0.f)) * scale + bias;
                        if (o < p.out && c0 + t < p.n) y[(size_t)(c0 + t) * p.ldy + o] = v[t];
                    }
                    if (p.stat_val) {
                        // row maximum over this warp's 32 features with one warp-wide integer reduction per row: floats map to
                        // unsigned keys of the same order; the lowest lane holding the maximum is the lowest index
#pragma unroll
                        for (int t = 0; t < 16; ++t) {
                            const bool live = o < p.out;
                            warp_bad |= (live && c0 + t < p.n && !isfinite(v[t])) ? 1 : 0;
                            const unsigned bits = __float_as_uint(v[t]);
                            unsigned key = (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
                            if (!live || v[t] != v[t]) key = 0u;       // (padding features and NaNs never win; the flag reports NaNs)
                            const unsigned top = __reduce_max_sync(0xffffffffu, key);
                            const unsigned who = __ballot_sync(0xffffffffu, key == top);
                            if (lane == 0 && c0 + t < p.n) {
                                bars->stat_val[quarter][c0 + t] = top == 0u ? -INFINITY : __uint_as_float((top & 0x80000000u) ? (top & 0x7fffffffu) : ~top);
                                bars->stat_arg[quarter][c0 + t] = tile * TILE_M + quarter * 32 + (__ffs(who) - 1);
                            }
                        }
                    }
                } else if (o < p.out) {
                    float *yo = y + (size_t)c0 * p.ldy + o;
                    if (stacked && c0 + 16 <= p.n) { // the usual case, kept short: sixteen full rows, hi + lo columns
#pragma unroll
                        for (int t = 0; t < 16; ++t, yo += p.ldy) ptx::red_add_f32(yo, (__uint_as_float(r[t]) + __uint_as_float(q[t])) * scale + bias);
                    } else {
#pragma unroll
                        for (int t = 0; t < 16; ++t) {
                            const int i = c0 + t;
                            if (i < p.n) {
                                float v = (__uint_as_float(r[t]) + (stacked ? __uint_as_float(q[t]) : 0.f)) * scale + bias;
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

// Pipeline depth.  With `shared_sm` (more CTAs than SMs) a CTA takes at most half an SM's shared memory, so that two
// are resident and one's tensor-core and epilogue phases overlap the other's loads.
int gemm_ws_stages(int n_pad, int use_lo, bool shared_sm) {
    const int stage_bytes = A_BYTES + n_pad * TILE_K * 2 * (use_lo ? 2 : 1);
    int s = (shared_sm ? SMEM_BUDGET_SHARED : SMEM_BUDGET) / stage_bytes;
    return s > MAX_STAGES ? MAX_STAGES : (s < 2 ? 2 : s);
}

cudaError_t gemm_ws_prepare() {
    cudaError_t e = cudaFuncSetAttribute(gemm_ws_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_ws_kernel<false>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_ws_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_ws_kernel<true>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    return e;
}

cudaError_t launch_gemm_ws(const void *map_w, const void *map_hi, const void *map_lo, float *y, const StepInfo *info, int ldy,
                           const float *bias, int n, int K, int out, int use_lo, int grid, int sm_count, int32_t *status, bool pdl,
                           cudaStream_t s, unsigned long long *trace, const GemmHeadStats *head, const float *w_scale, const uint8_t *w_codes) {
    GemmParams p;
    p.trace = trace;
    p.y = y; p.info = info; p.bias = bias; p.n = n; p.n_pad = (n + 15) & ~15;
    p.out = out; p.ldy = ldy; p.k_tiles = K / TILE_K; p.n_tiles = (out + TILE_M - 1) / TILE_M;
    p.use_lo = use_lo; p.status = status; p.w_scale = w_scale; p.w_codes = w_codes;
    const bool w8 = w_codes != nullptr; // the weights are 8-bit codes stored tile by tile; map_w is not used
    p.store = 0; p.stat_val = nullptr; p.stat_arg = nullptr; p.stat_bad = nullptr;
    const int stage_bytes = A_BYTES + p.n_pad * TILE_K * 2 * (use_lo ? 2 : 1);
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
    p.stages = gemm_ws_stages(p.n_pad, use_lo, grid > sm_count);
    if (p.stages > per_cta) p.stages = per_cta < 1 ? 1 : per_cta;
    p.landing = 0;
    if (w8) {
        // a short ring of compute stages (three cover the activation copy and the conversion ahead of the tensor cores), the
        // rest of the budget as landing slots: they are what covers the HBM latency
        int budget = (grid > sm_count ? SMEM_BUDGET_SHARED : SMEM_BUDGET);
        const int half_sm = 113 * 1024 - (int)sizeof(Barriers) - 1024; // what lets two CTAs share an SM
        if (grid > sm_count && budget > half_sm) budget = half_sm;
        if (per_cta > p.stages) { // more units than stages: the landing ring (otherwise tiles land inside their stages)
            if (p.stages > W8_PAIRS) p.stages = W8_PAIRS; // (one pair of converter warps per stage)
            while (p.stages > 1 && p.stages * stage_bytes + p.stages * A8_BYTES > budget) --p.stages;
            p.landing = (budget - p.stages * stage_bytes) / A8_BYTES;
            if (p.landing > MAX_LANDING) p.landing = MAX_LANDING;
            if (p.landing > per_cta) p.landing = per_cta;
            if (p.landing < p.stages) p.landing = p.stages;
        }
    }
    size_t smem = (size_t)p.stages * stage_bytes + (size_t)p.landing * A8_BYTES + sizeof(Barriers) + 1024;
    // Two CTAs per SM, not three: with a third one resident the slowest CTA of a projection ends later (measured: 1.19 ms per
    // GPT-2-large verification of 32 nodes against 1.09 ms), so a CTA asks for more than a third of an SM's shared memory.
    if (grid > sm_count && smem < 78 * 1024) smem = 78 * 1024;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(w8 && p.landing ? GEMM_THREADS_W8 : GEMM_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    if (w8) map_w = map_hi;
    return cudaLaunchKernelEx(&cfg, w8 ? gemm_ws_kernel<true> : gemm_ws_kernel<false>, *(const CUtensorMap *)map_w,
                              *(const CUtensorMap *)map_hi, *(const CUtensorMap *)(map_lo ? map_lo : map_hi), p);
}
