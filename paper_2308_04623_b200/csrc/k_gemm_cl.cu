// Weight-streaming small-M projection whose split-K partial sums are reduced INSIDE a thread-block
// cluster, through distributed shared memory, so that the epilogue sees finished sums (bf16 path,
// trees of up to 64 nodes).
//
//   acc[i, o] = sum_k X[i, k] * W[o, k],   i < n nodes, o < out
//
// As in the plain projection kernel the 128-wide MMA dimension runs over output features (weight tile
// [128 x 64] = operand A by TMA, activations [n_pad x 64] hi | lo = operand B by TMA, accumulator in
// tensor memory), and the step is bound by streaming W once from HBM (Section 2.2 of the paper).  What
// differs is who adds the partial sums.  One cluster of S CTAs owns one 128-feature output tile; CTA r
// multiplies its share of the k tiles, then the cluster does a reduce-scatter over node columns: every
// CTA lays its partial sums out by owner in its own shared memory (over the pipeline stages, which are
// free by then) and sends the block of columns owned by CTA t into t's shared memory with one bulk
// asynchronous copy that completes on an mbarrier of t; CTA t waits for its S - 1 blocks and adds the S
// partial sums of its columns in rank order (so the result is reproducible bit for bit).  With
// complete sums in hand the epilogue can do what used to need kernels of their own:
//   MODE_FOLD_STORE   y = rstd * (acc - mean * c1) + c2                    (LayerNorm folded in; QKV)
//   MODE_FOLD_GELU    planes = hi/lo bf16 of gelu(rstd * (acc - mean * c1) + c2)          (FC + GELU)
//   MODE_RESIDUAL     x += acc + bias; planes = hi/lo bf16 of x * gain; per-row sum and sum of squares
//                     of x over this tile's features                         (out-proj, MLP proj)
// A LayerNorm in front of a projection is applied algebraically: the projection runs on x * gain and
// c1 = W gain, c2 = W beta + bias are precomputed, so LN(x) W^T + b = rstd * (acc - mean * c1) + c2; the
// row statistics arrive as per-tile partial sums written by the previous MODE_RESIDUAL epilogue (or by
// the embedding kernel) and are added in tile order.  Nothing is accumulated in global memory, so no
// buffer has to be zeroed between layers.
//
// Every mbarrier wait is bounded; a CTA whose wait expires records an error word and still takes part
// in the cluster barriers, so its peers are never left waiting.
#include <cuda.h>
#include <cstring>

#include "sm100_ptx.cuh"
#include "ssd_internal.h"

namespace {
constexpr int TILE_M = 128;
constexpr int TILE_K = 64;
constexpr int UMMA_K = 16;
constexpr int A_BYTES = TILE_M * TILE_K * 2;
constexpr int CL_MAX_STAGES = 10;
constexpr int CL_THREADS = 320;     // warp 0 TMA producer, warp 1 MMA issuer, warps 2..9 epilogue
constexpr int EPI_THREADS = 256;
constexpr int CL_MAX_NODES = 64;   // n_pad this kernel serves
constexpr int CL_MAX_PARTS = 16;   // output tiles that write partial row statistics: d_model <= 2048

struct ClParams {
    int n, n_pad, out, k_tiles, n_tiles, S, stages, use_lo;
    int chunk, ldc;         // node columns a rank finishes (n_pad / S, a multiple of 4) and the row stride (floats) of a [128][chunk] block
    int pipe_bytes;         // pipeline stages, at least n_pad * 512 bytes: the staging area of the reduction lies over them
    // LayerNorm fold (MODE_FOLD_*)
    const float *stats_in;  // [parts][SSD_MAX_NODES][2] partial row sums / sums of squares
    int stats_parts;
    const float *c1, *c2;
    float inv_d, eps;
    // MODE_FOLD_STORE: y[n, ldy] fp32.  MODE_RESIDUAL: y = the residual stream x[n, ldy], read and written
    float *y;
    int ldy;
    const float *bias;      // MODE_RESIDUAL
    const float *gain;      // MODE_RESIDUAL: gain of the LayerNorm that follows (null: no planes wanted)
    __nv_bfloat16 *plane_hi, *plane_lo;
    int plane_ld;
    float *stats_out;       // MODE_RESIDUAL: [n_tiles][SSD_MAX_NODES][2]
    int32_t *status;
    unsigned long long *trace;
};

struct __align__(16) ClShared {
    uint64_t full[CL_MAX_STAGES];
    uint64_t empty[CL_MAX_STAGES];
    uint64_t acc_full;
    uint64_t red_full;              // completes when the other ranks' blocks of this CTA's columns have landed
    uint32_t tmem_base;
    uint32_t abort;
    float mean[CL_MAX_NODES], rstd[CL_MAX_NODES];
    float wsum[4][CL_MAX_NODES][2]; // the four epilogue warps' shares of a column's statistics
    float2 part[CL_MAX_NODES][CL_MAX_PARTS]; // partial statistics of this CTA's columns as loaded
};

__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 2, 256;" ::: "memory"); } // the eight epilogue warps
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// The cluster barrier is used for LIFETIME only (every CTA is running before anyone writes into it; no CTA leaves while a
// peer may still copy out of or into its shared memory); data visibility goes through mbarriers.  So the arrival is
// relaxed: a releasing arrival is a fence that waits for every outstanding access of the thread.
__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t map_to_rank(uint32_t smem_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
// Bulk copy from this CTA's shared memory into another CTA's of the cluster; completion is counted in bytes on an
// mbarrier of the destination CTA (both addresses already mapped to it).
__device__ __forceinline__ void bulk_copy_to_cluster(uint32_t dst_cluster_addr, uint32_t src_cta_addr, uint32_t bytes, uint32_t bar_cluster_addr) {
    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_cluster_addr),
                 "r"(src_cta_addr), "r"(bytes), "r"(bar_cluster_addr)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t *bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(ptx::smem_u32(bar)), "r"(parity)
        : "memory");
    return done != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster_bounded(uint64_t *bar, uint32_t parity, long long max_cycles = 500000000ll) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int it = 0; it < 256; ++it) {
            if (mbar_try_wait_cluster(bar, parity)) return true;
            __nanosleep(32);
        }
        if (clock64() - t0 > max_cycles) return false;
    }
}

__device__ __forceinline__ float gelu_tanh_fast(float z) { // 0.5 z (1 + tanh u) = z / (1 + exp(-2u))
    const float u2 = 1.5957691216057308f * (z + 0.044715f * z * z * z);
    return __fdividef(z, 1.0f + __expf(-u2));
}

__device__ __forceinline__ void fail(const ClParams &p, ClShared *sh, int code) {
    atomicExch(p.status, code);
    atomicExch(&sh->abort, 1u);
}

#ifdef CL_DEBUG_STAMPS // (working aid: finer-grained timestamps of one CTA's epilogue, compiled out by default)
__device__ unsigned long long g_dbg[64];
#define DBG(slot) do { if (p.trace && blockIdx.x == DBG_CTA && et == 0 && half == 0) g_dbg[MODE * 16 + (slot)] = ptx::globaltimer_ns(); } while (0)
#else
#define DBG(slot) do { } while (0)
#endif
#ifndef DBG_CTA
#define DBG_CTA 0
#endif
template <int MODE>
__global__ void __launch_bounds__(CL_THREADS, 2)
gemm_cl_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_hi,
               const __grid_constant__ CUtensorMap map_lo, const ClParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int b_bytes = p.n_pad * TILE_K * 2;
    const int stage_bytes = A_BYTES + b_bytes * (p.use_lo ? 2 : 1);
    float *red = reinterpret_cast<float *>(smem + (size_t)p.pipe_bytes);                // [S sources][128 rows][ldc]
    const int blk = TILE_M * p.ldc;                                                      // floats of one (source, destination) block
    ClShared *sh = reinterpret_cast<ClShared *>(reinterpret_cast<uint8_t *>(red) + (size_t)p.S * blk * 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = p.S, rank = (int)cluster_ctarank(), tile = blockIdx.x / S;
    const int k0 = (p.k_tiles * rank) / S, k1 = (p.k_tiles * (rank + 1)) / S, nk = k1 - k0;
    const bool stacked = p.use_lo != 0;                    // (n_pad <= 64: hi and lo columns fit one MMA, N = 2 n_pad)
    const int acc_cols = stacked ? 2 * p.n_pad : p.n_pad;
    const uint32_t tmem_cols = acc_cols <= 32 ? 32u : acc_cols <= 64 ? 64u : 128u;

    ptx::pdl_launch_dependents();
    if (threadIdx.x == 0) {
        ptx::trace_mark(p.trace, 0);
        for (int s = 0; s < p.stages; ++s) { ptx::mbar_init(&sh->full[s], 1); ptx::mbar_init(&sh->empty[s], 1); }
        ptx::mbar_init(&sh->acc_full, 1);
        ptx::mbar_init(&sh->red_full, 1);
        sh->abort = (*reinterpret_cast<volatile int32_t *>(p.status) != 0) ? 1u : 0u;
        ptx::fence_mbar_init();
        // what the other ranks will send: S - 1 blocks of this CTA's columns (nobody sends before the cluster barrier below)
        if (S > 1) ptx::mbar_arrive_expect_tx(&sh->red_full, (uint32_t)((S - 1) * blk * 4));
        // weights of the first stages: they depend on nothing that runs before this kernel
        if (!sh->abort && nk > 0) {
            ptx::prefetch_tensormap(&map_w);
            const uint64_t pol = ptx::policy_evict_first();
            const int pre = min(nk, p.stages);
            for (int j = 0; j < pre; ++j) {
                ptx::mbar_arrive_expect_tx(&sh->full[j], (uint32_t)stage_bytes);
                ptx::tma_load_2d_hint(smem + (size_t)j * stage_bytes, &map_w, (k0 + j) * TILE_K, tile * TILE_M, &sh->full[j], pol);
            }
        }
    }
    if (warp == 1) {
        ptx::tmem_alloc(&sh->tmem_base, tmem_cols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    // every CTA of the cluster is running (its shared memory exists) before anyone writes into it
    cluster_arrive_relaxed();
    cluster_wait();
    const uint32_t tmem_base = sh->tmem_base;
    const bool skip = sh->abort != 0 || nk <= 0;

    if (warp == 0) {
        // ===================== TMA producer =====================
        if (lane == 0 && !skip) {
            ptx::prefetch_tensormap(&map_hi);
            if (p.use_lo) ptx::prefetch_tensormap(&map_lo);
            const uint64_t pol = ptx::policy_evict_first();
            const int pre = min(nk, p.stages);
            ptx::pdl_grid_wait(); // the activation planes are written by the kernel before this one
            ptx::trace_mark(p.trace, 1);
            bool ok = true;
            int s = 0, round = 0;
            for (int j = 0; j < nk && ok; ++j) {
                uint8_t *st = smem + (size_t)s * stage_bytes;
                if (j >= pre) {
                    if (!ptx::mbar_wait_bounded(&sh->empty[s], (round - 1) & 1)) { fail(p, sh, 0x700 + s); ok = false; break; }
                    ptx::mbar_arrive_expect_tx(&sh->full[s], (uint32_t)stage_bytes);
                    ptx::tma_load_2d_hint(st, &map_w, (k0 + j) * TILE_K, tile * TILE_M, &sh->full[s], pol);
                }
                ptx::tma_load_2d(st + A_BYTES, &map_hi, (k0 + j) * TILE_K, 0, &sh->full[s]);
                if (p.use_lo) ptx::tma_load_2d(st + A_BYTES + b_bytes, &map_lo, (k0 + j) * TILE_K, 0, &sh->full[s]);
                if (sh->abort) ok = false;
                if (++s == p.stages) { s = 0; ++round; }
            }
            if (!ok) // a failed wait: let the copies already in flight land before shared memory is released
                for (int q = 0; q < p.stages; ++q) ptx::mbar_wait_bounded(&sh->full[q], 0, 20000000ll);
        }
    } else if (warp == 1) {
        // ===================== MMA issuer =====================
        if (lane == 0 && !skip) {
            const uint32_t idesc = ptx::umma_idesc_bf16(TILE_M, acc_cols);
            int s = 0, round = 0;
            for (int j = 0; j < nk; ++j) {
                if (!ptx::mbar_wait_bounded(&sh->full[s], round & 1)) { fail(p, sh, 0x800 + s); break; }
                const uint32_t a_addr = ptx::smem_u32(smem + (size_t)s * stage_bytes), b_addr = a_addr + A_BYTES;
#pragma unroll
                for (int k = 0; k < TILE_K / UMMA_K; ++k)
                    ptx::umma_bf16(tmem_base, ptx::umma_desc_k_sw128(a_addr + k * UMMA_K * 2), ptx::umma_desc_k_sw128(b_addr + k * UMMA_K * 2), idesc,
                                   (j == 0 && k == 0) ? 0u : 1u);
                if (j + p.stages < nk) ptx::umma_commit(&sh->empty[s]);
                if (j + 1 == nk) ptx::umma_commit(&sh->acc_full);
                if (sh->abort) break;
                if (++s == p.stages) { s = 0; ++round; }
            }
        }
    } else {
        // ===================== epilogue (warps 2..9) =====================
        // Two warps per quarter of the tensor memory's lanes: `half` 0 and 1 share the node columns between them (the
        // work of a thread here is a chain of dependent latencies, so more threads with less each is what shortens it).
        const int quarter = warp & 3;          // tensor-memory lanes this warp may read: 32 * quarter ...
        const int half = (warp - 2) >> 2;
        const int et = quarter * 32 + lane;    // = the accumulator row (output feature within the tile) of this thread
        const int o = tile * TILE_M + et;
        const bool o_ok = o < p.out;
        const int chunk = p.chunk, my_c0 = chunk * rank;
        // per-feature vectors do not depend on earlier kernels
        float f1 = 0.f, f2 = 0.f, gain = 0.f;
        if (MODE == MODE_RESIDUAL) {
            f2 = o_ok ? p.bias[o] : 0.f;
            gain = (o_ok && p.gain) ? p.gain[o] : 0.f;
        } else {
            f1 = o_ok ? p.c1[o] : 0.f;
            f2 = o_ok ? p.c2[o] : 0.f;
        }
        ptx::pdl_grid_wait();
        DBG(6);
        float xin[4]; // residual input of the first column group this thread finishes, fetched ahead of the accumulator
        if (MODE == MODE_RESIDUAL) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int q = 4 * half + j, i = my_c0 + q;
                xin[j] = (q < chunk && i < p.n && o_ok) ? __ldcg(p.y + (size_t)i * p.ldy + o) : 0.f;
            }
        } else {
            // statistics of the LayerNorm in front of this projection, for the columns this CTA finishes: one
            // (column, part) pair per thread, so the loads fly together; the parts are then added in order
            const int pairs = chunk * p.stats_parts, e0 = half * 128 + et;
            for (int e = e0; e < pairs; e += EPI_THREADS) {
                const int q = e / p.stats_parts, part = e - q * p.stats_parts, i = my_c0 + q;
                const float2 st = i < p.n ? __ldcg(reinterpret_cast<const float2 *>(p.stats_in + ((size_t)part * SSD_MAX_NODES + i) * 2)) : make_float2(0.f, 0.f);
                sh->part[q][part] = st;
            }
            epi_sync();
            for (int q = e0; q < chunk; q += EPI_THREADS) {
                float s1 = 0.f, s2 = 0.f;
                for (int part = 0; part < p.stats_parts; ++part) { s1 += sh->part[q][part].x; s2 += sh->part[q][part].y; }
                const float mean = s1 * p.inv_d;
                sh->mean[q] = mean;
                sh->rstd[q] = rsqrtf(fmaxf(s2 * p.inv_d - mean * mean, 0.f) + p.eps);
            }
            epi_sync();
        }
        DBG(7);
        // ---- this CTA's partial sums: tensor memory -> the owners' reduction buffers
        int good = skip ? 0 : 1;
        if (lane == 0 && good) good = ptx::mbar_wait_bounded<32>(&sh->acc_full, 0) ? 1 : 0;
        good = __shfl_sync(0xffffffffu, good, 0);
        if (!good && !skip && lane == 0) fail(p, sh, 0x900);
        if (et == 0 && half == 0) ptx::trace_mark(p.trace, 3);
        DBG(0);
        ptx::tc_fence_after_sync();
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16);
        // Staging: one [128 rows][ldc] block per destination rank (over the pipeline stages, which are free: every MMA that read
        // them has completed); this thread's row of the block of the rank that owns a column group.  The block this CTA keeps
        // goes straight into its own slot of the reduction buffer.  Rounds of sixteen columns alternate between the halves.
        {
            float *row_stg = reinterpret_cast<float *>(smem) + et * p.ldc, *row_own = red + (size_t)rank * blk + et * p.ldc;
            for (int c0 = 16 * half; c0 < p.n_pad; c0 += 32) {
                uint32_t r[16], q[16];
                if (good) {
                    ptx::tmem_ld_32x16(taddr + c0, r);
                    if (stacked) ptx::tmem_ld_32x16(taddr + p.n_pad + c0, q);
                    ptx::tmem_ld_wait();
                }
                int t = c0 / chunk, j = c0 - t * chunk; // owner of the next column group and the group's offset inside its chunk
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    float4 v;
                    v.x = good ? __uint_as_float(r[4 * g]) + (stacked ? __uint_as_float(q[4 * g]) : 0.f) : 0.f;
                    v.y = good ? __uint_as_float(r[4 * g + 1]) + (stacked ? __uint_as_float(q[4 * g + 1]) : 0.f) : 0.f;
                    v.z = good ? __uint_as_float(r[4 * g + 2]) + (stacked ? __uint_as_float(q[4 * g + 2]) : 0.f) : 0.f;
                    v.w = good ? __uint_as_float(r[4 * g + 3]) + (stacked ? __uint_as_float(q[4 * g + 3]) : 0.f) : 0.f;
                    if (chunk >= 4) {
                        *reinterpret_cast<float4 *>((t == rank ? row_own : row_stg + (size_t)t * blk) + j) = v;
                        j += 4;
                        if (j == chunk) { j = 0; ++t; }
                    } else { // chunks of two columns: the group belongs to two neighbouring ranks
                        *reinterpret_cast<float2 *>(t == rank ? row_own : row_stg + (size_t)t * blk) = make_float2(v.x, v.y);
                        *reinterpret_cast<float2 *>(t + 1 == rank ? row_own : row_stg + (size_t)(t + 1) * blk) = make_float2(v.z, v.w);
                        t += 2;
                    }
                }
            }
        }
        DBG(1);
        ptx::tc_fence_before_sync();
        if (S > 1) {
            ptx::fence_proxy_async_smem(); // the bulk copies read the staging area through the asynchronous proxy
            epi_sync();
            if (half == 0 && et < S && et != rank) { // one thread per destination
                const uint32_t t = (uint32_t)et;
                const uint32_t dst = map_to_rank(ptx::smem_u32(red) + (uint32_t)(rank * blk * 4), t);
                const uint32_t bar = map_to_rank(ptx::smem_u32(&sh->red_full), t);
                bulk_copy_to_cluster(dst, ptx::smem_u32(smem) + t * (uint32_t)(blk * 4), (uint32_t)(blk * 4), bar);
            }
            DBG(2);
            int got = 1;
            if (lane == 0) got = mbar_wait_cluster_bounded(&sh->red_full, 0) ? 1 : 0;
            got = __shfl_sync(0xffffffffu, got, 0);
            if (!got && lane == 0) fail(p, sh, 0xA00);
        } else {
            epi_sync(); // (one rank: the other half's columns were written by other threads)
        }
        DBG(3);
        cluster_arrive_relaxed(); // this CTA holds every block it was due; once all CTAs say so, none is still a copy's source
        DBG(8);
        // ---- finished sums of this CTA's columns, four columns at a time (independent chains), groups alternating between the halves
        for (int q0 = 4 * half; q0 < chunk; q0 += 8) {
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
            const float *src = red + et * p.ldc + q0;
            if (chunk >= 4) {
#pragma unroll 4
                for (int s = 0; s < S; ++s) {
                    const float4 v = *reinterpret_cast<const float4 *>(src + (size_t)s * blk);
                    acc[0] += v.x; acc[1] += v.y; acc[2] += v.z; acc[3] += v.w;
                }
            } else {
#pragma unroll 4
                for (int s = 0; s < S; ++s) {
                    const float2 v = *reinterpret_cast<const float2 *>(src + (size_t)s * blk);
                    acc[0] += v.x; acc[1] += v.y;
                }
            }
            // (values first, without branches, so that the four columns' chains interleave; then the guarded stores)
            if (MODE != MODE_RESIDUAL) {
                float v[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    v[j] = sh->rstd[q0 + j] * (acc[j] - sh->mean[q0 + j] * f1) + f2;
                    if (MODE == MODE_FOLD_GELU) v[j] = gelu_tanh_fast(v[j]);
                }
                if (MODE == MODE_FOLD_STORE) {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (q0 + j < chunk && my_c0 + q0 + j < p.n && o_ok) p.y[(size_t)(my_c0 + q0 + j) * p.ldy + o] = v[j];
                } else {
                    __nv_bfloat16 h[4], l[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) { h[j] = __float2bfloat16_rn(v[j]); l[j] = __float2bfloat16_rn(v[j] - __bfloat162float(h[j])); }
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (q0 + j < chunk && my_c0 + q0 + j < p.n && o_ok) {
                            const size_t at = (size_t)(my_c0 + q0 + j) * p.plane_ld + o;
                            p.plane_hi[at] = h[j];
                            if (p.plane_lo) p.plane_lo[at] = l[j];
                        }
                }
            } else {
                float v[4], s1[4], s2[4];
                __nv_bfloat16 h[4], l[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int i = my_c0 + q0 + j;
                    const bool live = q0 + j < chunk && i < p.n && o_ok;
                    float xi = xin[j];
                    if (q0 >= 8 && live) xi = __ldcg(p.y + (size_t)i * p.ldy + o);
                    v[j] = live ? xi + acc[j] + f2 : 0.f;
                    const float a = v[j] * gain;
                    h[j] = __float2bfloat16_rn(a);
                    l[j] = __float2bfloat16_rn(a - __bfloat162float(h[j]));
                    s1[j] = v[j]; s2[j] = v[j] * v[j];
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int i = my_c0 + q0 + j;
                    if (q0 + j < chunk && i < p.n && o_ok) {
                        p.y[(size_t)i * p.ldy + o] = v[j];
                        if (p.gain) {
                            const size_t at = (size_t)i * p.plane_ld + o;
                            p.plane_hi[at] = h[j];
                            if (p.plane_lo) p.plane_lo[at] = l[j];
                        }
                    }
                }
#pragma unroll
                for (int off = 16; off > 0; off >>= 1)
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        s1[j] += __shfl_xor_sync(0xffffffffu, s1[j], off);
                        s2[j] += __shfl_xor_sync(0xffffffffu, s2[j], off);
                    }
                if (lane == 0)
#pragma unroll
                    for (int j = 0; j < 4; ++j) { sh->wsum[quarter][q0 + j][0] = s1[j]; sh->wsum[quarter][q0 + j][1] = s2[j]; }
            }
        }
        if (MODE == MODE_RESIDUAL) {
            epi_sync();
            for (int q = half * 128 + et; q < chunk; q += EPI_THREADS) {
                const int i = my_c0 + q;
                if (i < p.n) { // (a column's four shares were written by the four warps of the half that finished it)
                    const float s1 = (sh->wsum[0][q][0] + sh->wsum[1][q][0]) + (sh->wsum[2][q][0] + sh->wsum[3][q][0]);
                    const float s2 = (sh->wsum[0][q][1] + sh->wsum[1][q][1]) + (sh->wsum[2][q][1] + sh->wsum[3][q][1]);
                    *reinterpret_cast<float2 *>(p.stats_out + ((size_t)tile * SSD_MAX_NODES + i) * 2) = make_float2(s1, s2);
                }
            }
        }
    }
    if (warp >= 2) { const int et = (warp & 3) * 32 + lane, half = (warp - 2) >> 2; DBG(4); }
    if (warp < 2) { // the producer and issuer warps take part in the cluster barrier too
        __syncwarp();
        cluster_arrive_relaxed();
    }
    cluster_wait(); // no CTA leaves while a peer may still be copying out of or into its shared memory
    if (warp == 1) { // the accumulator was read before the barrier
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, tmem_cols);
    }
    if (warp >= 2) { const int et = (warp & 3) * 32 + lane, half = (warp - 2) >> 2; DBG(5); }
    if (threadIdx.x == 64) ptx::trace_mark(p.trace, 2);
}

template <int MODE>
cudaError_t prepare_mode() {
    cudaError_t e = cudaFuncSetAttribute(gemm_cl_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_cl_kernel<MODE>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_cl_kernel<MODE>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    return e;
}
} // namespace

#ifdef CL_DEBUG_STAMPS // (working aid: finer-grained timestamps of one CTA's epilogue, compiled out by default)
extern "C" int ssd_debug_stamps(unsigned long long *out) { return (int)cudaMemcpyFromSymbol(out, g_dbg, sizeof(g_dbg)); }
#endif

cudaError_t gemm_cl_prepare() {
    cudaError_t e = prepare_mode<MODE_FOLD_STORE>();
    if (e == cudaSuccess) e = prepare_mode<MODE_FOLD_GELU>();
    if (e == cudaSuccess) e = prepare_mode<MODE_RESIDUAL>();
    return e;
}

bool gemm_cl_supports(int n, int d_model) { return gemm_cl_n_pad(n) <= CL_MAX_NODES && (d_model + TILE_M - 1) / TILE_M <= CL_MAX_PARTS; }

// Shared memory one CTA needs with `stages` pipeline stages.
// Row stride of a [128][chunk] block: chunk floats, plus four when that keeps 16-byte row accesses of a warp off the
// same banks (the stride in floats should be 4 mod 8).
static int cl_ldc(int chunk) { return chunk < 4 ? chunk + 4 : ((chunk / 4) % 2 ? chunk : chunk + 4); }
static int cl_pipe_bytes(int n_pad, int use_lo, int S, int stages) {
    const int stage_bytes = A_BYTES + n_pad * TILE_K * 2 * (use_lo ? 2 : 1), staging = S * TILE_M * cl_ldc(n_pad / S) * 4;
    return stages * stage_bytes > staging ? stages * stage_bytes : staging;
}
static size_t cl_smem(int n_pad, int use_lo, int S, int stages) {
    return (size_t)cl_pipe_bytes(n_pad, use_lo, S, stages) + (size_t)S * TILE_M * cl_ldc(n_pad / S) * 4 + sizeof(ClShared) + 1024;
}

// Rows of the activation operand this path uses for a tree of n nodes: whole 16-row boxes, at least 32 (so that the node
// columns split into chunks of four for up to eight ranks).
int gemm_cl_n_pad(int n) { const int r = (n + 15) & ~15; return r < 32 ? 32 : r; }

// Cluster size for a projection with `n_tiles` output tiles and `k_tiles` k tiles: as many CTAs per tile as `slots`
// resident CTAs allow, at most `max_cluster`, never more than there are k tiles; every rank finishes the same number of
// node columns, a multiple of four.
int gemm_cl_cluster_size(int n, int K, int out, int slots, int max_cluster) {
    const int n_pad = gemm_cl_n_pad(n), k_tiles = K / TILE_K, n_tiles = (out + TILE_M - 1) / TILE_M;
    int S = slots / n_tiles;
    if (S > max_cluster) S = max_cluster;
    if (S > k_tiles) S = k_tiles;
    if (S < 1) S = 1;
    while (S > 1 && (n_pad % (4 * S)) != 0 && n_pad != 2 * S) --S; // chunks of whole groups of four columns, or of exactly two
    return S;
}

cudaError_t launch_gemm_cl(const void *map_w, const void *map_hi, const void *map_lo, int n, int K, int out, int use_lo, int cluster,
                           bool two_per_sm, const GemmClEpilogue &ep, int32_t *status, bool pdl, cudaStream_t s, unsigned long long *trace) {
    ClParams p;
    memset(&p, 0, sizeof(p));
    p.n = n; p.n_pad = gemm_cl_n_pad(n); p.out = out; p.k_tiles = K / TILE_K; p.n_tiles = (out + TILE_M - 1) / TILE_M;
    if (ep.mode != MODE_RESIDUAL && ep.stats_parts > CL_MAX_PARTS) return cudaErrorInvalidValue;
    if (p.n_pad > CL_MAX_NODES || cluster < 1 || cluster > 16 || cluster > p.k_tiles || (p.n_pad % (4 * cluster) && p.n_pad != 2 * cluster)) return cudaErrorInvalidValue;
    p.S = cluster; p.use_lo = use_lo; p.chunk = p.n_pad / cluster; p.ldc = cl_ldc(p.chunk);
    p.stats_in = ep.stats_in; p.stats_parts = ep.stats_parts; p.c1 = ep.c1; p.c2 = ep.c2; p.inv_d = ep.inv_d; p.eps = ep.eps;
    p.y = ep.y; p.ldy = ep.ldy; p.bias = ep.bias; p.gain = ep.gain; p.plane_hi = ep.plane_hi; p.plane_lo = ep.plane_lo; p.plane_ld = ep.plane_ld;
    p.stats_out = ep.stats_out; p.status = status; p.trace = trace;
    // pipeline depth: every k tile of a CTA resident if that fits, else as deep as the budget allows
    const int per_cta = (p.k_tiles + cluster - 1) / cluster;
    const size_t budget = two_per_sm ? 112 * 1024 : 226 * 1024;
    int stages = per_cta < CL_MAX_STAGES ? per_cta : CL_MAX_STAGES;
    while (stages > 1 && cl_smem(p.n_pad, use_lo, cluster, stages) > budget) --stages;
    if (cl_smem(p.n_pad, use_lo, cluster, stages) > 226 * 1024) return cudaErrorInvalidValue;
    p.stages = stages;
    p.pipe_bytes = cl_pipe_bytes(p.n_pad, use_lo, cluster, stages);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.n_tiles * cluster);
    cfg.blockDim = dim3(CL_THREADS);
    cfg.dynamicSmemBytes = cl_smem(p.n_pad, use_lo, cluster, stages);
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 2 : 1;
    const CUtensorMap *mw = (const CUtensorMap *)map_w, *mh = (const CUtensorMap *)map_hi, *ml = (const CUtensorMap *)(map_lo ? map_lo : map_hi);
    switch (ep.mode) {
    case MODE_FOLD_STORE: return cudaLaunchKernelEx(&cfg, gemm_cl_kernel<MODE_FOLD_STORE>, *mw, *mh, *ml, p);
    case MODE_FOLD_GELU: return cudaLaunchKernelEx(&cfg, gemm_cl_kernel<MODE_FOLD_GELU>, *mw, *mh, *ml, p);
    case MODE_RESIDUAL: return cudaLaunchKernelEx(&cfg, gemm_cl_kernel<MODE_RESIDUAL>, *mw, *mh, *ml, p);
    default: return cudaErrorInvalidValue;
    }
}
