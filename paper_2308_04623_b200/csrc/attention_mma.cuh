// Tree-masked attention work item on mma.sync tensor-core tiles (shared by the stand-alone
// attention kernel and the persistent forward kernel).
//
// One work item = (head, 16-node tile, key split), executed by NW warps.  A node's
// keys are the kv_len committed cache rows (no mask) and the tree nodes that are its ancestors
// or itself (ancestor bit mask), under one softmax (Section 3.1 of the paper).  The key range is
// cut in blocks of 16 keys; a split owns a contiguous range of blocks, its warps take blocks
// round-robin, each keeping an online softmax (running max, running sum, un-normalised output)
// for the 16 nodes, and the warps' partial results are merged through shared memory.  With one
// split the item writes the normalised output as bf16 hi/lo planes; with several splits it
// writes (max, sum, un-normalised output) and the consumer merges the splits.
//
// Layouts.  K cache of a head: [cap, 64] bf16 (key-major).  V cache of a head: TRANSPOSED,
// [64, cap] bf16 (dimension-major), so that the P.V product finds consecutive keys contiguous.
// The batch's own K/V rows are converted from the fp32 projections, kept in shared memory
// together with the last partly-filled 16-key block of the prefix, and (by one item per head)
// stored into the cache's scratch slots kv_len + i.
//
// Precision: q and the softmax weights enter the tensor cores as bf16 hi + lo pairs (two MMAs),
// K and V are the cache's bf16 values, accumulation and the softmax are fp32.
#pragma once
#include "sm100_ptx.cuh"
#include "ssd_internal.h"
#include "w8_planes.cuh"

namespace attn {
constexpr int DH = 64;
constexpr int NW_MAX = 9;        // most warps a work item runs on (9 x 2 key blocks = the 256 + 32 keys of the usual step)
constexpr int KROW = DH + 8;     // shared-memory K row stride (elements): 144 B, spreads banks
constexpr int MAX_SPLITS = 4;
constexpr int QROW = DH + 4;     // shared-memory row stride (floats) of the 16 query rows

__host__ __device__ inline size_t smem_bytes(int n, int NW = NW_MAX, bool staged = false, int splits = 1) {
    // sized for the worst prefix alignment: up to 15 prefix-tail keys plus n tree keys (none when the tree's rows are read from the cache)
    const int lk_pad = staged ? 0 : (n + 15 + 15) & ~15;
    const int vrow = lk_pad + 8;
    return (size_t)lk_pad * KROW * 2 + (size_t)DH * vrow * 2 + (size_t)NW * 16 * 66 * 4 + (size_t)16 * QROW * 4 + 16 * SSD_ANC_WORDS * 8 + 16 +
           (splits > 1 ? (size_t)splits * 16 * 66 * 4 : 0); // (key splits merged inside a cluster: one partial result per split, in the first CTA)
}

// Where an item's result goes.
struct Output {
    __nv_bfloat16 *o_hi, *o_lo; // one split: normalised output planes [n, d] (o_lo may be null)
    float *part_o;              // several splits: [split][max_nodes][d] un-normalised sums
    float *part_ml;             // several splits: [split][max_nodes][n_head][2] running max and sum
    int max_nodes, n_head;
    int cluster_merge;          // several splits that are the CTAs of ONE thread-block cluster (split = rank): each sends its partial
                                // result to the first CTA's shared memory, which merges them and writes the output as with one split
    uint8_t *planes8;           // one split, 8-bit projections: the output as four e4m3 planes [4][rows][d] instead of o_hi / o_lo
    size_t plane_stride;
};

__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo_elem, float hi_elem) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo_elem, hi_elem);
    return *reinterpret_cast<uint32_t *>(&v);
}
// hi = bf16(v), lo = bf16(v - hi) for a pair of values
__device__ __forceinline__ void split_pair(float x, float y, uint32_t &hi, uint32_t &lo) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
    hi = *reinterpret_cast<const uint32_t *>(&h);
    lo = pack_bf16(x - __low2float(h), y - __high2float(h));
}
// barrier among the 256 threads of the work item (named barrier `bar_id`)
__device__ __forceinline__ void item_sync(int bar_id, int threads) { asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(threads) : "memory"); }

// K and V fragments of one 16-key block for one lane
struct BlockFrags {
    uint4 k[2][2]; // [8-key tile m][dims 0..31 | 32..63] : 8 dims each for this lane's key row
    uint2 v[8];    // [dims tile]: 4 keys of this lane's dimension row
};

// NW warps run the item; tid: 0..32*NW-1 within it.  smem_raw: 16-byte aligned, smem_bytes(n, NW) bytes.
// PREFETCH: fetch the next block's fragments while the current one is computed (worth its 32
// registers only when a warp handles several blocks).
// PDL_WAIT: the item runs in a kernel launched as a programmatic dependent: the committed cache rows of its
// first blocks (written by earlier steps) are requested first, then it waits for the kernel that produced `qkv`.
// LO: q and the softmax weights enter the tensor cores as hi + lo pairs (two MMAs each); without it as one bf16 value, which
// rounds them as coarsely as the cache already rounds K and V.
// STAGED: a kernel before this one has already written the tree's K / V rows (bf16) to the cache's scratch slots kv_len + i and zeroed
// the rest of the last 16-key block: every block is read from the cache, nothing is staged in shared memory (large trees: with
// sixteen 16-node tiles per head, sixteen CTAs would otherwise each convert and stage the whole tree's keys).
template <int NW, bool PREFETCH, bool PDL_WAIT = false, bool LO = true, bool STAGED = false>
__device__ __forceinline__ void work_item(int tid, int bar_id, unsigned char *smem_raw, int h, int tile0, int split, int n_splits,
                                          bool store_scratch, const float *__restrict__ qkv, const StepInfo *__restrict__ info,
                                          size_t layer_offset, const TreeMeta &meta, int n, int d, int cap, const Output &out,
                                          unsigned long long *trace = nullptr) {
    const int warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int P = info->kv_len, Pf = P & ~15, n_keys = P + n;
    const int local_keys = STAGED ? 0 : n_keys - Pf; // keys held in shared memory: prefix tail + tree
    const int lk_pad = (local_keys + 15) & ~15;
    const int vrow = lk_pad + 8;                    // shared V^T row stride (elements)
    __nv_bfloat16 *kc = reinterpret_cast<__nv_bfloat16 *>(info->kbase) + layer_offset + (size_t)h * cap * DH;  // [cap, 64]
    __nv_bfloat16 *vc = reinterpret_cast<__nv_bfloat16 *>(info->vbase) + layer_offset + (size_t)h * cap * DH;  // [64, cap]
    __nv_bfloat16 *s_k = reinterpret_cast<__nv_bfloat16 *>(smem_raw);             // [lk_pad][KROW]
    __nv_bfloat16 *s_v = s_k + (size_t)lk_pad * KROW;                              // [64][vrow]
    float *s_merge = reinterpret_cast<float *>(s_v + (size_t)DH * vrow);           // [NW][16][66]: m, l, o[64]
    float *s_q = s_merge + (size_t)NW * 16 * 66;                                   // [16][QROW] query rows of the tile (fp32)
    uint64_t *s_anc = reinterpret_cast<uint64_t *>(s_q + 16 * QROW);               // [16][SSD_ANC_WORDS] ancestor masks of the tile's rows
    float *s_cl = reinterpret_cast<float *>(s_anc + 16 * SSD_ANC_WORDS);           // [n_splits][16][66] (cluster merge, used in the first CTA)

    const int n_blocks = (n_keys + 15) >> 4;
    const int b_lo = (n_blocks * split) / n_splits, b_hi = (n_blocks * (split + 1)) / n_splits;
    const bool need_local = !STAGED && (store_scratch || (b_hi << 4) > Pf);

    // ---- first blocks' K/V fragments from the cache (global): they depend on no kernel of this step
    auto load_global = [&](int b, BlockFrags &f) {
        const int kb = b << 4;
#pragma unroll
        for (int m = 0; m < 2; ++m) {
            const __nv_bfloat16 *kr = kc + (size_t)(kb + 4 * (g >> 1) + 2 * m + (g & 1)) * DH;
            f.k[m][0] = *reinterpret_cast<const uint4 *>(kr + 8 * t);
            f.k[m][1] = *reinterpret_cast<const uint4 *>(kr + 32 + 8 * t);
        }
#pragma unroll
        for (int dt = 0; dt < 8; ++dt) f.v[dt] = *reinterpret_cast<const uint2 *>(vc + (size_t)(8 * dt + g) * cap + kb + 4 * t);
    };
    auto load_local = [&](int b, BlockFrags &f) {
        const int kb = (b << 4) - Pf;
#pragma unroll
        for (int m = 0; m < 2; ++m) {
            const __nv_bfloat16 *kr = s_k + (size_t)(kb + 4 * (g >> 1) + 2 * m + (g & 1)) * KROW;
            f.k[m][0] = *reinterpret_cast<const uint4 *>(kr + 8 * t);
            f.k[m][1] = *reinterpret_cast<const uint4 *>(kr + 32 + 8 * t);
        }
#pragma unroll
        for (int dt = 0; dt < 8; ++dt) f.v[dt] = *reinterpret_cast<const uint2 *>(s_v + (size_t)(8 * dt + g) * vrow + kb + 4 * t);
    };
    auto load_late = [&](int blk, BlockFrags &f) { // a block that holds rows of this step's tree
        if (STAGED) load_global(blk, f);
        else load_local(blk, f);
    };
    BlockFrags cur, nxt;
    int b = b_lo + warp;
    if (b < b_hi && (b << 4) < Pf) load_global(b, cur);
    bool nxt_ready = false; // the second block of this warp, when it is a committed one, is requested here as well
    if (PREFETCH && b + NW < b_hi && ((b + NW) << 4) < Pf) { load_global(b + NW, nxt); nxt_ready = true; }
    // ancestor masks of the tile's rows (written by the tree-preparation kernel); rows past the tree see nothing
    for (int e = tid; e < 16 * SSD_ANC_WORDS; e += NW * 32) {
        const int row = tile0 + e / SSD_ANC_WORDS;
        s_anc[e] = row < n ? meta.anc[row * SSD_ANC_WORDS + (e % SSD_ANC_WORDS)] : 0ull;
    }
    if (PDL_WAIT) {
        ptx::pdl_grid_wait();
        if (tid == 0) ptx::trace_mark(trace, 1);
    }

    // ---- the tile's query rows: one coalesced 16-byte load per thread into shared memory (every warp needs all of them)
    for (int e = tid; e < 16 * (DH / 4); e += NW * 32) {
        const int r = e >> 4, c = (e & 15) * 4, row = tile0 + r;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (row < n) { // (L2 loads: inside the persistent kernel these values come from other SMs)
            v = __ldcg(reinterpret_cast<const float4 *>(qkv + (size_t)row * 3 * d + h * DH + c));
        }
        *reinterpret_cast<float4 *>(s_q + r * QROW + c) = v;
    }
    // ---- stage the local keys: tail of the prefix (from the cache) and the tree's own rows
    if (need_local) {
        // One (key row, 8-dim group) per step: 16-byte loads/stores for K.  V is kept transposed; the lanes holding
        // two neighbouring keys of the same dims swap halves, so that each writes 4 dims x 2 keys as 32-bit words
        // (half as many stores as one 16-bit store per value: the store queue is what this phase waits for).
        for (int e = tid; e < lk_pad * (DH / 8); e += NW * 32) { // (the same trip count for every lane of a warp)
            const int r = e >> 3, c = (e & 7) * 8, key = Pf + r;
            const bool tree_row = key >= P && key < n_keys;
            uint4 kq = make_uint4(0, 0, 0, 0);
            uint32_t vw[4] = {0u, 0u, 0u, 0u}; // this key's V, dims c + 2i (low half) and c + 2i + 1 (high half)
            if (key < P) {
                kq = *reinterpret_cast<const uint4 *>(kc + (size_t)key * DH + c);
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    vw[i] = (uint32_t)__bfloat16_as_ushort(vc[(size_t)(c + 2 * i) * cap + key]) |
                            ((uint32_t)__bfloat16_as_ushort(vc[(size_t)(c + 2 * i + 1) * cap + key]) << 16);
            } else if (tree_row) {
                const int j = key - P;
                const float *kf = qkv + (size_t)j * 3 * d + d + h * DH + c, *vf = qkv + (size_t)j * 3 * d + 2 * d + h * DH + c;
                float4 k0 = __ldcg(reinterpret_cast<const float4 *>(kf)), k1 = __ldcg(reinterpret_cast<const float4 *>(kf + 4));
                float4 v0 = __ldcg(reinterpret_cast<const float4 *>(vf)), v1 = __ldcg(reinterpret_cast<const float4 *>(vf + 4));
                float kk[8] = {k0.x, k0.y, k0.z, k0.w, k1.x, k1.y, k1.z, k1.w}, vf8[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
                kq.x = pack_bf16(kk[0], kk[1]); kq.y = pack_bf16(kk[2], kk[3]); kq.z = pack_bf16(kk[4], kk[5]); kq.w = pack_bf16(kk[6], kk[7]);
#pragma unroll
                for (int i = 0; i < 4; ++i) vw[i] = pack_bf16(vf8[2 * i], vf8[2 * i + 1]);
                if (store_scratch) *reinterpret_cast<uint4 *>(kc + (size_t)key * DH + c) = kq; // scratch slot of the cache, apart from the committed rows
            }
            *reinterpret_cast<uint4 *>(s_k + (size_t)r * KROW + c) = kq;
            // swap with the lane of key r ^ 1 (8 lanes away): the even key's lane keeps dims c..c+3, the odd key's c+4..c+7
            const bool odd = r & 1;
            const uint32_t got0 = __shfl_xor_sync(0xffffffffu, odd ? vw[0] : vw[2], 8), got1 = __shfl_xor_sync(0xffffffffu, odd ? vw[1] : vw[3], 8);
            const bool both_tree = __shfl_xor_sync(0xffffffffu, tree_row ? 1 : 0, 8) && tree_row;
            const uint32_t mine0 = odd ? vw[2] : vw[0], mine1 = odd ? vw[3] : vw[1];
            const uint32_t ev0 = odd ? got0 : mine0, od0 = odd ? mine0 : got0, ev1 = odd ? got1 : mine1, od1 = odd ? mine1 : got1;
            const uint32_t pair[4] = {__byte_perm(ev0, od0, 0x5410), __byte_perm(ev0, od0, 0x7632), __byte_perm(ev1, od1, 0x5410),
                                      __byte_perm(ev1, od1, 0x7632)}; // dims cc + i: even key low half, odd key high half
            const int cc = c + (odd ? 4 : 0), r_even = r & ~1;
#pragma unroll
            for (int i = 0; i < 4; ++i) *reinterpret_cast<uint32_t *>(s_v + (size_t)(cc + i) * vrow + r_even) = pair[i];
            if (store_scratch && tree_row) {
                if (both_tree) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) *reinterpret_cast<uint32_t *>(vc + (size_t)(cc + i) * cap + (Pf + r_even)) = pair[i];
                } else { // the neighbouring key is not a row of this tree: this lane writes all eight dims of its own
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        vc[(size_t)(c + 2 * i) * cap + key] = __ushort_as_bfloat16((unsigned short)(vw[i] & 0xffffu));
                        vc[(size_t)(c + 2 * i + 1) * cap + key] = __ushort_as_bfloat16((unsigned short)(vw[i] >> 16));
                    }
                }
            }
        }
    }
    item_sync(bar_id, NW * 32);
    if (tid == 0) ptx::trace_mark(trace, 3); // local keys staged

    // A fragments of q (hi and lo parts); k-step s covers real dims base(s) + 8t + {0..3}: the order the 16-byte K loads imply
    uint32_t qh[4][4], ql[4][4];
#pragma unroll
    for (int s = 0; s < 4; ++s) {
        const int base = 32 * (s >> 1) + 4 * (s & 1) + 8 * t;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const float4 v = *reinterpret_cast<const float4 *>(s_q + (g + 8 * half) * QROW + base);
            split_pair(v.x, v.y, qh[s][half], ql[s][half]);
            split_pair(v.z, v.w, qh[s][2 + half], ql[s][2 + half]);
        }
    }

    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    float oacc[8][4];
#pragma unroll
    for (int dt = 0; dt < 8; ++dt)
#pragma unroll
        for (int q = 0; q < 4; ++q) oacc[dt][q] = 0.f;

    if (b < b_hi && (b << 4) >= Pf) load_late(b, cur);
    while (b < b_hi) {
        const int kb = b << 4, nb = b + NW;
        if (PREFETCH && nb < b_hi && !nxt_ready) { // fetch the next block while this one is computed
            if ((nb << 4) < Pf) load_global(nb, nxt);
            else load_late(nb, nxt);
        }
        nxt_ready = false;
        const bool tree_block = kb + 16 > P; // only such blocks need the ancestor mask
        // scores of the two 8-key tiles; tile m, column c <-> real key kb + 4*(c/2) + 2m + (c%2)
        float sc[2][4];
#pragma unroll
        for (int m = 0; m < 2; ++m) {
            float c[4] = {0.f, 0.f, 0.f, 0.f}, cl[4] = {0.f, 0.f, 0.f, 0.f}; // q's high and low parts: two chains of four, not one of eight
            const uint4 k0 = cur.k[m][0], k1 = cur.k[m][1];
            if (LO) {
                mma_bf16(c, qh[0], k0.x, k0.y); mma_bf16(cl, ql[0], k0.x, k0.y);
                mma_bf16(c, qh[1], k0.z, k0.w); mma_bf16(cl, ql[1], k0.z, k0.w);
                mma_bf16(c, qh[2], k1.x, k1.y); mma_bf16(cl, ql[2], k1.x, k1.y);
                mma_bf16(c, qh[3], k1.z, k1.w); mma_bf16(cl, ql[3], k1.z, k1.w);
            } else { // (two chains of two: cl takes the second half of the dimensions)
                mma_bf16(c, qh[0], k0.x, k0.y); mma_bf16(cl, qh[2], k1.x, k1.y);
                mma_bf16(c, qh[1], k0.z, k0.w); mma_bf16(cl, qh[3], k1.z, k1.w);
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) c[q] += cl[q];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                bool ok = true;
                if (tree_block) {
                    const int rk = kb + 4 * t + 2 * m + (q & 1); // real key of this accumulator column
                    ok = rk < P;
                    if (!ok && rk < n_keys) {
                        const int j = rk - P;
                        ok = (s_anc[(g + 8 * (q >> 1)) * SSD_ANC_WORDS + (j >> 6)] >> (j & 63)) & 1ull;
                    }
                }
                sc[m][q] = ok ? c[q] * 0.125f : -INFINITY; // 1/sqrt(64)
            }
        }
        // online softmax, rows g (half 0) and g+8 (half 1)
        uint32_t ph[4], pl[4]; // A fragment of P: a0 (row g, tile 0), a1 (row g+8, tile 0), a2 (row g, tile 1), a3 (row g+8, tile 1)
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            float bm = fmaxf(fmaxf(sc[0][2 * half], sc[0][2 * half + 1]), fmaxf(sc[1][2 * half], sc[1][2 * half + 1]));
            bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 1));
            bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 2));
            const float m_new = fmaxf(m_run[half], bm);
            float alpha = 1.f, p00 = 0.f, p01 = 0.f, p10 = 0.f, p11 = 0.f;
            if (m_new != -INFINITY) {
                alpha = (m_run[half] == -INFINITY) ? 0.f : __expf(m_run[half] - m_new);
                p00 = __expf(sc[0][2 * half] - m_new); p01 = __expf(sc[0][2 * half + 1] - m_new);
                p10 = __expf(sc[1][2 * half] - m_new); p11 = __expf(sc[1][2 * half + 1] - m_new);
            }
            m_run[half] = m_new;
            l_run[half] = l_run[half] * alpha + (p00 + p01 + p10 + p11);
#pragma unroll
            for (int dt = 0; dt < 8; ++dt) { oacc[dt][2 * half] *= alpha; oacc[dt][2 * half + 1] *= alpha; }
            split_pair(p00, p01, ph[half], pl[half]);
            split_pair(p10, p11, ph[2 + half], pl[2 + half]);
        }
        // O += P . V ; B fragment of dims tile dt: V^T[8dt + g][kb + 4t .. +3]
#pragma unroll
        for (int dt = 0; dt < 8; ++dt) {
            mma_bf16(oacc[dt], ph, cur.v[dt].x, cur.v[dt].y);
            if (LO) mma_bf16(oacc[dt], pl, cur.v[dt].x, cur.v[dt].y);
        }
        b = nb;
        if (PREFETCH) {
            cur = nxt;
        } else if (b < b_hi) {
            if ((b << 4) < Pf) load_global(b, cur);
            else load_late(b, cur);
        }
    }
    // row sums over the four lanes of a quad
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        l_run[half] += __shfl_xor_sync(0xffffffffu, l_run[half], 1);
        l_run[half] += __shfl_xor_sync(0xffffffffu, l_run[half], 2);
    }
    // ---- merge the warps' partial softmaxes
    float *mine = s_merge + (size_t)warp * 16 * 66;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        float *row = mine + (size_t)(g + 8 * half) * 66;
        if (t == 0) { row[0] = m_run[half]; row[1] = l_run[half]; }
#pragma unroll
        for (int dt = 0; dt < 8; ++dt) {
            row[2 + 8 * dt + 2 * t] = oacc[dt][2 * half];
            row[2 + 8 * dt + 2 * t + 1] = oacc[dt][2 * half + 1];
        }
    }
    item_sync(bar_id, NW * 32);
    // 256 (row, 4-dim group) slots: slot -> (row r = slot / 16, dims 4*(slot % 16) .. +3)
    for (int slot = tid; slot < 256; slot += NW * 32) {
        const int r = slot >> 4, c0 = (slot & 15) * 4, row = tile0 + r;
        if (row < n) {
            float M = -INFINITY;
#pragma unroll
            for (int w = 0; w < NW; ++w) M = fmaxf(M, s_merge[((size_t)w * 16 + r) * 66]);
            float L = 0.f, acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int w = 0; w < NW; ++w) { // (unrolled: the warps' partial results are fetched together, not one after the other)
                const float *src = s_merge + ((size_t)w * 16 + r) * 66;
                const float wgt = (src[0] == -INFINITY) ? 0.f : __expf(src[0] - M);
                L += src[1] * wgt;
#pragma unroll
                for (int q = 0; q < 4; ++q) acc[q] += src[2 + c0 + q] * wgt;
            }
            const size_t at = (size_t)row * d + h * DH + c0;
            if (n_splits > 1 && out.cluster_merge) { // this split's (max, sum, un-normalised output) of the row -> the first CTA of the cluster
                const uint32_t dst = ptx::mapa_shared(ptx::smem_u32(s_cl + ((size_t)split * 16 + r) * 66), 0);
                if (c0 == 0) { ptx::st_cluster_f32(dst, M); ptx::st_cluster_f32(dst + 4, L); }
#pragma unroll
                for (int q = 0; q < 4; ++q) ptx::st_cluster_f32(dst + (2 + c0 + q) * 4, acc[q]);
            } else if (n_splits == 1) {
                const float inv = 1.0f / L; // a node always sees itself, so L > 0
                if (out.planes8) { w8::store4(out.planes8, out.plane_stride, at, acc[0] * inv, acc[1] * inv, acc[2] * inv, acc[3] * inv); continue; }
                uint32_t h0, l0, h1, l1;
                split_pair(acc[0] * inv, acc[1] * inv, h0, l0);
                split_pair(acc[2] * inv, acc[3] * inv, h1, l1);
                *reinterpret_cast<uint2 *>(out.o_hi + at) = make_uint2(h0, h1);
                if (out.o_lo) *reinterpret_cast<uint2 *>(out.o_lo + at) = make_uint2(l0, l1);
            } else {
                *reinterpret_cast<float4 *>(out.part_o + (size_t)split * out.max_nodes * d + at) = make_float4(acc[0], acc[1], acc[2], acc[3]);
                if (c0 == 0)
                    *reinterpret_cast<float2 *>(out.part_ml + (((size_t)split * out.max_nodes + row) * out.n_head + h) * 2) = make_float2(M, L);
            }
        }
    }
    if (n_splits > 1 && out.cluster_merge) {
        ptx::cluster_arrive_release();
        ptx::cluster_wait_acquire();
        if (split == 0) { // the same merge once more, over the splits' results
            for (int slot = tid; slot < 256; slot += NW * 32) {
                const int r = slot >> 4, c0 = (slot & 15) * 4, row = tile0 + r;
                if (row >= n) continue;
                float M = -INFINITY;
                for (int w = 0; w < n_splits; ++w) M = fmaxf(M, s_cl[((size_t)w * 16 + r) * 66]);
                float L = 0.f, acc[4] = {0.f, 0.f, 0.f, 0.f};
                for (int w = 0; w < n_splits; ++w) {
                    const float *src = s_cl + ((size_t)w * 16 + r) * 66;
                    const float wgt = (src[0] == -INFINITY) ? 0.f : __expf(src[0] - M);
                    L += src[1] * wgt;
#pragma unroll
                    for (int q = 0; q < 4; ++q) acc[q] += src[2 + c0 + q] * wgt;
                }
                const size_t at = (size_t)row * d + h * DH + c0;
                const float inv = 1.0f / L; // a node always sees itself, so L > 0
                if (out.planes8) { w8::store4(out.planes8, out.plane_stride, at, acc[0] * inv, acc[1] * inv, acc[2] * inv, acc[3] * inv); continue; }
                uint32_t h0, l0, h1, l1;
                split_pair(acc[0] * inv, acc[1] * inv, h0, l0);
                split_pair(acc[2] * inv, acc[3] * inv, h1, l1);
                *reinterpret_cast<uint2 *>(out.o_hi + at) = make_uint2(h0, h1);
                if (out.o_lo) *reinterpret_cast<uint2 *>(out.o_lo + at) = make_uint2(l0, l1);
            }
        }
    }
}
} // namespace attn
