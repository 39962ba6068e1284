// Acceptance walk down the token tree (Section 2.3 of the paper; top-k sampling per Section 4).
//
// Greedy: the verifier "agrees" with a child when the child's token is the arg-max of the
// parent's logits row.  Sampling: sibling-wise rejection sampling with a residual update, which
// keeps the verifier's next-token distribution exactly.  Every comparison that decides an
// integer (accept/refuse, which token) is taken in fp64; the uniforms come from Philox4x32-10
// keyed by (seed) and counted by (step, decision index), so a decision's uniform depends only
// on the node it concerns, never on the order of evaluation.
#include <cstring>
#include <mutex>

#include "sm100_ptx.cuh"
#include "ssd_internal.h"

namespace {
constexpr int ACC_THREADS = 1024;

// ---- Philox4x32-10 (Salmon et al., SC'11) ------------------------------------------------
__device__ __forceinline__ double uniform24(uint64_t seed, uint64_t step, uint32_t index) {
    uint32_t c0 = (uint32_t)step, c1 = (uint32_t)(step >> 32), c2 = index, c3 = 0u;
    uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ k0; c1 = lo1; c2 = hi0 ^ c3 ^ k1; c3 = lo0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    return (double)(c0 >> 8) * (1.0 / 16777216.0);
}

// ---- greedy -----------------------------------------------------------------------------
// gridDim.y CTAs per node row, each over a contiguous part of the vocabulary: arg-max of the part with the lowest
// index winning ties, and a non-finite flag.  Results at [row * gridDim.y + part].
__global__ void __launch_bounds__(256) row_argmax_kernel(const float *__restrict__ logits, int V, float *__restrict__ part_val,
                                                         int32_t *__restrict__ part_arg, int32_t *__restrict__ part_bad) {
    __shared__ float s_val[8];
    __shared__ int s_idx[8];
    __shared__ int s_bad[8];
    const float *z = logits + (size_t)blockIdx.x * V;
    const int chunk = (V + gridDim.y - 1) / gridDim.y, v_lo = min(V, (int)blockIdx.y * chunk), v_hi = min(V, v_lo + chunk);
    float best = -INFINITY;
    int bi = 0x7fffffff, bad = 0;
    for (int v = v_lo + threadIdx.x; v < v_hi; v += 256) {
        const float x = z[v];
        bad |= !isfinite(x);
        if (x > best || (x == best && v < bi)) { best = x; bi = v; }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, best, off);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
        bad |= __shfl_xor_sync(0xffffffffu, bad, off);
        if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
    }
    if ((threadIdx.x & 31) == 0) { s_val[threadIdx.x >> 5] = best; s_idx[threadIdx.x >> 5] = bi; s_bad[threadIdx.x >> 5] = bad; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w) {
            if (s_val[w] > best || (s_val[w] == best && s_idx[w] < bi)) { best = s_val[w]; bi = s_idx[w]; }
            bad |= s_bad[w];
        }
        const int at = blockIdx.x * gridDim.y + blockIdx.y;
        part_val[at] = best;
        part_arg[at] = bi;
        part_bad[at] = bad;
    }
}

// The walk, by one warp; a row's arg-max is the best of its `parts` parts (the parts are in index order, so among equal
// maxima the lowest part holds the lowest index): the lanes take the parts round-robin.  `result` may be pinned host memory.
__global__ void greedy_walk_kernel(NodeList tokens, NodeList parent, int n, int parts, const float *__restrict__ part_val,
                                   const int32_t *__restrict__ part_arg, const int32_t *__restrict__ part_bad, int32_t *__restrict__ result,
                                   const int32_t *__restrict__ dev_status) {
    const int lane = threadIdx.x;
    int cur = 0, np = 1;
    if (lane == 0) {
        result[3] = dev_status ? *dev_status : 0; // the forward's error word rides along with the walk's few result words
        result[4] = 0;
    }
    for (;;) {
        float best = -INFINITY;
        int want = 0x7fffffff, bad = 0;
        for (int q = lane; q < parts; q += 32) {
            const size_t at = (size_t)cur * parts + q;
            bad |= part_bad[at];
            const float v = part_val[at];
            const int a = part_arg[at];
            if (v > best || (v == best && a < want)) { best = v; want = a; }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, best, off);
            const int oa = __shfl_xor_sync(0xffffffffu, want, off);
            bad |= __shfl_xor_sync(0xffffffffu, bad, off);
            if (ov > best || (ov == best && oa < want)) { best = ov; want = oa; }
        }
        if (bad) { if (lane == 0) { result[1] = -1; result[2] = SSD_ERR_BAD_ARG; result[0] = 1; } return; }
        int next = -1;
        for (int c = cur + 1; c < n && next < 0; ++c) // (the same scan in every lane)
            if (parent.v[c] == cur && tokens.v[c] == want) next = c;
        if (next < 0) { if (lane == 0) { result[1] = want; result[2] = SSD_OK; result[0] = np; } return; }
        if (lane == 0) result[4 + np] = next;
        ++np;
        cur = next;
    }
}

// ---- sampling ---------------------------------------------------------------------------
struct BlockScratch {
    double d[32];
    int i[32];
    unsigned hist[2048];  // radix selection: counts per digit (up to 11 bits a round)
    unsigned cand[4096];  // ... and the keys still in the running after the first round
    unsigned sel_prefix, sel_k;
    int flag;
};

__device__ __forceinline__ double block_sum(double v, BlockScratch &s) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s.d[threadIdx.x >> 5] = v;
    __syncthreads();
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < ACC_THREADS / 32; ++w) t += s.d[w];
    return t;
}
__device__ __forceinline__ double block_max(double v, BlockScratch &s) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, off));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s.d[threadIdx.x >> 5] = v;
    __syncthreads();
    double t = -INFINITY;
#pragma unroll
    for (int w = 0; w < ACC_THREADS / 32; ++w) t = fmax(t, s.d[w]);
    return t;
}
__device__ __forceinline__ int block_min_int(int v, BlockScratch &s) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v = min(v, __shfl_xor_sync(0xffffffffu, v, off));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s.i[threadIdx.x >> 5] = v;
    __syncthreads();
    int t = 0x7fffffff;
#pragma unroll
    for (int w = 0; w < ACC_THREADS / 32; ++w) t = min(t, s.i[w]);
    return t;
}
__device__ __forceinline__ int block_max_int(int v, BlockScratch &s) { return -block_min_int(-v, s); }

__device__ __forceinline__ unsigned orderable(float f) {
    const unsigned u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float from_orderable(unsigned u) {
    return __uint_as_float((u & 0x80000000u) ? (u & 0x7fffffffu) : ~u);
}

// k-th largest value of z[0..V) by most-significant-digit radix selection (exact, integer work).
//
// One selection round: among the keys that agree with s.sel_prefix on the bits above shift + bits, count how many fall into
// each value of the next `bits` bits, find the digit that holds the s.sel_k-th largest of them, and narrow prefix and rank.
// The digit is found by all threads (chunk sums, a scan over the block, then the owner of the chunk walks it), not by one
// thread walking the histogram.  KeyAt(i) is the i-th key; `aggregate`: the lanes of a warp that hit the same bin are counted
// by one of them (logits share their leading bits, so in the first rounds most keys of a warp fall into a few bins).
constexpr int SEL_MAX_BITS = 11, SEL_CAND = 4096;
template <class KeyAt>
__device__ void select_round(KeyAt key_at, int count, int shift, int bits, bool aggregate, BlockScratch &s) {
    const int tid = threadIdx.x, nbins = 1 << bits;
    for (int b = tid; b < nbins; b += ACC_THREADS) s.hist[b] = 0u;
    __syncthreads();
    const unsigned prefix = s.sel_prefix, kk = s.sel_k;
    const unsigned himask = (shift + bits >= 32) ? 0u : (0xffffffffu << (shift + bits));
    const unsigned dmask = (unsigned)nbins - 1u;
    for (int base = 0; base < count; base += ACC_THREADS) { // the same trip count for every thread
        const int i = base + tid;
        const unsigned key = i < count ? key_at(i) : 0u;
        const bool in = i < count && (key & himask) == prefix;
        const unsigned bin = (key >> shift) & dmask;
        if (aggregate) {
            const unsigned voters = __ballot_sync(0xffffffffu, in);
            if (in) {
                const unsigned peers = __match_any_sync(voters, bin);
                if ((tid & 31) == __ffs(peers) - 1) atomicAdd(&s.hist[bin], (unsigned)__popc(peers));
            }
        } else if (in) {
            atomicAdd(&s.hist[bin], 1u);
        }
    }
    __syncthreads();
    // bins in descending order, `per` consecutive ones per thread
    const int per = (nbins + ACC_THREADS - 1) / ACC_THREADS, d0 = tid * per;
    unsigned mine = 0;
    for (int j = 0; j < per; ++j) { const int d = d0 + j; if (d < nbins) mine += s.hist[nbins - 1 - d]; }
    unsigned incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned t = __shfl_up_sync(0xffffffffu, incl, off);
        if ((tid & 31) >= off) incl += t;
    }
    if ((tid & 31) == 31) s.i[tid >> 5] = (int)incl;
    __syncthreads();
    unsigned before = 0;
    for (int w = 0; w < (tid >> 5); ++w) before += (unsigned)s.i[w];
    const unsigned excl = before + incl - mine;
    __syncthreads(); // (s.i is free again, and nobody reads the old prefix after this point)
    if (excl < kk && kk <= excl + mine) { // exactly one thread: the k-th largest lies in its chunk
        unsigned cum = excl;
        for (int j = 0; j < per; ++j) {
            const int b = nbins - 1 - (d0 + j);
            const unsigned h = s.hist[b];
            if (cum + h >= kk) { s.sel_prefix = prefix | ((unsigned)b << shift); s.sel_k = kk - cum; break; }
            cum += h;
        }
    }
    __syncthreads();
}

// Keys of the row that pass `keep` -> s.cand (in no particular order); returns how many there are (possibly more than fit).
template <class Keep>
__device__ int gather_keys(const float *__restrict__ z, int V, Keep keep, BlockScratch &s) {
    const int tid = threadIdx.x;
    if (tid == 0) s.flag = 0;
    __syncthreads();
    for (int base = 0; base < V; base += ACC_THREADS) {
        const int v = base + tid;
        const unsigned key = v < V ? orderable(z[v]) : 0u;
        const bool in = v < V && keep(key);
        const unsigned voters = __ballot_sync(0xffffffffu, in);
        if (voters) {
            int at = 0;
            if ((tid & 31) == 0) at = atomicAdd(&s.flag, __popc(voters));
            at = __shfl_sync(0xffffffffu, at, 0) + __popc(voters & ((1u << (tid & 31)) - 1u));
            if (in && at < SEL_CAND) s.cand[at] = key;
        }
    }
    __syncthreads();
    const int n = s.flag;
    __syncthreads();
    return n;
}
// The k-th largest of the first `count` keys in s.cand: four rounds of eight bits.
__device__ unsigned kth_of_cand(int count, int k, BlockScratch &s) {
    if (threadIdx.x == 0) { s.sel_prefix = 0u; s.sel_k = (unsigned)k; }
    __syncthreads();
    const unsigned *cand = s.cand;
    auto from_cand = [cand](int i) { return cand[i]; };
    for (int shift = 24; shift >= 0; shift -= 8) select_round(from_cand, count, shift, 8, shift >= 16, s);
    return s.sel_prefix;
}

// `my_max`: the largest logit among the ones this thread looked at in the pass before (thread t: z[t], z[t + ACC_THREADS], ...).
// For k up to the number of threads, the k-th largest of those maxima is a lower bound of the k-th largest of the row - k
// different entries are at least as large - so only the entries at or above it, usually a few times k, stay in the running:
// they are gathered into shared memory in one pass over the row and the selection is finished there.  The histogram rounds
// over the whole row are the general path (a larger k, or too many entries at or above the bound: ties, a narrow row): the
// first round looks at the top 11 bits (sign, exponent, two fraction bits: a quarter of a binade per bin), the keys of the bin
// the k-th largest falls into are gathered, and the remaining 21 bits are settled in shared memory; should more than SEL_CAND
// keys share those 11 bits, the later rounds read the row again instead.  (Counting a whole row into a histogram in shared
// memory is slow - 50 us for a GPT-2 vocabulary - because most logits fall into a few bins and the additions to one bin queue up.)
__device__ float kth_largest(const float *__restrict__ z, int V, int k, BlockScratch &s, float my_max) {
    const int tid = threadIdx.x;
    if (k <= ACC_THREADS) {
        __syncthreads();
        s.cand[tid] = orderable(my_max);
        __syncthreads();
        const unsigned bound = kth_of_cand(ACC_THREADS, k, s);
        const int cands = gather_keys(z, V, [bound](unsigned key) { return key >= bound; }, s);
        if (cands <= SEL_CAND) return from_orderable(kth_of_cand(cands, k, s));
    }
    if (tid == 0) { s.sel_prefix = 0u; s.sel_k = (unsigned)k; }
    __syncthreads();
    auto from_row = [z](int i) { return orderable(z[i]); };
    select_round(from_row, V, 32 - SEL_MAX_BITS, SEL_MAX_BITS, true, s);
    const unsigned top = s.sel_prefix >> (32 - SEL_MAX_BITS);
    const int cands = gather_keys(z, V, [top](unsigned key) { return (key >> (32 - SEL_MAX_BITS)) == top; }, s);
    const unsigned *cand = s.cand;
    auto from_cand = [cand](int i) { return cand[i]; };
    const int rounds[3][2] = {{13, 8}, {5, 8}, {0, 5}};
    for (int r = 0; r < 3; ++r) {
        if (cands <= SEL_CAND) select_round(from_cand, cands, rounds[r][0], rounds[r][1], false, s);
        else select_round(from_row, V, rounds[r][0], rounds[r][1], true, s);
    }
    return from_orderable(s.sel_prefix);
}

// Target law of one node, r[v] = softmax(z / T) over the kept entries (all, or the top_k largest logits, ties kept),
// in fp64 by the whole CTA; returns 1 if the row holds a non-finite value (r is then unspecified).
// With `total` given the row is left UNNORMALISED (r[v] = exp(z[v] / T - max), *total = their sum, the same value in every thread):
// the acceptance rule works on r and its total (see node_decide), which spares V fp64 divisions here and V more per refusal.
// The exponentials are what the law costs (fp64, ~60 multiply-adds each, at an SM's fp64 rate some 20 us for a GPT-2
// vocabulary), so a row can be cut into `parts` slices for as many CTAs: each looks at the whole row for the checks, the
// maximum and the cut, exponentiates its own slice only and returns that slice's sum (unnormalised rows only).
__device__ int row_law(const float *__restrict__ z, int V, double temperature, int top_k, double *__restrict__ r, BlockScratch &s,
                       double *total = nullptr, int part = 0, int parts = 1) {
    const int tid = threadIdx.x;
    // one pass for the finiteness check and the maximum (the largest entry survives any top-k cut, and dividing by a positive
    // temperature keeps the order: the maximum of the kept z / T is z_max / T)
    int bad = 0;
    float zmax = -INFINITY;
    for (int v = tid; v < V; v += ACC_THREADS) { const float zv = z[v]; bad |= !isfinite(zv); zmax = fmaxf(zmax, zv); }
    if (block_max_int(bad, s)) return 1;
    float thr = -INFINITY;
    if (top_k > 0 && top_k < V) thr = kth_largest(z, V, top_k, s, zmax);
    // (x / 1.0 is x exactly: at temperature 1 the fp64 division, a large part of this function's time, is skipped)
    const bool unit_t = temperature == 1.0;
    const double zm = block_max((double)zmax, s);
    const double mx = unit_t ? zm : zm / temperature;
    double acc = 0.0;
    const int v0 = (int)(((long long)V * part) / parts), v1 = (int)(((long long)V * (part + 1)) / parts);
    for (int v = v0 + tid; v < v1; v += ACC_THREADS) {
        const double p = (z[v] >= thr) ? exp((unit_t ? (double)z[v] : (double)z[v] / temperature) - mx) : 0.0;
        r[v] = p;
        acc += p;
    }
    const double den = block_sum(acc, s);
    if (total) *total = den;
    else
        for (int v = tid; v < V; v += ACC_THREADS) r[v] /= den;
    __syncthreads();
    return 0;
}

// One CTA per node: the rows' laws do not depend on the walk, so they are computed side by side before it (the walk
// then only compares, subtracts and scans); rows[i] is overwritten by the walk if node i is visited and a child refused.
// With a top-k cut a row's law is positive at few indices: list them (ascending), so that the walk's residual updates
// and its inverse-CDF scan touch those entries only instead of the whole vocabulary.
__device__ void list_support(const double *__restrict__ r, int V, int32_t *__restrict__ idx, int32_t *__restrict__ cnt, BlockScratch &s) {
    // warp w lists its contiguous share of the row, its lanes reading consecutive entries (ascending order is kept: by
    // iteration, then by lane); a first pass counts, a scan over the warps gives each its place, a second pass writes
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, warps = ACC_THREADS / 32;
    const int chunk = (V + warps - 1) / warps, v0 = min(V, warp * chunk), v1 = min(V, v0 + chunk);
    int mine = 0;
    for (int base = v0; base < v1; base += 32) { // (the same trip count for the lanes of a warp)
        const int v = base + lane;
        mine += __popc(__ballot_sync(0xffffffffu, v < v1 && r[v] > 0.0));
    }
    __syncthreads();
    if (lane == 0) s.i[warp] = mine;
    __syncthreads();
    int at = 0, total = 0;
    for (int w = 0; w < warps; ++w) {
        if (w < warp) at += s.i[w];
        total += s.i[w];
    }
    if (total <= SSD_ACC_SUPPORT) {
        for (int base = v0; base < v1; base += 32) {
            const int v = base + lane;
            const bool pos = v < v1 && r[v] > 0.0;
            const unsigned m = __ballot_sync(0xffffffffu, pos);
            if (pos) idx[at + __popc(m & ((1u << lane) - 1u))] = v;
            at += __popc(m);
        }
    }
    if (tid == 0) *cnt = total <= SSD_ACC_SUPPORT ? total : -1;
    __syncthreads();
}

constexpr int ACC_MAX_PARTS = 8; // slices a row's law is computed in (one CTA each)
__global__ void __launch_bounds__(ACC_THREADS) row_law_kernel(const float *__restrict__ logits, NodeList nodes, int use_list, int V, double temperature,
                                                              int top_k, double *__restrict__ rows, double *__restrict__ row_total,
                                                              int32_t *__restrict__ row_bad) {
    __shared__ BlockScratch s;
    const int row = blockIdx.x, node = use_list ? nodes.v[row] : row;
    double total = 1.0;
    const int bad = row_law(logits + (size_t)node * V, V, temperature, top_k, rows + (size_t)row * V, s, &total, blockIdx.y, gridDim.y);
    if (threadIdx.x == 0) {
        row_total[row * ACC_MAX_PARTS + blockIdx.y] = total;
        if (blockIdx.y == 0) row_bad[row] = bad; // (every slice sees the whole row: the same verdict)
    }
}
// The row's total from its slices' sums, in slice order (the same value in every thread and in every run).
__device__ __forceinline__ double row_total_of(const double *__restrict__ row_total, int row, int parts) {
    double t = 0.0;
    for (int p = 0; p < parts; ++p) t += row_total[row * ACC_MAX_PARTS + p];
    return t;
}
inline int law_parts(int rows) { // as many slices as keep all CTAs of the launch on the GPU at once
    int p = 148 / (rows > 0 ? rows : 1);
    return p < 1 ? 1 : (p > ACC_MAX_PARTS ? ACC_MAX_PARTS : p);
}

// Inverse-CDF draw from r (fp64, not necessarily normalised) by the whole CTA: ONE thread writes to *token_out the smallest v
// whose running sum exceeds u * sum(r); if rounding leaves none, the largest v with r[v] > 0.
__device__ void draw_from(const double *__restrict__ r, int V, double u, int32_t *__restrict__ token_out, BlockScratch &s) {
    const int tid = threadIdx.x;
    const int chunk = (V + ACC_THREADS - 1) / ACC_THREADS;
    const int v0 = min(V, tid * chunk), v1 = min(V, v0 + chunk);
    double csum = 0.0;
    int last_pos = -1;
    for (int v = v0; v < v1; ++v) { csum += r[v]; if (r[v] > 0.0) last_pos = v; }
    // inclusive scan of the chunk sums over the block
    double incl = csum;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const double t = __shfl_up_sync(0xffffffffu, incl, off);
        if ((tid & 31) >= off) incl += t;
    }
    __syncthreads();
    if ((tid & 31) == 31) s.d[tid >> 5] = incl;
    __syncthreads();
    double warp_base = 0.0, total = 0.0;
    for (int w = 0; w < ACC_THREADS / 32; ++w) {
        if (w < (tid >> 5)) warp_base += s.d[w];
        total += s.d[w];
    }
    incl += warp_base;
    const double target = u * total;
    const int first = block_min_int(incl > target ? tid : 0x7fffffff, s);
    const int fallback = block_max_int(last_pos, s);
    if (first == 0x7fffffff) {
        if (tid == 0) *token_out = fallback;
    } else if (tid == first) {
        double run = incl - csum;
        int pick = -1, lp = -1;
        for (int v = v0; v < v1; ++v) {
            if (r[v] > 0.0) lp = v;
            run += r[v];
            if (run > target) { pick = v; break; }
        }
        *token_out = pick >= 0 ? pick : lp;
    }
}

// What happens at node `cur`, whose target law is r (with its support list sup[0..cnt) if cnt >= 0): its children are
// tried in index order, each refusal replacing r by the renormalised residual.  Returns the accepted child (the same
// value in every thread), or -1 after ONE thread has written the extra token, drawn from r by inverse CDF, to *token_out.
// The outcome depends on cur's own logits, its children's proposal rows and the counter-based uniforms only - not on how
// the walk reached cur - so all nodes can be decided side by side.
//
// Proposal rows come dense (draft[c, :]) or as short lists (sp.idx / sp.val, [n][sp.entries], distinct indices, < 0 = unused).
// r is UNNORMALISED throughout, its total `norm` beside it (r_true = r / norm): the test u q[x] < r_true[x] becomes
// u q[x] norm < r[x], the residual max(0, r - q norm) with its own sum as the new total - no division anywhere.  With lists and a
// dense law a refusal touches the listed entries only (the residual differs from r there and nowhere else; the new total is
// norm minus what they lost): O(entries) per refusal instead of two passes over the vocabulary.  The extra token's inverse CDF
// sums r itself, so it needs no total.
struct SparseRows { const int32_t *idx; const float *val; int entries; };
__device__ __forceinline__ float q_at(const float *__restrict__ draft, const SparseRows &sp, int c, int V, int v) {
    if (!sp.idx) return draft[(size_t)c * V + v];
    for (int e = 0; e < sp.entries; ++e)
        if (sp.idx[(size_t)c * sp.entries + e] == v) return sp.val[(size_t)c * sp.entries + e];
    return 0.f;
}
__device__ int node_decide(double *r, int cnt, const int32_t *__restrict__ sup, const float *__restrict__ draft, const SparseRows sp,
                           const NodeList &tokens, const NodeList &parent, int n, int V, uint64_t seed, uint64_t step, int cur,
                           int32_t *__restrict__ token_out, BlockScratch &s, double norm, double *r_alt = nullptr) {
    // (norm: the total of r on entry; r_alt: a second row of V values, or null)
    const int tid = threadIdx.x;
    for (int c = cur + 1; c < n; ++c) {
        if (parent.v[c] != cur) continue;
        const float *q = draft ? draft + (size_t)c * V : nullptr;
        const int x = tokens.v[c];
        const double u = uniform24(seed, step, 2u * (uint32_t)c);
        if (u * (double)q_at(draft, sp, c, V, x) * norm < r[x]) return c; // every thread evaluates the same test on the same values
        // refusal: r <- max(0, r - q) renormalised (unchanged if nothing is left)
        __syncthreads(); // all threads have read r[x] before anyone rewrites it
        if (cnt >= 0) { // one support entry per thread
            const int iv = tid < cnt ? sup[tid] : 0;
            const double val = tid < cnt ? fmax(r[iv] - (double)q_at(draft, sp, c, V, iv) * norm, 0.0) : 0.0;
            const double Z = block_sum(val, s);
            if (Z > 0.0) {
                if (tid < cnt) r[iv] = val;
                norm = Z;
            }
        } else if (sp.idx) { // listed entries only
            double lost = 0.0;
            for (int e = tid; e < sp.entries; e += ACC_THREADS) {
                const int v = sp.idx[(size_t)c * sp.entries + e];
                if (v >= 0 && v < V) lost += r[v] - fmax(r[v] - (double)sp.val[(size_t)c * sp.entries + e] * norm, 0.0);
            }
            const double left = norm - block_sum(lost, s);
            if (left > 0.0) {
                for (int e = tid; e < sp.entries; e += ACC_THREADS) {
                    const int v = sp.idx[(size_t)c * sp.entries + e];
                    if (v >= 0 && v < V) r[v] = fmax(r[v] - (double)sp.val[(size_t)c * sp.entries + e] * norm, 0.0);
                }
                norm = left;
            }
        } else {
            double zs = 0.0;
            if (r_alt) { // one pass: the residual goes to the other row while it is summed, and becomes r only if something is left
                for (int v = tid; v < V; v += ACC_THREADS) { const double nv = fmax(r[v] - (double)q[v] * norm, 0.0); r_alt[v] = nv; zs += nv; }
                const double Z = block_sum(zs, s);
                if (Z > 0.0) { double *t = r; r = r_alt; r_alt = t; norm = Z; }
            } else {
                for (int v = tid; v < V; v += ACC_THREADS) zs += fmax(r[v] - (double)q[v] * norm, 0.0);
                const double Z = block_sum(zs, s);
                if (Z > 0.0) {
                    for (int v = tid; v < V; v += ACC_THREADS) r[v] = fmax(r[v] - (double)q[v] * norm, 0.0);
                    norm = Z;
                }
            }
        }
        __syncthreads();
    }
    // extra token from the residual by inverse CDF
    const double u = uniform24(seed, step, 2u * (uint32_t)cur + 1u);
    if (cnt >= 0) { // few entries: one thread scans them in index order
        if (tid == 0) {
            double total = 0.0;
            for (int i = 0; i < cnt; ++i) total += r[sup[i]];
            const double target = u * total;
            double run = 0.0;
            int pick = -1, lp = -1;
            for (int i = 0; i < cnt; ++i) {
                const int v = sup[i];
                if (r[v] > 0.0) lp = v;
                run += r[v];
                if (run > target) { pick = v; break; }
            }
            if (pick < 0) // (nothing beyond the target: the last positive entry, as in the full scan)
                for (int i = cnt - 1; i >= 0 && lp < 0; --i)
                    if (r[sup[i]] > 0.0) lp = sup[i];
            *token_out = pick >= 0 ? pick : lp;
        }
        return -1;
    }
    draw_from(r, V, u, token_out, s);
    return -1;
}

// The walk in one CTA, computing each visited row's law itself (the entry point that may not allocate, and the
// fall-back when the per-row scratch could not be had).
__global__ void __launch_bounds__(ACC_THREADS) sample_walk_kernel(const float *__restrict__ logits, const float *__restrict__ draft,
                                                                  NodeList tokens, NodeList parent, int n, int V, double temperature,
                                                                  int top_k, uint64_t seed, uint64_t step, double *__restrict__ r,
                                                                  int32_t *__restrict__ result, const int32_t *__restrict__ dev_status) {
    __shared__ BlockScratch s;
    const int tid = threadIdx.x;
    int cur = 0, np = 1;
    if (tid == 0) { result[3] = dev_status ? *dev_status : 0; result[4] = 0; }
    for (;;) {
        // a visited row must be finite
        double total = 1.0;
        if (row_law(logits + (size_t)cur * V, V, temperature, top_k, r, s, &total)) {
            if (tid == 0) { result[0] = 1; result[1] = -1; result[2] = SSD_ERR_BAD_ARG; }
            return;
        }
        const int c = node_decide(r, -1, nullptr, draft, SparseRows{nullptr, nullptr, 0}, tokens, parent, n, V, seed, step, cur, result + 1, s, total);
        if (c < 0) {
            if (tid == 0) { result[0] = np; result[2] = SSD_OK; }
            return;
        }
        if (tid == 0) result[4 + np] = c;
        ++np;
        cur = c;
        __syncthreads();
    }
}

// One CTA per node, after row_law_kernel: next[p] = the child accepted at p, -1 if none (bonus[p] then holds the extra
// token), -2 if p's logits are unusable.
__global__ void __launch_bounds__(ACC_THREADS) node_decide_kernel(const float *__restrict__ draft, SparseRows sp, NodeList tokens, NodeList parent, int n, int V,
                                                                  uint64_t seed, uint64_t step, double *__restrict__ rows, double *__restrict__ rows_alt,
                                                                  const double *__restrict__ row_total, int parts, int cut,
                                                                  const int32_t *__restrict__ row_bad, int32_t *__restrict__ sup_idx,
                                                                  int32_t *__restrict__ sup_cnt, int32_t *__restrict__ next,
                                                                  int32_t *__restrict__ bonus) {
    __shared__ BlockScratch s;
    const int p = blockIdx.x;
    if (row_bad[p]) {
        if (threadIdx.x == 0) next[p] = -2;
        return;
    }
    // with a top-k cut the law is positive at few indices: list them (ascending), so that the residual updates and the
    // inverse-CDF scan touch those entries only
    if (sup_cnt) {
        if (cut) list_support(rows + (size_t)p * V, V, sup_idx + (size_t)p * SSD_ACC_SUPPORT, sup_cnt + p, s);
        else if (threadIdx.x == 0) sup_cnt[p] = -1;
        __syncthreads();
    }
    const int cnt = sup_cnt ? sup_cnt[p] : -1;
    const int c = node_decide(rows + (size_t)p * V, cnt, cnt >= 0 ? sup_idx + (size_t)p * SSD_ACC_SUPPORT : nullptr, draft, sp, tokens, parent, n, V,
                              seed, step, p, bonus + p, s, row_total_of(row_total, p, parts), rows_alt ? rows_alt + (size_t)p * V : nullptr);
    if (threadIdx.x == 0) next[p] = c;
}

// Follows next[] from the root.  `result` may be pinned host memory.
__global__ void chain_walk_kernel(const int32_t *__restrict__ next, const int32_t *__restrict__ bonus, int n, int32_t *__restrict__ result,
                                  const int32_t *__restrict__ dev_status) {
    if (threadIdx.x != 0) return;
    int cur = 0, np = 1;
    result[3] = dev_status ? *dev_status : 0;
    result[4] = 0;
    for (;;) {
        const int c = next[cur];
        if (c == -2) { result[1] = -1; result[2] = SSD_ERR_BAD_ARG; result[0] = 1; return; }
        if (c < 0 || np >= n) { result[1] = bonus[cur]; result[2] = SSD_OK; result[0] = np; return; }
        result[4 + np++] = c;
        cur = c;
    }
}
} // namespace

cudaError_t launch_accept(const float *logits, const float *draft_probs, const NodeList &tokens, const NodeList &parent, int n,
                          int vocab, int mode, float temperature, int top_k, uint64_t seed, uint64_t step,
                          const AcceptScratch &sc, cudaStream_t s, int *launches) {
    if (mode == SSD_GREEDY) {
        if (sc.head_parts > 0) { // the LM head left the rows' statistics per output tile: nothing of the logits is read again
            greedy_walk_kernel<<<1, 32, 0, s>>>(tokens, parent, n, sc.head_parts, sc.head_val, sc.head_arg, sc.head_bad, sc.result, sc.dev_status);
            *launches += 1;
        } else {
            const int parts = sc.arg_parts > 0 ? sc.arg_parts : 1;
            row_argmax_kernel<<<dim3(n, parts), 256, 0, s>>>(logits, vocab, sc.row_val, sc.row_arg, sc.row_bad);
            greedy_walk_kernel<<<1, 32, 0, s>>>(tokens, parent, n, parts, sc.row_val, sc.row_arg, sc.row_bad, sc.result, sc.dev_status);
            *launches += 2;
        }
    } else {
        double *rows = (sc.rows && sc.rows_cap >= n && n > 1) ? sc.rows : nullptr;
        if (rows) {
            // every node is decided by a CTA of its own (its law, then its children in order), then a walk follows the decisions
            int32_t *next = sc.row_arg, *bonus = sc.row_arg + n; // (row_arg holds 4 ints per node on this path)
            const int parts = law_parts(n);
            row_law_kernel<<<dim3(n, parts), ACC_THREADS, 0, s>>>(logits, tokens, 0, vocab, (double)temperature, top_k, rows, sc.row_total, sc.row_bad);
            const SparseRows sp = {sc.sp_idx, sc.sp_val, sc.sp_entries}; // (lists instead of dense rows: draft_probs is then not read)
            node_decide_kernel<<<n, ACC_THREADS, 0, s>>>(draft_probs, sp, tokens, parent, n, vocab, seed, step, rows, sc.rows_alt, sc.row_total, parts, (top_k > 0 && top_k < vocab) ? 1 : 0,
                                                         sc.row_bad, sc.sup_idx, sc.sup_cnt, next, bonus);
            chain_walk_kernel<<<1, 32, 0, s>>>(next, bonus, n, sc.result, sc.dev_status);
            *launches += 3;
        } else {
            sample_walk_kernel<<<1, ACC_THREADS, 0, s>>>(logits, draft_probs, tokens, parent, n, vocab, (double)temperature, top_k, seed, step,
                                                         sc.r, sc.result, sc.dev_status);
            *launches += 1;
        }
    }
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Proposals of one stage for the stage above (Sections 3.1 / 3.2: a tree of likely continuations is assembled from
// the lower model's distributions - "the second or third most likely tokens" - or from draws of them).  For each
// listed node: its law (the same fp64 softmax with temperature and top-k cut that the acceptance rule uses as a
// node's target), written out as an fp32 row if asked, and `picks` candidate next tokens: the most probable ones in
// order (greedy), or independent inverse-CDF draws with the counter-based uniforms u(seed, step, 1024 + 16 node + t).
// One CTA per listed node; `scratch` holds one fp64 row per CTA.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(ACC_THREADS) propose_children_kernel(const float *__restrict__ logits, NodeList nodes, int V, double temperature,
                                                                       int top_k, int mode, int picks, uint64_t seed, uint64_t step,
                                                                       double *__restrict__ scratch, const double *__restrict__ row_total, int parts,
                                                                       const int32_t *__restrict__ row_bad, float *__restrict__ rows_out,
                                                                       int32_t *__restrict__ tokens_out, int32_t *__restrict__ bad_out) {
    __shared__ BlockScratch s;
    __shared__ int32_t s_pick;
    const int j = blockIdx.x, node = nodes.v[j], tid = threadIdx.x;
    double *r = scratch + (size_t)j * V;
    // (row_law_kernel has left the law of listed node j in scratch row j, unnormalised: the picks and draws do not need it
    //  otherwise, the row written out is divided on its way)
    const double total = row_total_of(row_total, j, parts);
    const int bad = row_bad[j];
    if (tid == 0) bad_out[j] = bad;
    if (bad) {
        for (int t = tid; t < picks; t += ACC_THREADS) tokens_out[j * picks + t] = -1;
        return;
    }
    if (rows_out)
        for (int v = tid; v < V; v += ACC_THREADS) rows_out[(size_t)j * V + v] = (float)(r[v] / total);
    for (int t = 0; t < picks; ++t) {
        if (mode == SSD_GREEDY) { // the most probable token not yet picked; ties towards the lower id
            double best = -1.0;
            int arg = 0x7fffffff;
            for (int v = tid; v < V; v += ACC_THREADS)
                if (r[v] > best) { best = r[v]; arg = v; } // (ascending v per thread: the first maximum is the lowest id)
            const double top = block_max(best, s);
            const int pick = block_min_int(best == top ? arg : 0x7fffffff, s);
            if (tid == 0) { tokens_out[j * picks + t] = pick; r[pick] = -1.0; }
            __syncthreads();
        } else {
            const double u = uniform24(seed, step, 1024u + 16u * (uint32_t)node + (uint32_t)t);
            draw_from(r, V, u, &s_pick, s);
            __syncthreads();
            if (tid == 0) tokens_out[j * picks + t] = s_pick;
        }
    }
}

cudaError_t launch_propose_children(const float *logits, const NodeList &nodes, int m, int vocab, int mode, float temperature, int top_k, int picks,
                                    uint64_t seed, uint64_t step, double *scratch, double *row_total, int32_t *row_bad, float *rows_out,
                                    int32_t *tokens_out, int32_t *bad_out, cudaStream_t s) {
    const int parts = law_parts(m);
    row_law_kernel<<<dim3(m, parts), ACC_THREADS, 0, s>>>(logits, nodes, 1, vocab, (double)temperature, top_k, scratch, row_total, row_bad);
    propose_children_kernel<<<m, ACC_THREADS, 0, s>>>(logits, nodes, vocab, (double)temperature, top_k, mode, picks, seed, step, scratch, row_total, parts,
                                                      row_bad, rows_out, tokens_out, bad_out);
    return cudaGetLastError();
}

// rows[j, :] = 0 except rows[j, idx[j, e]] = val[j, e] for the listed entries (idx < 0: unused slot): proposal rows given
// as short index / value lists (a trigram row has four non-zeros, a deterministic proposal one) made dense for the
// acceptance kernels.  One CTA per row.
__global__ void __launch_bounds__(256) expand_sparse_rows_kernel(const int32_t *__restrict__ idx, const float *__restrict__ val, int entries, int V,
                                                                 float *__restrict__ rows) {
    float *row = rows + (size_t)blockIdx.x * V;
    if ((V & 3) == 0 && (reinterpret_cast<uintptr_t>(row) & 15) == 0) {
        float4 *r4 = reinterpret_cast<float4 *>(row);
        for (int v = threadIdx.x; v < V / 4; v += 256) r4[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    } else {
        for (int v = threadIdx.x; v < V; v += 256) row[v] = 0.f;
    }
    __syncthreads();
    for (int e = threadIdx.x; e < entries; e += 256) {
        const int v = idx[(size_t)blockIdx.x * entries + e];
        if (v >= 0 && v < V) row[v] = val[(size_t)blockIdx.x * entries + e];
    }
}
cudaError_t launch_expand_sparse_rows(const int32_t *idx, const float *val, int n, int entries, int vocab, float *rows, cudaStream_t s) {
    expand_sparse_rows_kernel<<<n, 256, 0, s>>>(idx, val, entries, vocab, rows);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// A wait that runs out, for testing the failure path without touching the production kernels: one warp waits, with
// the same bounded wait the projection kernels use, on an mbarrier at which nothing ever arrives (no copy, no MMA and
// no tensor memory is in flight), records the error word when the limit expires and returns.
// ---------------------------------------------------------------------------------------------
__global__ void expired_wait_kernel(int32_t *status, long long limit_cycles) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) { ptx::mbar_init(&bar, 1); ptx::fence_mbar_init(); }
    __syncwarp();
    if (threadIdx.x == 0 && !ptx::mbar_wait_bounded(&bar, 0, limit_cycles)) atomicExch(status, 0xE00);
}
cudaError_t launch_expired_wait(int32_t *status, long long limit_cycles, cudaStream_t s) {
    expired_wait_kernel<<<1, 32, 0, s>>>(status, limit_cycles);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Acceptance walk for callers that must not allocate (no counterpart in the paper).
//
// All device scratch of this entry point lives in the fixed arrays below, which every GPU that
// loads the library reserves until the process exits (about 0.5 MB).  Host code may not pass
// the array NAMES to a kernel - on the host they are only stand-ins for the symbols - so the
// device addresses are looked up once per device with cudaGetSymbolAddress and cached.
// ---------------------------------------------------------------------------------------------
static __device__ __align__(256) double g_noalloc_residual[SSD_NOALLOC_MAX_VOCAB];
static __device__ __align__(256) float g_noalloc_row_val[SSD_MAX_NODES];
static __device__ __align__(256) int32_t g_noalloc_row_arg[SSD_MAX_NODES];
static __device__ __align__(256) int32_t g_noalloc_row_bad[SSD_MAX_NODES];
static __device__ __align__(256) int32_t g_noalloc_result[SSD_MAX_NODES + 4];

namespace {
constexpr int NOALLOC_MAX_DEVICES = 64;
struct NoAllocScratch {
    bool ready;
    AcceptScratch sc;
};
NoAllocScratch g_noalloc[NOALLOC_MAX_DEVICES]; // zero-initialised; one slot per device ordinal
std::mutex g_noalloc_mutex;                     // guards the one-time set-up (a static mutex allocates nothing)

// First use on a device (with that device current): resolve the symbols' device addresses.
cudaError_t noalloc_setup(int device, AcceptScratch *out) {
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    NoAllocScratch &slot = g_noalloc[device];
    if (!slot.ready) {
        void *r = nullptr, *val = nullptr, *arg = nullptr, *bad = nullptr, *res = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&r, g_noalloc_residual);
        if (e == cudaSuccess) e = cudaGetSymbolAddress(&val, g_noalloc_row_val);
        if (e == cudaSuccess) e = cudaGetSymbolAddress(&arg, g_noalloc_row_arg);
        if (e == cudaSuccess) e = cudaGetSymbolAddress(&bad, g_noalloc_row_bad);
        if (e == cudaSuccess) e = cudaGetSymbolAddress(&res, g_noalloc_result);
        if (e != cudaSuccess) return e;
        slot.sc.r = (double *)r;
        slot.sc.row_val = (float *)val;
        slot.sc.row_arg = (int32_t *)arg;
        slot.sc.row_bad = (int32_t *)bad;
        slot.sc.result = (int32_t *)res;
        slot.sc.dev_status = nullptr;
        slot.sc.head_parts = 0;
        slot.sc.sp_idx = nullptr; slot.sc.sp_val = nullptr; slot.sc.sp_entries = 0; slot.sc.rows_alt = nullptr;
        slot.ready = true;
    }
    *out = slot.sc;
    return cudaSuccess;
}
} // namespace

extern "C" int ssd_accept_tree_noalloc(int device, void *cuda_stream, const float *logits, const float *draft_probs, const int32_t *tokens,
                                       const int32_t *parent_idx, int32_t n_nodes, int32_t vocab, const ssd_sampling *sampling,
                                       ssd_rng *rng_state, int32_t *path_out, int32_t *n_path_out, int32_t *next_token_out) {
    if (!logits || !tokens || !parent_idx || !sampling || !rng_state || !path_out || !n_path_out || !next_token_out) return SSD_ERR_BAD_ARG;
    if (sampling->mode != SSD_GREEDY && sampling->mode != SSD_SAMPLING) return SSD_ERR_BAD_ARG;
    if (sampling->mode == SSD_SAMPLING && (!draft_probs || !(sampling->temperature > 0.f) || sampling->top_k < 0)) return SSD_ERR_BAD_ARG;
    if (device < 0 || device >= NOALLOC_MAX_DEVICES) return SSD_ERR_BAD_ARG;
    // the fixed scratch bounds the problem size
    if (vocab < 1 || vocab > SSD_NOALLOC_MAX_VOCAB) return SSD_ERR_UNSUPPORTED;
    if (n_nodes < 1 || n_nodes > SSD_MAX_NODES) return SSD_ERR_INVALID_TREE;
    if (parent_idx[0] != -1) return SSD_ERR_INVALID_TREE;
    for (int i = 1; i < n_nodes; ++i)
        if (parent_idx[i] < 0 || parent_idx[i] >= i) return SSD_ERR_INVALID_TREE;
    for (int i = 0; i < n_nodes; ++i)
        if (tokens[i] < 0 || tokens[i] >= vocab) return SSD_ERR_BAD_ARG;

    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return SSD_ERR_CUDA;
    if (prev != device && cudaSetDevice(device) != cudaSuccess) return SSD_ERR_CUDA;
    int rc = SSD_OK;
    AcceptScratch sc;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    int32_t host[SSD_MAX_NODES + 4]; // on the stack: no allocation on the host either
    NodeList tk, pr;
    memcpy(tk.v, tokens, sizeof(int32_t) * n_nodes);
    memcpy(pr.v, parent_idx, sizeof(int32_t) * n_nodes);
    int launched = 0;
    cudaError_t e = noalloc_setup(device, &sc);
    if (e == cudaSuccess)
        e = launch_accept(logits, draft_probs, tk, pr, n_nodes, vocab, sampling->mode, sampling->temperature, sampling->top_k, rng_state->seed,
                          rng_state->step, sc, s, &launched);
    if (e == cudaSuccess) e = cudaMemcpyAsync(host, sc.result, sizeof(int32_t) * (n_nodes + 4), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) {
        cudaGetLastError();
        rc = SSD_ERR_CUDA;
    } else {
        rng_state->step += 1;
        const int np = host[0];
        if (np < 1 || np > n_nodes) {
            rc = SSD_ERR_CUDA;
        } else {
            *n_path_out = np;
            *next_token_out = host[1];
            memcpy(path_out, host + 4, sizeof(int32_t) * np);
            rc = host[2];
        }
    }
    if (prev != device) cudaSetDevice(prev);
    return rc;
}
