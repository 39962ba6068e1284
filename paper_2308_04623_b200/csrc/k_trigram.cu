// The lowest speculation stage: a Katz back-off trigram model that proposes a small token tree.
//
// Section 4 of the paper names it (the third model of the staged pipeline, Section 3.2), and its closing list
// asks for lowest-level drafts that answer in under 10 microseconds.  The paper gives no formula; the reading
// taken here: counts over a token stream, absolute discount D = 0.5,
//     P3(w | a, b) = (c3(a,b,w) - D) / c3(a,b,.)  if seen, else alpha3(a,b) * P2(w | b)      (same one level down,
//     P1(w) = c1(w) / N), alpha = discounted mass / (1 - lower-order mass of the seen tokens),
// a context never seen backs off entirely, and the proposals of a context are its four most probable next
// tokens (ties towards the lower id).
//
// Build (host, once per stream): the counts, then for every context the stream contains its four best
// continuations with their probabilities, all in fp64 with sums taken in token order; what goes to the device
// is a table of answers: an open-addressing hash keyed by (a, b), a direct-indexed array keyed by b for contexts
// that back off to the bigram level, and the unigram list.  Lookup (device): one warp; its lanes probe
// consecutive slots of the hash at once.  A proposal tree of eight nodes is four dependent lookups.
#include <algorithm>
#include <cstring>
#include <new>
#include <unordered_map>
#include <vector>

#include "ssd_internal.h"

namespace {
constexpr int TRI_TOP = 4;
constexpr double TRI_DISCOUNT = 0.5;
constexpr uint64_t TRI_EMPTY = ~0ull;

struct TriEntry {
    int32_t tok[TRI_TOP];
    float prob[TRI_TOP];
};

__host__ __device__ inline uint64_t tri_hash(uint64_t key) { // splitmix64 finaliser
    key ^= key >> 30; key *= 0xbf58476d1ce4e5b9ull;
    key ^= key >> 27; key *= 0x94d049bb133111ebull;
    key ^= key >> 31;
    return key;
}

struct TriTables {
    const uint64_t *keys;   // [cap] (a << 32 | b) or TRI_EMPTY
    const TriEntry *vals;   // [cap]
    uint64_t mask;          // cap - 1
    const TriEntry *bi;     // [vocab]; tok[0] < 0: token never seen as a context
    TriEntry uni;
    int vocab;
};

// The whole warp looks (a, b) up: trigram context, else bigram context, else the unigram list.
__device__ __forceinline__ TriEntry tri_lookup(const TriTables &t, int a, int b, int lane) {
    if (a >= 0 && a < t.vocab && b >= 0 && b < t.vocab) {
        const uint64_t key = ((uint64_t)(uint32_t)a << 32) | (uint32_t)b;
        uint64_t slot = tri_hash(key) & t.mask;
        for (uint64_t probed = 0; probed <= t.mask; probed += 32) { // (bounded: at most one pass over the table)
            const uint64_t at = (slot + lane) & t.mask;
            const uint64_t k = t.keys[at];
            const unsigned hit = __ballot_sync(0xffffffffu, k == key), empty = __ballot_sync(0xffffffffu, k == TRI_EMPTY);
            // linear probing: the key, if present, sits before the first empty slot of its probe sequence
            const int first_hit = hit ? __ffs(hit) - 1 : 32, first_empty = empty ? __ffs(empty) - 1 : 32;
            if (first_hit < first_empty) return t.vals[(slot + first_hit) & t.mask];
            if (empty) break;
            slot = (slot + 32) & t.mask;
        }
    }
    if (b >= 0 && b < t.vocab && t.bi[b].tok[0] >= 0) return t.bi[b];
    return t.uni;
}

// contexts[q] = (a, b) -> out[q]: one warp per query.
__global__ void trigram_lookup_kernel(TriTables t, const int32_t *__restrict__ contexts, int m, TriEntry *__restrict__ out) {
    const int q = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (q >= m) return;
    const TriEntry e = tri_lookup(t, contexts[2 * q], contexts[2 * q + 1], lane);
    if (lane == 0) out[q] = e;
}

// Fills a tree: node 0 holds `root`, preceded by `prev1`; the children of a node, in index order, get the best
// continuations of (token before the node, the node's token).  One warp; result = tokens[n] then probabilities[n] (as
// float bits) in `result` (may be pinned host memory).
__global__ void trigram_tree_kernel(TriTables t, int prev1, int root, NodeList parent, int n, int32_t *__restrict__ result) {
    __shared__ int s_tok[SSD_MAX_NODES], s_before[SSD_MAX_NODES];
    __shared__ float s_prob[SSD_MAX_NODES];
    const int lane = threadIdx.x;
    if (lane == 0) { s_tok[0] = root; s_before[0] = prev1; s_prob[0] = 0.f; }
    __syncwarp();
    for (int p = 0; p < n; ++p) {
        // children of p: indices above p (parent[i] < i), found by all lanes together
        int rank = 0;
        bool fetched = false;
        TriEntry e;
        for (int base = p + 1; base < n; base += 32) {
            const int i = base + lane;
            const bool mine = i < n && parent.v[i] == p;
            const unsigned kids = __ballot_sync(0xffffffffu, mine);
            if (kids && !fetched) { e = tri_lookup(t, s_before[p], s_tok[p], lane); fetched = true; }
            if (mine) {
                const int r = rank + __popc(kids & ((1u << lane) - 1u));
                // (more children than stored continuations: the extra ones repeat the last stored one)
                const int pick = r < TRI_TOP ? r : TRI_TOP - 1;
                s_tok[i] = e.tok[pick]; s_prob[i] = e.prob[pick]; s_before[i] = s_tok[p];
            }
            rank += __popc(kids);
        }
        __syncwarp();
    }
    for (int i = lane; i < n; i += 32) { result[i] = s_tok[i]; result[n + i] = __float_as_int(s_prob[i]); }
}

// ---------------------------------------------------------------------------------------------------------------
// host side: counts and the per-context answers
// ---------------------------------------------------------------------------------------------------------------
struct Cand { double p; int w; };
inline bool better(const Cand &x, const Cand &y) { return x.p > y.p || (x.p == y.p && x.w < y.w); }

typedef std::vector<std::pair<int, long long>> Seen; // (token, count), ascending token

struct Builder {
    int V;
    long long N;
    std::vector<long long> c1;
    std::vector<int> uni_order;                       // tokens by (count descending, id ascending)
    std::unordered_map<int, Seen> c2;
    std::unordered_map<uint64_t, Seen> c3;
    std::unordered_map<int, double> alpha2;

    double p1(int w) const { return (double)c1[w] / (double)N; }
    static long long total(const Seen &s) { long long t = 0; for (auto &e : s) t += e.second; return t; }
    static long long count_of(const Seen &s, int w) {
        auto it = std::lower_bound(s.begin(), s.end(), std::make_pair(w, 0ll), [](const std::pair<int, long long> &x, const std::pair<int, long long> &y) { return x.first < y.first; });
        return (it != s.end() && it->first == w) ? it->second : 0;
    }
    double p2(int w, int b) const {
        auto it = c2.find(b);
        if (it == c2.end()) return p1(w);
        const long long c = count_of(it->second, w);
        if (c > 0) return ((double)c - TRI_DISCOUNT) / (double)total(it->second);
        return alpha2.at(b) * p1(w);
    }
    // The k best tokens by `prob(w)` among those not in `skip`, where the tokens of `seen` have their own probabilities and
    // all others are ranked by `lower(w)` scaled by `alpha`: merge of the seen list and a scan of `lower_order`.
    template <typename LowerFn>
    void unseen_best(const Seen &seen_here, const Seen *skip, double alpha, const std::vector<int> &lower_order, LowerFn lower, int k, std::vector<Cand> &out) const {
        int found = 0;
        for (size_t at = 0; at < lower_order.size() && found < k; ++at) {
            const int w = lower_order[at];
            if (count_of(seen_here, w) > 0 || (skip && count_of(*skip, w) > 0)) continue;
            out.push_back(Cand{alpha * lower(w), w});
            ++found;
        }
    }
};

void top_k(std::vector<Cand> &c, int k, TriEntry &e) {
    std::sort(c.begin(), c.end(), better);
    for (int q = 0; q < TRI_TOP; ++q) {
        if (q < (int)c.size() && q < k) { e.tok[q] = c[q].w; e.prob[q] = (float)c[q].p; }
        else { e.tok[q] = q > 0 ? e.tok[q - 1] : 0; e.prob[q] = 0.f; }
    }
}
} // namespace

struct ssd_trigram {
    int device;
    cudaStream_t stream;
    int vocab;
    uint64_t *d_keys;
    TriEntry *d_vals, *d_bi, *d_out;
    int32_t *d_ctx;
    int32_t *h_result; // pinned
    TriTables t;
    size_t contexts;
};

extern "C" {

int ssd_trigram_build(const int32_t *stream_tokens, int64_t n_tokens, int32_t vocab, int device, void *cuda_stream, ssd_trigram **out) {
    if (out) *out = nullptr;
    if (!stream_tokens || !out || n_tokens < 3 || vocab < TRI_TOP || vocab > (1 << 24)) return SSD_ERR_BAD_ARG;
    for (int64_t i = 0; i < n_tokens; ++i)
        if (stream_tokens[i] < 0 || stream_tokens[i] >= vocab) return SSD_ERR_BAD_ARG;
    Builder B;
    B.V = vocab; B.N = n_tokens;
    B.c1.assign(vocab, 0);
    std::unordered_map<int, std::unordered_map<int, long long>> m2;
    std::unordered_map<uint64_t, std::unordered_map<int, long long>> m3;
    for (int64_t i = 0; i < n_tokens; ++i) {
        const int w = stream_tokens[i];
        ++B.c1[w];
        if (i >= 1) ++m2[stream_tokens[i - 1]][w];
        if (i >= 2) ++m3[((uint64_t)(uint32_t)stream_tokens[i - 2] << 32) | (uint32_t)stream_tokens[i - 1]][w];
    }
    auto sorted = [](const std::unordered_map<int, long long> &m) { Seen s(m.begin(), m.end()); std::sort(s.begin(), s.end()); return s; };
    for (auto &kv : m2) B.c2[kv.first] = sorted(kv.second);
    for (auto &kv : m3) B.c3[kv.first] = sorted(kv.second);
    B.uni_order.resize(vocab);
    for (int w = 0; w < vocab; ++w) B.uni_order[w] = w;
    std::stable_sort(B.uni_order.begin(), B.uni_order.end(), [&](int x, int y) { return B.c1[x] > B.c1[y]; });
    // back-off weights of the bigram level (sums in ascending token order)
    for (auto &kv : B.c2) {
        double lower = 0.0;
        for (auto &e : kv.second) lower += B.p1(e.first);
        const long long tot = Builder::total(kv.second);
        B.alpha2[kv.first] = lower < 1.0 ? (TRI_DISCOUNT * (double)kv.second.size() / (double)tot) / (1.0 - lower) : 0.0;
    }
    // ---- answers
    TriEntry uni;
    {
        std::vector<Cand> c;
        for (int q = 0; q < TRI_TOP; ++q) c.push_back(Cand{B.p1(B.uni_order[q]), B.uni_order[q]});
        top_k(c, TRI_TOP, uni);
    }
    std::vector<TriEntry> bi(vocab);
    for (int b = 0; b < vocab; ++b) { bi[b].tok[0] = -1; for (int q = 0; q < TRI_TOP; ++q) bi[b].prob[q] = 0.f; }
    const Seen none;
    for (auto &kv : B.c2) {
        const int b = kv.first;
        const Seen &s2 = kv.second;
        const long long tot = Builder::total(s2);
        std::vector<Cand> c;
        for (auto &e : s2) c.push_back(Cand{((double)e.second - TRI_DISCOUNT) / (double)tot, e.first});
        B.unseen_best(s2, nullptr, B.alpha2[b], B.uni_order, [&](int w) { return B.p1(w); }, TRI_TOP, c);
        top_k(c, TRI_TOP, bi[b]);
    }
    size_t cap = 64;
    while (cap < 2 * B.c3.size() + 64) cap <<= 1;
    std::vector<uint64_t> keys(cap, TRI_EMPTY);
    std::vector<TriEntry> vals(cap);
    for (auto &kv : B.c3) {
        const int b = (int)(uint32_t)kv.first;
        const Seen &s3 = kv.second;
        const long long tot = Builder::total(s3);
        double lower = 0.0;
        for (auto &e : s3) lower += B.p2(e.first, b);
        const double alpha3 = lower < 1.0 ? (TRI_DISCOUNT * (double)s3.size() / (double)tot) / (1.0 - lower) : 0.0;
        std::vector<Cand> c;
        for (auto &e : s3) c.push_back(Cand{((double)e.second - TRI_DISCOUNT) / (double)tot, e.first});
        // unseen after (a, b): ranked by P2(. | b): the tokens seen after b (own probabilities) and the rest by unigram count
        auto it2 = B.c2.find(b);
        if (it2 != B.c2.end()) {
            const Seen &s2 = it2->second;
            const long long tot2 = Builder::total(s2);
            std::vector<int> by_p2;
            for (auto &e : s2) by_p2.push_back(e.first);
            std::stable_sort(by_p2.begin(), by_p2.end(), [&](int x, int y) { return Builder::count_of(s2, x) > Builder::count_of(s2, y); });
            B.unseen_best(s3, nullptr, alpha3, by_p2, [&](int w) { return ((double)Builder::count_of(s2, w) - TRI_DISCOUNT) / (double)tot2; }, TRI_TOP, c);
            const double a2 = B.alpha2[b];
            B.unseen_best(s3, &s2, alpha3, B.uni_order, [&](int w) { return a2 * B.p1(w); }, TRI_TOP, c);
        } else {
            B.unseen_best(s3, nullptr, alpha3, B.uni_order, [&](int w) { return B.p1(w); }, TRI_TOP, c);
        }
        TriEntry e;
        top_k(c, TRI_TOP, e);
        uint64_t slot = tri_hash(kv.first) & (cap - 1);
        while (keys[slot] != TRI_EMPTY) slot = (slot + 1) & (cap - 1);
        keys[slot] = kv.first;
        vals[slot] = e;
    }
    // ---- device tables
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return SSD_ERR_CUDA;
    if (prev != device && cudaSetDevice(device) != cudaSuccess) return SSD_ERR_CUDA;
    ssd_trigram *t = new (std::nothrow) ssd_trigram();
    if (!t) return SSD_ERR_NOMEM;
    memset(t, 0, sizeof(*t));
    t->device = device; t->stream = (cudaStream_t)cuda_stream; t->vocab = vocab; t->contexts = B.c3.size();
    cudaError_t e = cudaMalloc((void **)&t->d_keys, cap * sizeof(uint64_t));
    if (e == cudaSuccess) e = cudaMalloc((void **)&t->d_vals, cap * sizeof(TriEntry));
    if (e == cudaSuccess) e = cudaMalloc((void **)&t->d_bi, (size_t)vocab * sizeof(TriEntry));
    if (e == cudaSuccess) e = cudaMalloc((void **)&t->d_out, 4096 * sizeof(TriEntry));
    if (e == cudaSuccess) e = cudaMalloc((void **)&t->d_ctx, 4096 * 2 * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMallocHost((void **)&t->h_result, 2 * SSD_MAX_NODES * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemcpyAsync(t->d_keys, keys.data(), cap * sizeof(uint64_t), cudaMemcpyHostToDevice, t->stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(t->d_vals, vals.data(), cap * sizeof(TriEntry), cudaMemcpyHostToDevice, t->stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(t->d_bi, bi.data(), (size_t)vocab * sizeof(TriEntry), cudaMemcpyHostToDevice, t->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(t->stream);
    if (prev != device) cudaSetDevice(prev);
    if (e != cudaSuccess) { cudaGetLastError(); ssd_trigram_destroy(t); return e == cudaErrorMemoryAllocation ? SSD_ERR_NOMEM : SSD_ERR_CUDA; }
    t->t.keys = t->d_keys; t->t.vals = t->d_vals; t->t.mask = cap - 1; t->t.bi = t->d_bi; t->t.uni = uni; t->t.vocab = vocab;
    *out = t;
    return SSD_OK;
}

void ssd_trigram_destroy(ssd_trigram *t) {
    if (!t) return;
    int prev = -1;
    cudaGetDevice(&prev);
    if (prev != t->device) cudaSetDevice(t->device);
    cudaStreamSynchronize(t->stream);
    cudaFree(t->d_keys); cudaFree(t->d_vals); cudaFree(t->d_bi); cudaFree(t->d_out); cudaFree(t->d_ctx);
    if (t->h_result) cudaFreeHost(t->h_result);
    if (prev >= 0 && prev != t->device) cudaSetDevice(prev);
    delete t;
}

int ssd_trigram_lookup(ssd_trigram *t, const int32_t *contexts, int32_t m, int32_t *tokens_out, float *probs_out) {
    if (!t || !contexts || !tokens_out || !probs_out || m < 1 || m > 4096) return SSD_ERR_BAD_ARG;
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return SSD_ERR_CUDA;
    if (prev != t->device && cudaSetDevice(t->device) != cudaSuccess) return SSD_ERR_CUDA;
    std::vector<TriEntry> host(m);
    cudaError_t e = cudaMemcpyAsync(t->d_ctx, contexts, sizeof(int32_t) * 2 * m, cudaMemcpyHostToDevice, t->stream);
    if (e == cudaSuccess) {
        trigram_lookup_kernel<<<(m + 3) / 4, 128, 0, t->stream>>>(t->t, t->d_ctx, m, t->d_out);
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaMemcpyAsync(host.data(), t->d_out, sizeof(TriEntry) * m, cudaMemcpyDeviceToHost, t->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(t->stream);
    if (prev != t->device) cudaSetDevice(prev);
    if (e != cudaSuccess) { cudaGetLastError(); return SSD_ERR_CUDA; }
    for (int q = 0; q < m; ++q)
        for (int r = 0; r < TRI_TOP; ++r) { tokens_out[q * TRI_TOP + r] = host[q].tok[r]; probs_out[q * TRI_TOP + r] = host[q].prob[r]; }
    return SSD_OK;
}

int ssd_trigram_propose(ssd_trigram *t, int32_t prev1, int32_t root, const int32_t *parent_idx, int32_t n_nodes, int32_t *tokens_out, float *probs_out) {
    if (!t || !parent_idx || !tokens_out || !probs_out) return SSD_ERR_BAD_ARG;
    if (n_nodes < 1 || n_nodes > SSD_MAX_NODES || parent_idx[0] != -1) return SSD_ERR_INVALID_TREE;
    for (int i = 1; i < n_nodes; ++i)
        if (parent_idx[i] < 0 || parent_idx[i] >= i) return SSD_ERR_INVALID_TREE;
    if (root < 0 || root >= t->vocab) return SSD_ERR_BAD_ARG;
    {   // a context has four stored continuations: no node may have more children
        int kids[SSD_MAX_NODES] = {0};
        for (int i = 1; i < n_nodes; ++i)
            if (++kids[parent_idx[i]] > TRI_TOP) return SSD_ERR_INVALID_TREE;
    }
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return SSD_ERR_CUDA;
    if (prev != t->device && cudaSetDevice(t->device) != cudaSuccess) return SSD_ERR_CUDA;
    NodeList pr;
    memcpy(pr.v, parent_idx, sizeof(int32_t) * n_nodes);
    trigram_tree_kernel<<<1, 32, 0, t->stream>>>(t->t, prev1, root, pr, n_nodes, t->h_result); // results straight into pinned host memory
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaStreamSynchronize(t->stream);
    if (prev != t->device) cudaSetDevice(prev);
    if (e != cudaSuccess) { cudaGetLastError(); return SSD_ERR_CUDA; }
    memcpy(tokens_out, t->h_result, sizeof(int32_t) * n_nodes);
    memcpy(probs_out, t->h_result + n_nodes, sizeof(float) * n_nodes);
    return SSD_OK;
}

int ssd_trigram_contexts(const ssd_trigram *t, int64_t *count) {
    if (!t || !count) return SSD_ERR_BAD_ARG;
    *count = (int64_t)t->contexts;
    return SSD_OK;
}

} // extern "C"
