"""Seeded synthetic inputs for the tree-verification hot path.

This module holds input *generators only*: model shapes, random weights, token
trees, prefixes and draft-probability rows.  It contains none of the method's
arithmetic (no transformer maths, no acceptance rule, no random-number scheme
of the method itself), so both the CPU oracle's tests and the CUDA library's
tests may draw the same arrays from it without sharing any code of the method.

Everything is a pure function of (configuration, seed) through
``numpy.random.default_rng``.  The shapes follow the paper's workload
(Section 4: a GPT-2-Large verifier, a GPT-2 draft, 16-bit weights, batch 1,
context 1024); the paper's trained weights and prompts are not available, so
weights are random N(0, 0.02) and token ids are uniform.
"""
from __future__ import annotations

import numpy as np

# ----------------------------------------------------------------------------
# Model shapes (GPT-2 family, Section 4 of the paper names GPT-2-Large and a
# small GPT-2 draft; the XL shape is the scaling sweep).
# ----------------------------------------------------------------------------
CONFIGS = {
    "tiny": dict(n_layer=4, d_model=256, n_head=4, d_head=64, d_ff=1024, vocab=1024,
                 n_ctx=1024, max_nodes=256, dtype="fp32"),
    "tiny_bf16": dict(n_layer=4, d_model=256, n_head=4, d_head=64, d_ff=1024, vocab=1024,
                      n_ctx=1024, max_nodes=256, dtype="bf16"),
    # odd sizes: vocabulary not a multiple of any tile, three heads
    "ragged_bf16": dict(n_layer=2, d_model=192, n_head=3, d_head=64, d_ff=768, vocab=1000 + 37,
                        n_ctx=256, max_nodes=256, dtype="bf16"),
    "gpt2_small": dict(n_layer=12, d_model=768, n_head=12, d_head=64, d_ff=3072, vocab=50257,
                       n_ctx=1024, max_nodes=256, dtype="bf16"),
    "gpt2_large": dict(n_layer=36, d_model=1280, n_head=20, d_head=64, d_ff=5120, vocab=50257,
                       n_ctx=1024, max_nodes=256, dtype="bf16"),
    "gpt2_xl": dict(n_layer=48, d_model=1600, n_head=25, d_head=64, d_ff=6400, vocab=50257,
                    n_ctx=1024, max_nodes=256, dtype="bf16"),
}

LN_EPS = 1e-5


def config(name: str, **overrides) -> dict:
    c = dict(CONFIGS[name])
    c.update(overrides)
    c["ln_eps"] = LN_EPS
    return c


# ----------------------------------------------------------------------------
# bf16 helpers (storage format conversion only)
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even); returns the 16-bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """fp32 array whose values are exactly representable in bf16."""
    return bf16_bits_to_f32(f32_to_bf16_bits(a))


# ----------------------------------------------------------------------------
# Weights
# ----------------------------------------------------------------------------
# Fixed tensor order of the one random stream (so a seed names one model).
_PER_LAYER = ("ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o",
              "ln2_g", "ln2_b", "w_fc", "b_fc", "w_proj", "b_proj")


def make_weights(cfg: dict, seed: int = 0, qk_gain: float = 1.0) -> dict:
    """Random GPT-2-style weights.

    Every matrix is ``[out_features, in_features]`` row-major; ``w_qkv`` stacks
    the query, key and value projections (each head-major) along its rows.
    All matrices, embeddings and biases are N(0, 0.02); LayerNorm gains are
    1 + N(0, 0.02) and LayerNorm biases N(0, 0.02), so that every bias and gain
    path is exercised.  For a bf16 model every tensor is rounded to bf16 once,
    here; the returned fp32 arrays then hold exactly-representable values and
    ``bf16_bits`` gives the 16-bit patterns of the same numbers.

    ``qk_gain`` multiplies the query and key rows of ``w_qkv`` (a "sharpened"
    test model whose attention is far from uniform, so that a wrong mask or
    position shows up in the logits).
    """
    rng = np.random.default_rng(seed)
    L, d, F, V, C = cfg["n_layer"], cfg["d_model"], cfg["d_ff"], cfg["vocab"], cfg["n_ctx"]
    bf16 = cfg["dtype"] != "fp32"   # ("bf16_w8": a bf16 model whose matrices the library holds as 8-bit codes)

    def normal(*shape):
        return (rng.standard_normal(shape, dtype=np.float32) * np.float32(0.02))

    def fin(a):
        return round_to_bf16(a) if bf16 else np.ascontiguousarray(a, dtype=np.float32)

    w = {"wte": fin(normal(V, d)), "wpe": fin(normal(C, d)),
         "lnf_g": fin(1.0 + normal(d)), "lnf_b": fin(normal(d))}
    shapes = {"ln1_g": (d,), "ln1_b": (d,), "w_qkv": (3 * d, d), "b_qkv": (3 * d,),
              "w_o": (d, d), "b_o": (d,), "ln2_g": (d,), "ln2_b": (d,),
              "w_fc": (F, d), "b_fc": (F,), "w_proj": (d, F), "b_proj": (d,)}
    for name in _PER_LAYER:
        w[name] = []
    for _ in range(L):
        for name in _PER_LAYER:
            a = normal(*shapes[name])
            if name in ("ln1_g", "ln2_g"):
                a = a + np.float32(1.0)
            if name == "w_qkv" and qk_gain != 1.0:
                a[: 2 * d] *= np.float32(qk_gain)
            w[name].append(fin(a))
    return w


def bf16_bits(weights: dict) -> dict:
    """16-bit patterns of a bf16 model's tensors (same structure as the input)."""
    out = {}
    for k, v in weights.items():
        out[k] = [f32_to_bf16_bits(t) for t in v] if isinstance(v, list) else f32_to_bf16_bits(v)
    return out


def n_params(cfg: dict) -> int:
    L, d, F, V, C = cfg["n_layer"], cfg["d_model"], cfg["d_ff"], cfg["vocab"], cfg["n_ctx"]
    return L * (12 * d * d + 13 * d) + V * d + C * d + 2 * d if F == 4 * d else \
        L * (4 * d * d + 2 * d * F + 9 * d + F) + V * d + C * d + 2 * d


# ----------------------------------------------------------------------------
# Token trees.  parent_idx[0] = -1 (the root is the last emitted token) and
# 0 <= parent_idx[i] < i for every other node.
# ----------------------------------------------------------------------------
def tree_complete_binary(depth: int = 3) -> np.ndarray:
    n = 2 ** (depth + 1) - 1
    return np.array([-1] + [(i - 1) // 2 for i in range(1, n)], dtype=np.int32)


def tree_branching(n_nodes: int, branching=(4, 2, 2, 1, 1)) -> np.ndarray:
    """Breadth-first tree in which a node at depth k gets ``branching[k]`` children,
    truncated at ``n_nodes`` nodes."""
    parent, depth = [-1], [0]
    i = 0
    while i < len(parent) and len(parent) < n_nodes:
        k = branching[depth[i]] if depth[i] < len(branching) else 0
        for _ in range(k):
            if len(parent) < n_nodes:
                parent.append(i)
                depth.append(depth[i] + 1)
        i += 1
    if len(parent) != n_nodes:
        raise ValueError("branching rule yields only %d nodes" % len(parent))
    return np.array(parent, dtype=np.int32)


def tree_chain(n_nodes: int) -> np.ndarray:
    return np.arange(-1, n_nodes - 1, dtype=np.int32)


def tree_chain_plus_branch() -> np.ndarray:
    """Eight nodes: a chain 0-1-4-6-7 of first choices, second and third choices at
    depth 1 (nodes 2, 3) and a second choice at depth 2 (node 5)."""
    return np.array([-1, 0, 0, 0, 1, 1, 4, 6], dtype=np.int32)


def tree_random(n_nodes: int, max_depth: int, rng: np.random.Generator) -> np.ndarray:
    """Random parents with depth <= max_depth, then stably sorted by depth (BFS order)."""
    parent, depth = [-1], [0]
    for i in range(1, n_nodes):
        cand = [j for j in range(i) if depth[j] <= max_depth - 1]
        p = int(cand[rng.integers(len(cand))])
        parent.append(p)
        depth.append(depth[p] + 1)
    order = sorted(range(n_nodes), key=lambda j: (depth[j], j))
    new_of_old = {old: new for new, old in enumerate(order)}
    out = np.empty(n_nodes, dtype=np.int32)
    for new, old in enumerate(order):
        out[new] = -1 if parent[old] < 0 else new_of_old[parent[old]]
    return out


def tree_depths(parent_idx) -> np.ndarray:
    d = np.zeros(len(parent_idx), dtype=np.int32)
    for i in range(1, len(parent_idx)):
        d[i] = d[parent_idx[i]] + 1
    return d


def path_to(parent_idx, i: int) -> list:
    """Node indices from the root to node i, inclusive."""
    p = []
    while i >= 0:
        p.append(int(i))
        i = int(parent_idx[i])
    return p[::-1]


# ----------------------------------------------------------------------------
# Tokens and draft rows
# ----------------------------------------------------------------------------
def uniform_tokens(n: int, vocab: int, rng: np.random.Generator) -> np.ndarray:
    return rng.integers(0, vocab, size=n, dtype=np.int64).astype(np.int32)


def draft_rows_gamma(n_nodes: int, vocab: int, rng: np.random.Generator, alpha: float = 0.5) -> np.ndarray:
    """One Dirichlet(alpha) row per node (normalised Gamma(alpha) draws), fp32."""
    g = rng.standard_gamma(alpha, size=(n_nodes, vocab))
    g /= g.sum(axis=1, keepdims=True)
    return np.ascontiguousarray(g, dtype=np.float32)


def trigram_next(a: int, b: int, vocab: int, seed: int = 7, k: int = 4):
    """Synthetic trigram table entry: k distinct ids seeded by (a, b) with Zipf(1.1)
    weights (rank^-1.1, normalised).  Returns (ids int32[k], probs float32[k])."""
    rng = np.random.default_rng([seed, int(a), int(b)])
    ids = rng.choice(vocab, size=k, replace=False).astype(np.int32)
    wts = np.arange(1, k + 1, dtype=np.float64) ** -1.1
    return ids, (wts / wts.sum()).astype(np.float32)


def trigram_tree(prev2: int, prev1: int, root_token: int, vocab: int, seed: int = 7):
    """The eight-node chain-plus-branch tree filled from the synthetic trigram table.

    Returns (tokens int32[8], parent_idx int32[8], draft_rows float32[8, vocab]) where
    row c is the proposal distribution node c's own token was taken from with the
    earlier siblings removed and renormalised (row 0 is unused and uniform)."""
    parent = tree_chain_plus_branch()
    n = len(parent)
    tokens = np.zeros(n, dtype=np.int32)
    tokens[0] = root_token
    rows = np.zeros((n, vocab), dtype=np.float32)
    rows[0] = 1.0 / vocab
    # context of a node = the two tokens before its own position
    ctx = {0: (prev1, root_token)}
    children = {}
    for i in range(1, n):
        children.setdefault(int(parent[i]), []).append(i)
    for p in range(n):
        kids = children.get(p, [])
        if not kids:
            continue
        ids, pr = trigram_next(ctx[p][0], ctx[p][1], vocab, seed)
        remaining = pr.astype(np.float64).copy()
        for rank, c in enumerate(kids):
            tokens[c] = ids[rank]
            row = np.zeros(vocab, dtype=np.float64)
            row[ids] = remaining / remaining.sum()
            rows[c] = row.astype(np.float32)
            remaining[rank] = 0.0
            ctx[c] = (ctx[p][1], int(ids[rank]))
    return tokens, parent, rows


# ----------------------------------------------------------------------------
# Algorithmic bytes of one verify step (what the method has to move through HBM:
# every block weight and the LM head once, prefix K/V once per layer, tree K/V
# written once and read once, fp32 logits written once).
# ----------------------------------------------------------------------------
def algorithmic_bytes(cfg: dict, prefix: int, n_nodes: int) -> int:
    L, d, F, V = cfg["n_layer"], cfg["d_model"], cfg["d_ff"], cfg["vocab"]
    wb = 4 if cfg["dtype"] == "fp32" else 2
    mb = 1 if cfg["dtype"] == "bf16_w8" else wb          # bytes per matrix entry
    matrices = L * (4 * d * d + 2 * d * F) + V * d
    scales = 4 * (L * (5 * d + F) + V) if cfg["dtype"] == "bf16_w8" else 0   # one fp32 scale per output row
    weights = mb * matrices + scales + wb * L * (9 * d + F)
    kv = L * 2 * d * wb * (prefix + 2 * n_nodes)
    logits = 4 * n_nodes * V
    return weights + kv + logits
