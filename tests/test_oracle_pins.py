"""Pins of the CPU oracle's transformer, tree batch and cache (no GPU).

Each test ties the oracle to something other than its own formulas: brute-force
sequential decoding, torch's library routines, a published known-answer set, or
an invariant the paper states (speculation leaves the output unchanged).
"""
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import ssd_synth
from oracle import ssd_oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------------------
# Philox4x32-10 against its published known-answer vectors
# ---------------------------------------------------------------------------
def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) if not l.startswith("#") and l.strip()]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        assert list(ssd_oracle.philox4x32_10(v[0:4], v[4:6])) == v[6:10]


def test_uniform_is_24_bit_fraction_of_first_word():
    out = ssd_oracle.philox4x32_10([5, 0, 12, 0], [99, 0])
    assert ssd_oracle.uniform(99, 5, 12) == float(int(out[0]) >> 8) / 2 ** 24
    # 64-bit seed and step are split low word first
    out = ssd_oracle.philox4x32_10([1, 2, 3, 0], [4, 5])
    assert ssd_oracle.uniform(4 + (5 << 32), 1 + (2 << 32), 3) == float(int(out[0]) >> 8) / 2 ** 24


# ---------------------------------------------------------------------------
# The GPT-2 block against torch's library routines (fp64)
# ---------------------------------------------------------------------------
def torch_gpt2_logits(cfg, w, seq):
    """Plain GPT-2 forward built only from torch library ops; all positions."""
    t = lambda a: torch.from_numpy(np.asarray(a)).double()
    T, d, H, dh = len(seq), cfg["d_model"], cfg["n_head"], cfg["d_head"]
    ids = torch.as_tensor(np.asarray(seq), dtype=torch.long)
    x = F.embedding(ids, t(w["wte"])) + F.embedding(torch.arange(T), t(w["wpe"]))
    for l in range(cfg["n_layer"]):
        a = F.layer_norm(x, (d,), t(w["ln1_g"][l]), t(w["ln1_b"][l]), cfg["ln_eps"])
        q, k, v = F.linear(a, t(w["w_qkv"][l]), t(w["b_qkv"][l])).split(d, dim=-1)
        sh = lambda z: z.view(T, H, dh).transpose(0, 1)
        o = F.scaled_dot_product_attention(sh(q), sh(k), sh(v), is_causal=True)
        x = x + F.linear(o.transpose(0, 1).reshape(T, d), t(w["w_o"][l]), t(w["b_o"][l]))
        m = F.layer_norm(x, (d,), t(w["ln2_g"][l]), t(w["ln2_b"][l]), cfg["ln_eps"])
        h = F.gelu(F.linear(m, t(w["w_fc"][l]), t(w["b_fc"][l])), approximate="tanh")
        x = x + F.linear(h, t(w["w_proj"][l]), t(w["b_proj"][l]))
    x = F.layer_norm(x, (d,), t(w["lnf_g"]), t(w["lnf_b"]), cfg["ln_eps"])
    return F.linear(x, t(w["wte"])).numpy()


@pytest.mark.parametrize("which", ["tiny", "sharp"])
def test_sequential_logits_match_torch_library_ops(which, tiny_model, sharp_model):
    cfg, w, model = tiny_model if which == "tiny" else sharp_model
    seq = ssd_synth.uniform_tokens(23, cfg["vocab"], np.random.default_rng(11))
    ref = torch_gpt2_logits(cfg, w, seq)
    got = model.sequential_logits(seq, all_positions=True)
    assert np.abs(got - ref).max() < 1e-10
    assert np.abs(model.sequential_logits(seq) - ref[-1]).max() < 1e-10
    # the sharpened model's logits do depend on order (a mask/position slip would show)
    if which == "sharp":
        swapped = seq.copy()
        swapped[[3, 4]] = swapped[[4, 3]]
        assert np.abs(model.sequential_logits(swapped) - ref[-1]).max() > 1e-3


# ---------------------------------------------------------------------------
# Tree batch == sequential decoding of every root-to-node path
# ---------------------------------------------------------------------------
def _check_tree_against_sequential(cfg, model, prefix, tokens, parent, tol=1e-9, chunk=64):
    kv = model.new_kv()
    kv.prefill(prefix, chunk=chunk)
    assert len(kv) == len(prefix)
    logits = kv.verify_tree(tokens, parent)
    assert len(kv) == len(prefix)  # verify leaves the committed length alone
    worst = 0.0
    for i in range(len(tokens)):
        nodes = ssd_synth.path_to(parent, i)
        seq = np.concatenate([prefix, tokens[nodes]]).astype(np.int32)
        worst = max(worst, np.abs(logits[i] - model.sequential_logits(seq)).max())
    assert worst < tol, worst
    return kv, logits


@pytest.mark.parametrize("which", ["tiny", "sharp"])
def test_binary_tree_equals_sequential(which, tiny_model, sharp_model):
    cfg, w, model = tiny_model if which == "tiny" else sharp_model
    rng = np.random.default_rng(1001)
    prefix = ssd_synth.uniform_tokens(64, cfg["vocab"], rng)
    parent = ssd_synth.tree_complete_binary(3)
    tokens = ssd_synth.uniform_tokens(len(parent), cfg["vocab"], rng)
    _check_tree_against_sequential(cfg, model, prefix, tokens, parent)


def test_sharp_model_detects_wrong_mask_or_position(sharp_model):
    """Sanity of the pin itself: on the sharpened model, siblings' logits differ and a
    node's logits differ from those of the same token one level up."""
    cfg, w, model = sharp_model
    rng = np.random.default_rng(5)
    prefix = ssd_synth.uniform_tokens(16, cfg["vocab"], rng)
    parent = np.array([-1, 0, 0, 1], dtype=np.int32)
    tokens = ssd_synth.uniform_tokens(4, cfg["vocab"], rng)
    tokens[3] = tokens[2]  # same token at depth 1 (node 2) and depth 2 (node 3)
    kv = model.new_kv()
    kv.prefill(prefix)
    lg = kv.verify_tree(tokens, parent)
    assert np.abs(lg[2] - lg[3]).max() > 1e-3


@pytest.mark.parametrize("shape", ["random", "chain", "star", "empty_prefix"])
def test_other_trees_equal_sequential(shape, sharp_model):
    cfg, w, model = sharp_model
    rng = np.random.default_rng(77)
    prefix = ssd_synth.uniform_tokens(0 if shape == "empty_prefix" else 9, cfg["vocab"], rng)
    parent = {"random": ssd_synth.tree_random(12, 4, rng), "chain": ssd_synth.tree_chain(6),
              "star": np.array([-1, 0, 0, 0, 0, 0], dtype=np.int32),
              "empty_prefix": ssd_synth.tree_branching(7, (2, 2))}[shape]
    tokens = ssd_synth.uniform_tokens(len(parent), cfg["vocab"], rng)
    _check_tree_against_sequential(cfg, model, prefix, tokens, parent)


def test_single_node_tree_is_a_plain_decode_step(tiny_model):
    cfg, w, model = tiny_model
    rng = np.random.default_rng(3)
    seq = ssd_synth.uniform_tokens(12, cfg["vocab"], rng)
    kv = model.new_kv()
    ref = torch_gpt2_logits(cfg, w, seq)
    for i, tok in enumerate(seq):  # token-by-token decoding with the cache
        lg = kv.verify_tree([tok], [-1])
        kv.commit([0])
        assert np.abs(lg[0] - ref[i]).max() < 1e-10
    assert len(kv) == len(seq)


# ---------------------------------------------------------------------------
# Commit: the cache after accepting a path equals the cache of sequential decoding
# ---------------------------------------------------------------------------
def test_commit_equals_sequential_cache(sharp_model):
    cfg, w, model = sharp_model
    rng = np.random.default_rng(21)
    prefix = ssd_synth.uniform_tokens(10, cfg["vocab"], rng)
    parent = ssd_synth.tree_complete_binary(3)
    tokens = ssd_synth.uniform_tokens(len(parent), cfg["vocab"], rng)
    path = [0, 2, 5, 12]
    kv = model.new_kv()
    kv.prefill(prefix)
    kv.verify_tree(tokens, parent)
    kv.commit(path)
    assert len(kv) == len(prefix) + len(path)
    ref = model.new_kv()  # sequential: one token at a time
    for tok in np.concatenate([prefix, tokens[path]]):
        ref.verify_tree([tok], [-1])
        ref.commit([0])
    for l in range(cfg["n_layer"]):
        for which in (0, 1):
            a, b = kv.read(l, which, 0, len(kv)), ref.read(l, which, 0, len(ref))
            assert np.abs(a - b).max() < 1e-10
    # and the next step sees exactly the sequential state
    nxt = ssd_synth.uniform_tokens(3, cfg["vocab"], rng)
    lg = kv.verify_tree(nxt, [-1, 0, 0])
    seq = np.concatenate([prefix, tokens[path], nxt[[0, 2]]]).astype(np.int32)
    assert np.abs(lg[2] - model.sequential_logits(seq)).max() < 1e-9


def test_commit_rejects_non_paths(tiny_model):
    cfg, w, model = tiny_model
    kv = model.new_kv()
    kv.verify_tree([1, 2, 3, 4], [-1, 0, 0, 1])
    for bad in ([1], [0, 3], [0, 2, 3], [0, 1, 2], [0, 0]):
        with pytest.raises(ssd_oracle.OracleError) as e:
            kv.commit(bad)
        assert e.value.code == ssd_oracle.ORC_BAD_PATH
    kv.commit([0, 1, 3])
    with pytest.raises(ssd_oracle.OracleError):  # a second commit without a new verify
        kv.commit([0])


def test_invalid_trees_are_refused(tiny_model):
    cfg, w, model = tiny_model
    kv = model.new_kv()
    for toks, par, code in (([1, 2], [0, 0], ssd_oracle.ORC_INVALID_TREE), ([1, 2], [-1, 1], ssd_oracle.ORC_INVALID_TREE),
                            ([1, 2, 3], [-1, 2, 0], ssd_oracle.ORC_INVALID_TREE), ([1, cfg["vocab"]], [-1, 0], ssd_oracle.ORC_BAD_ARG),
                            ([], [], ssd_oracle.ORC_INVALID_TREE)):
        with pytest.raises(ssd_oracle.OracleError) as e:
            kv.verify_tree(toks, par)
        assert e.value.code == code


# ---------------------------------------------------------------------------
# Greedy staged decoding emits exactly the tokens of greedy autoregressive decoding
# ---------------------------------------------------------------------------
def test_greedy_tree_decoding_equals_autoregressive(tiny_model):
    cfg, w, model = tiny_model
    rng = np.random.default_rng(2024)
    V, n_new = cfg["vocab"], 48
    prompt = ssd_synth.uniform_tokens(8, V, rng)
    # reference: plain greedy decoding from scratch
    seq = list(prompt)
    for _ in range(n_new):
        seq.append(int(np.argmax(model.sequential_logits(np.array(seq, dtype=np.int32)))))
    want = seq[len(prompt):]
    # staged: trees whose nodes sometimes carry the right continuation (a proposer of
    # mixed quality: the true next tokens with probability 0.7, otherwise random ids)
    kv = model.new_kv()
    kv.prefill(prompt[:-1])
    root, got, steps = int(prompt[-1]), [], 0
    while len(got) < n_new:
        parent = ssd_synth.tree_random(int(rng.integers(1, 10)), 4, rng)
        tokens = ssd_synth.uniform_tokens(len(parent), V, rng)
        tokens[0] = root
        depth = ssd_synth.tree_depths(parent)
        for i in range(1, len(parent)):
            k = len(got) + depth[i] - 1
            if k < n_new and rng.random() < 0.7:
                tokens[i] = want[k]
        logits = kv.verify_tree(tokens, parent)
        path, nxt, _ = ssd_oracle.accept_tree(logits, None, tokens, parent, mode=0)
        kv.commit(path)
        got.extend(int(tokens[c]) for c in path[1:])
        got.append(nxt)
        root = nxt
        steps += 1
    assert got[:n_new] == want
    assert steps < n_new  # speculation did accept something


# ---------------------------------------------------------------------------
# 8-bit weight encoding (e4m3 codes + per-row power-of-two scale)
# ---------------------------------------------------------------------------
def test_e4m3_table_landmarks():
    """The code table against the format's published landmarks: 0x38 = 1, 0x7e = 448 (largest), 0x08 = 2^-6 (smallest
    normal), 0x01 = 2^-9 (smallest sub-normal), 0x7f not a number, 126 positive values strictly ascending, sign symmetric."""
    from oracle import w8_oracle
    v = w8_oracle.code_values()
    assert v[0x00] == 0.0 and v[0x38] == 1.0 and v[0x7E] == 448.0 and v[0x08] == 2.0 ** -6 and v[0x01] == 2.0 ** -9
    assert v[0x40] == 2.0 and v[0x3C] == 1.5 and v[0x07] == 7 * 2.0 ** -9
    assert np.isnan(v[0x7F]) and np.isnan(v[0xFF])
    assert np.all(np.diff(v[:127]) > 0)
    assert np.array_equal(v[128:255], -v[0:127])


def test_e4m3_encode_ties_saturation_and_grid():
    from oracle import w8_oracle
    enc, v = w8_oracle.encode, w8_oracle.code_values()
    # ties go to the even pattern: 1.0625 lies between 1.0 (0x38) and 1.125 (0x39); 1.1875 between 0x39 and 1.25 (0x3a)
    assert list(enc([1.0625, 1.1875, -1.0625, -1.1875])) == [0x38, 0x3A, 0xB8, 0xBA]
    # across an exponent boundary: 1.9375 is halfway between 1.875 (0x3f) and 2.0 (0x40)
    assert list(enc([1.9375])) == [0x40]
    # sub-normal ties: 2^-10 is halfway between 0 and 2^-9 -> 0; 3 * 2^-10 halfway between codes 1 and 2 -> 2
    assert list(enc([2.0 ** -10, 3 * 2.0 ** -10])) == [0x00, 0x02]
    assert list(enc([1e9, -1e9, 448.0, 464.0, 0.0])) == [0x7E, 0xFE, 0x7E, 0x7E, 0x00]
    # every finite code encodes to itself
    codes = np.array([c for c in range(256) if c not in (0x7F, 0xFF, 0x80)], dtype=np.uint8)
    assert np.array_equal(enc(v[codes]), codes)


def test_e4m3_encode_matches_torch_cast_in_range():
    """A library routine as the pin: torch's float8_e4m3fn cast rounds to nearest even too (in range; it does not saturate)."""
    from oracle import w8_oracle
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.standard_normal(20000) * s for s in (1e-3, 0.05, 1.0, 30.0, 150.0)]).astype(np.float32)
    x = x[np.abs(x) <= 448.0]
    want = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = w8_oracle.encode(x.astype(np.float64))
    same = (got == want) | ((x == 0) & ((got & 0x7F) == 0) & ((want & 0x7F) == 0))
    assert same.all()


def test_w8_row_scale_rule_and_error_bound():
    from oracle import w8_oracle
    w = np.zeros((6, 8), dtype=np.float32)
    w[0, 3] = 448.0; w[1, 0] = -449.0; w[2, 7] = 224.0; w[3, 1] = 224.5; w[5, 2] = 0.02
    s = w8_oracle.row_scales(w)
    assert list(s[:5]) == [1.0, 2.0, 0.5, 1.0, 1.0]           # (row 4 is all zeros)
    assert s[5] == 2.0 ** -14 and 0.02 <= 448 * s[5] and 0.02 > 448 * s[5] / 2
    # decode(encode(w)) differs from w by at most half a code step: relative 2^-4 in the normal range, absolute
    # scale * 2^-10 below it
    rng = np.random.default_rng(11)
    W = (rng.standard_normal((64, 512)) * 0.02).astype(np.float32)
    q, sc = w8_oracle.quantise_rows(W)
    D = w8_oracle.dequantise_rows(q, sc)
    err = np.abs(D.astype(np.float64) - W)
    bound = np.maximum(np.abs(W) * 2.0 ** -4, sc[:, None].astype(np.float64) * 2.0 ** -10)
    assert (err <= bound).all()
    assert (np.abs(q.astype(np.int32) & 0x7F).max(axis=1) >= 0x70).all()   # every row uses the top octave of the format
    # on its own grid the encoding is lossless, whatever scale the second pass picks
    q2, sc2 = w8_oracle.quantise_rows(D)
    assert np.array_equal(w8_oracle.dequantise_rows(q2, sc2), D)
    # and the grid values are bf16 numbers
    assert np.array_equal(ssd_synth.round_to_bf16(D), D)


def test_four_e4m3_planes_carry_sixteen_bits():
    """The operand format of the 8-bit projections, restated with the oracle's encoder: p0 = rn(x / 16), p1 = rn(x - 16 p0),
    p2 = rn(16 r2), p3 = rn(256 r3) give x = 16 p0 + p1 + p2 / 16 + p3 / 256 to 2^-17 relative or 2^-18 absolute, whichever is
    larger, for |x| up to 7168; three planes to 2^-13 / 2^-14; two to 2^-9 / 2^-10."""
    from oracle import w8_oracle
    val = w8_oracle.code_values()
    rn = lambda a: val[w8_oracle.encode(a)]
    rng = np.random.default_rng(3)
    x = np.concatenate([rng.standard_normal(50000) * s for s in (1e-4, 1e-2, 1.0, 40.0, 2000.0)])
    x = x[np.abs(x) <= 7168.0]
    p0 = rn(x / 16); r1 = x - 16 * p0
    p1 = rn(r1); r2 = r1 - p1
    p2 = rn(16 * r2); r3 = r2 - p2 / 16
    p3 = rn(256 * r3)
    for planes, approx, rel, ab in ((4, 16 * p0 + p1 + p2 / 16 + p3 / 256, 2.0 ** -17, 2.0 ** -18),
                                    (3, 16 * p0 + p1 + p2 / 16, 2.0 ** -13, 2.0 ** -14), (2, 16 * p0 + p1, 2.0 ** -9, 2.0 ** -10)):
        err = np.abs(approx - x)
        assert (err <= np.maximum(rel * np.abs(x), ab)).all(), planes
