"""GPU parity: the CUDA path against the CPU oracle on the same seeded inputs, through the C ABI."""
import numpy as np
import pytest
import torch

import ssd_synth
from oracle import ssd_oracle

pytestmark = pytest.mark.gpu

TOL_F32 = 1e-4   # fp32 configuration (stated target)
TOL_BF16 = 3e-2  # bf16 weights (stated target)


def forward_launches(n_layer, n, w8=False):
    """Kernels of one default-path bf16 forward: tree preparation, clearing of the logits, embedding; eight per layer - nine from 128
    nodes on, where a kernel of its own writes the tree's K / V rows to the cache; final LayerNorm and LM head."""
    return 3 + (8 + (1 if n >= 128 else 0)) * n_layer + 2


@pytest.fixture(scope="module")
def ssd():
    import paper_2308_04623_b200 as m
    return m


@pytest.fixture(scope="module")
def util():
    from tests import gpu_util
    return gpu_util


@pytest.fixture(scope="module")
def tiny(util):
    p = util.Pair("tiny", seed=0)
    yield p
    p.close()


@pytest.fixture(scope="module")
def sharp(util):
    p = util.Pair("tiny", seed=1, qk_gain=8.0)
    yield p
    p.close()


def reset(p):
    p.kv.reset()
    p.okv.reset()


# --------------------------------------------------------------------------- verify
@pytest.mark.parametrize("which", ["tiny", "sharp"])
def test_config1_binary_tree_logits(which, tiny, sharp):
    p = tiny if which == "tiny" else sharp
    reset(p)
    rng = np.random.default_rng(1001)
    prefix = ssd_synth.uniform_tokens(64, p.V, rng)
    parent = ssd_synth.tree_complete_binary(3)
    tokens = ssd_synth.uniform_tokens(len(parent), p.V, rng)
    p.prefill(prefix)
    got, want, _ = p.verify(tokens, parent)
    assert np.isfinite(got).all()
    assert np.abs(got - want).max() <= TOL_F32
    # scratch K/V rows of the batch equal the oracle's
    for l in range(p.cfg["n_layer"]):
        for which_kv in (0, 1):
            a = p.ctx.kv_read(p.kv, l, which_kv, 0, 64 + len(parent))
            b = p.okv.read(l, which_kv, 0, 64 + len(parent))
            assert np.abs(a - b).max() <= 1e-4


@pytest.mark.parametrize("shape", ["single", "chain", "star", "random40", "empty_prefix", "wide200", "max256"])
def test_tree_shapes_fp32(shape, sharp):
    p = sharp
    reset(p)
    rng = np.random.default_rng(hash(shape) % 1000)
    P = 0 if shape == "empty_prefix" else 37
    parent = {"single": np.array([-1], dtype=np.int32), "chain": ssd_synth.tree_chain(9),
              "star": np.array([-1] + [0] * 11, dtype=np.int32), "random40": ssd_synth.tree_random(40, 6, rng),
              "empty_prefix": ssd_synth.tree_branching(17, (4, 2, 1)), "wide200": ssd_synth.tree_random(200, 8, rng),
              "max256": ssd_synth.tree_random(256, 8, rng)}[shape]
    tokens = ssd_synth.uniform_tokens(len(parent), p.V, rng)
    p.prefill(ssd_synth.uniform_tokens(P, p.V, rng))
    got, want, _ = p.verify(tokens, parent)
    assert np.abs(got - want).max() <= TOL_F32


def test_verify_twice_overwrites_scratch_and_is_deterministic(sharp):
    p = sharp
    reset(p)
    rng = np.random.default_rng(5)
    p.prefill(ssd_synth.uniform_tokens(20, p.V, rng))
    parent = ssd_synth.tree_branching(12, (3, 2, 1))
    t1, t2 = ssd_synth.uniform_tokens(12, p.V, rng), ssd_synth.uniform_tokens(12, p.V, rng)
    a1, _, _ = p.verify(t1, parent)
    p.verify(t2, parent)
    a3, want, _ = p.verify(t1, parent)
    assert len(p.kv) == 20
    assert np.array_equal(a1, a3)
    assert np.abs(a3 - want).max() <= TOL_F32


@pytest.mark.parametrize("name", ["tiny_bf16", "ragged_bf16"])
def test_bf16_models_logits(name, util):
    p = util.Pair(name, seed=3)
    try:
        rng = np.random.default_rng(8)
        p.prefill(ssd_synth.uniform_tokens(70, p.V, rng))
        for n, br in ((32, (4, 2, 2, 1, 1)), (19, (3, 3, 1, 1)), (1, ())):
            parent = ssd_synth.tree_branching(n, br)
            tokens = ssd_synth.uniform_tokens(n, p.V, rng)
            got, want, _ = p.verify(tokens, parent)
            assert np.isfinite(got).all()
            assert np.abs(got - want).max() <= TOL_BF16
    finally:
        p.close()


# --------------------------------------------------------------------------- accept
def _accept_both(p, logits_np, draft_np, tokens, parent, mode, seed, step, temperature=1.0, top_k=0):
    import paper_2308_04623_b200 as ssd
    from tests import gpu_util
    lg = gpu_util.device_f32(logits_np)
    dp = gpu_util.device_f32(draft_np) if draft_np is not None else None
    rng = ssd.binding.ssd_rng(seed, step)
    T = float(np.float32(temperature))
    path, nxt = p.ctx.accept_tree(lg.data_ptr(), dp.data_ptr() if dp is not None else None, tokens, parent, mode=mode,
                                  temperature=T, top_k=top_k, rng=rng)
    assert rng.step == step + 1
    opath, onxt, margin = ssd_oracle.accept_tree(logits_np, draft_np, tokens, parent, mode=mode, temperature=T, top_k=top_k,
                                                 seed=seed, step=step, max_nodes=p.cfg["max_nodes"])
    return (path, nxt), (opath, onxt), margin


def test_config1_accept_on_oracle_logits_greedy_and_sampling(tiny):
    """The acceptance kernels are fed the ORACLE's logits, so both sides decide on identical inputs;
    paths, lengths and emitted tokens must then be bit-equal."""
    p = tiny
    reset(p)
    rng = np.random.default_rng(1001)
    prefix = ssd_synth.uniform_tokens(64, p.V, rng)
    parent = ssd_synth.tree_complete_binary(3)
    tokens = ssd_synth.uniform_tokens(len(parent), p.V, rng)
    p.okv.prefill(prefix)
    logits = p.okv.verify_tree(tokens, parent).astype(np.float32)
    draft = ssd_synth.draft_rows_gamma(len(parent), p.V, rng)
    got, want, _ = _accept_both(p, logits, None, tokens, parent, 0, 0, 0)
    assert got == want
    # make the greedy walk go deep: plant the arg-max tokens along a path
    tk = tokens.copy()
    for c in (1, 4, 9):
        tk[c] = int(np.argmax(logits[(c - 1) // 2]))
    got, want, _ = _accept_both(p, logits, None, tk, parent, 0, 0, 0)
    assert got == want and len(got[0]) >= 2
    fragile = 0
    for step in range(200):
        got, want, margin = _accept_both(p, logits, draft, tokens, parent, 1, 42, step)
        if got != want:
            assert margin < 1e-9, (step, got, want, margin)
            fragile += 1
    assert fragile == 0


def test_sampling_walk_goes_deep_and_matches(tiny):
    """Draft rows close to the target so that children are accepted and refusals update the residual."""
    p = tiny
    V = p.V
    rng = np.random.default_rng(77)
    parent = ssd_synth.tree_branching(24, (3, 2, 2, 1, 1))
    n = len(parent)
    logits = (rng.normal(size=(n, V)) * 2.5).astype(np.float32)
    probs = np.exp(logits.astype(np.float64))
    probs /= probs.sum(axis=1, keepdims=True)
    draft = np.zeros((n, V), dtype=np.float32)
    tokens = np.zeros(n, dtype=np.int32)
    for c in range(1, n):
        mix = 0.7 * probs[parent[c]] + 0.3 * rng.dirichlet(np.full(V, 0.5))
        draft[c] = mix.astype(np.float32)
        tokens[c] = rng.choice(V, p=mix / mix.sum())
    deep = fragile = 0
    for step in range(300):
        got, want, margin = _accept_both(p, logits, draft, tokens, parent, 1, 7, step)
        if got != want:
            assert margin < 1e-9, (step, got, want, margin)
            fragile += 1
        deep += len(want[0]) > 2
    assert deep > 20
    for step in range(100):  # top-k and temperature warp
        got, want, margin = _accept_both(p, logits, draft, tokens, parent, 1, 9, step, temperature=0.7, top_k=50)
        if got != want:
            assert margin < 1e-9, (step, got, want, margin)
            fragile += 1
    print("draws forgiven for a margin below 1e-9:", fragile)
    assert fragile == 0


def test_accept_special_rows(tiny):
    p = tiny
    V = p.V
    lg = np.zeros((3, V), dtype=np.float32)
    lg[0, [5, 900]] = 3.0  # tie: lowest index wins
    got, want, _ = _accept_both(p, lg, None, [0, 900, 5], [-1, 0, 0], 0, 0, 0)
    assert got == want == ([0, 2], 0)
    import paper_2308_04623_b200 as ssd
    bad = lg.copy()
    bad[0, 17] = np.nan
    from tests import gpu_util
    for mode, dp in ((0, None), (1, np.full((3, V), 1.0 / V, dtype=np.float32))):
        d = gpu_util.device_f32(bad)
        q = gpu_util.device_f32(dp) if dp is not None else None
        with pytest.raises(ssd.SsdError) as e:
            p.ctx.accept_tree(d.data_ptr(), q.data_ptr() if q is not None else None, [0, 1, 2], [-1, 0, 0], mode=mode)
        assert e.value.code == ssd.SSD_ERR_BAD_ARG


def test_sampling_at_a_large_vocabulary_star_tree_ties_and_long_support(ssd):
    """The sampling rule on hand-made logits at a 50257-word vocabulary (a context without weights is enough for
    acceptance): a star of 40 children (many refusals at one node), top-k cuts whose kept set is short, tied, and -
    with 3000 logits tied at the k-th value - longer than the support list the kernel keeps per row; rows that send the
    selection of the k-th largest down each of its paths; k = 1 and k = V - 1."""
    import torch
    cfg = ssd_synth.config("gpt2_small")
    V = cfg["vocab"]
    ctx = ssd.Context(cfg, device=0, stream=torch.cuda.current_stream().cuda_stream)
    try:
        rng = np.random.default_rng(2024)
        n = 41
        parent = np.array([-1] + [0] * 40, dtype=np.int32)
        tokens = np.concatenate([[7], rng.choice(V, size=40, replace=False)]).astype(np.int32)
        logits = rng.normal(0.0, 2.0, size=(n, V)).astype(np.float32)
        logits[0, tokens[1:]] += 4.0                     # the children are plausible, so several tests are close calls
        tied = logits.copy()
        tied[:, rng.choice(V, size=3000, replace=False)] = 9.0   # 3000 ties at the top: any k <= 3000 keeps them all
        draft = ssd_synth.draft_rows_gamma(n, V, rng)
        # the k-th largest is found by radix selection, whose first round looks at a logit's top 11 bits and whose later rounds
        # work on the logits sharing them if they are few: a row inside one quarter of a binade (all share them), and the same
        # row negated (the order of the bit patterns turns round below zero)
        narrow = rng.uniform(8.0, 9.99, size=(n, V)).astype(np.float32)
        narrow[0, tokens[1:]] = 9.995
        below = (-narrow).astype(np.float32)
        lg_dev, tied_dev, dp_dev, narrow_dev, below_dev = (torch.from_numpy(a).cuda() for a in (logits, tied, draft, narrow, below))
        fragile = 0
        for lg_np, lg_d, top_k in ((logits, lg_dev, 0), (logits, lg_dev, 50), (logits, lg_dev, 1000), (tied, tied_dev, 50), (tied, tied_dev, 0),
                                   (narrow, narrow_dev, 50), (narrow, narrow_dev, 5000), (below, below_dev, 50), (logits, lg_dev, 1), (logits, lg_dev, V - 1)):
            for step in range(3):
                srng = ssd.binding.ssd_rng(5, step)
                got = ctx.accept_tree(lg_d.data_ptr(), dp_dev.data_ptr(), tokens, parent, mode=ssd.SSD_SAMPLING, temperature=1.0,
                                      top_k=top_k, rng=srng)
                opath, onxt, margin = ssd_oracle.accept_tree(lg_np, draft, tokens, parent, mode=1, temperature=1.0, top_k=top_k,
                                                             seed=5, step=step, max_nodes=cfg["max_nodes"])
                if got != (opath, onxt):
                    assert margin < 1e-9, (top_k, step, margin)
                    fragile += 1
        print("draws forgiven for a margin below 1e-9:", fragile)
        assert fragile == 0
    finally:
        ctx.close()


# --------------------------------------------------------------------------- whole steps
def test_steps_verify_accept_commit_then_verify(sharp):
    """Several full steps: GPU logits -> GPU accept -> GPU commit; the oracle is driven with the same
    accepted paths; logits, paths and the committed cache agree at every step."""
    import paper_2308_04623_b200 as ssd
    p = sharp
    reset(p)
    rng = np.random.default_rng(31)
    p.prefill(ssd_synth.uniform_tokens(11, p.V, rng))
    root = int(rng.integers(p.V))
    srng = ssd.binding.ssd_rng(5, 0)
    accepted_any = False
    for step in range(6):
        parent = ssd_synth.tree_random(int(rng.integers(2, 30)), 5, rng)
        tokens = ssd_synth.uniform_tokens(len(parent), p.V, rng)
        tokens[0] = root
        got, want, buf = p.verify(tokens, parent)
        assert np.abs(got - want).max() <= TOL_F32
        # plant the verifier's favourite tokens on some children so the walk accepts
        if step % 2 == 0:
            for c in range(1, len(parent)):
                if rng.random() < 0.6:
                    tokens[c] = int(np.argmax(want[parent[c]]))
            got, want, buf = p.verify(tokens, parent)
        mode = ssd.SSD_GREEDY if step % 2 == 0 else ssd.SSD_SAMPLING
        draft = ssd_synth.draft_rows_gamma(len(parent), p.V, rng)
        from tests import gpu_util
        dp = gpu_util.device_f32(draft)
        st = srng.step
        path, nxt = p.ctx.accept_tree(buf.data_ptr(), dp.data_ptr(), tokens, parent, mode=mode, rng=srng)
        opath, onxt, margin = ssd_oracle.accept_tree(got.astype(np.float32), draft, tokens, parent, mode=mode, seed=5, step=st)
        assert (path, nxt) == (opath, onxt)
        accepted_any |= len(path) > 1
        before = len(p.kv)
        p.commit(path)
        assert len(p.kv) == len(p.okv) == before + len(path)
        for l in range(p.cfg["n_layer"]):
            for which_kv in (0, 1):
                a = p.ctx.kv_read(p.kv, l, which_kv, 0, len(p.kv))
                assert np.abs(a - p.okv.read(l, which_kv, 0, len(p.kv))).max() <= 1e-4
        root = nxt
    assert accepted_any


def test_commit_moves_exactly_the_path_rows(tiny):
    """Bit-exact gather: rows kv_len + path[j] land at kv_len + j, everything else below stays."""
    p = tiny
    reset(p)
    rng = np.random.default_rng(2)
    p.prefill(ssd_synth.uniform_tokens(5, p.V, rng))
    parent = ssd_synth.tree_complete_binary(3)
    p.verify(ssd_synth.uniform_tokens(15, p.V, rng), parent)
    L = p.cfg["n_layer"]
    before = [[p.ctx.kv_read(p.kv, l, w, 0, 5 + 15) for w in (0, 1)] for l in range(L)]
    path = [0, 2, 5, 12]
    p.commit(path)
    for l in range(L):
        for w in (0, 1):
            after = p.ctx.kv_read(p.kv, l, w, 0, 5 + len(path))
            assert np.array_equal(after[:5], before[l][w][:5])
            for j, c in enumerate(path):
                assert np.array_equal(after[5 + j], before[l][w][5 + c])


@pytest.mark.parametrize("path", [[0, 2, 5, 12], [0], [0, 1, 3, 7, 15, 31]])
def test_bf16_commit_moves_exactly_the_path_rows(path, util):
    """The same bit-exact gather on the bf16 cache, whose V is stored transposed and moved by a kernel of its own:
    K and V scratch rows are read before the commit and must sit, bit for bit, at their committed slots after it; the
    prefix rows stay as they were.  (An odd prefix length, so that pairs of transposed-V keys straddle slots.)"""
    p = util.Pair("ragged_bf16", seed=4)
    try:
        rng = np.random.default_rng(12)
        P = 37
        p.prefill(ssd_synth.uniform_tokens(P, p.V, rng), chunk=32)
        parent = ssd_synth.tree_complete_binary(5)  # 63 nodes; [0, 1, 3, 7, 15, 31] is its leftmost path
        n = len(parent)
        p.verify(ssd_synth.uniform_tokens(n, p.V, rng), parent)
        L = p.cfg["n_layer"]
        before = [[p.ctx.kv_read(p.kv, l, w, 0, P + n) for w in (0, 1)] for l in range(L)]
        p.commit(path)
        assert len(p.kv) == P + len(path)
        for l in range(L):
            for w in (0, 1):
                after = p.ctx.kv_read(p.kv, l, w, 0, P + len(path))
                assert np.array_equal(after[:P], before[l][w][:P])
                for j, c in enumerate(path):
                    assert np.array_equal(after[P + j], before[l][w][P + c]), (l, w, j, c)
                assert np.abs(after).max() > 0
    finally:
        p.close()


# --------------------------------------------------------------------------- errors
def test_error_codes_without_device_faults(tiny, ssd):
    p = tiny
    reset(p)
    buf = torch.empty((4, p.V), dtype=torch.float32, device="cuda")

    def code(fn):
        with pytest.raises(ssd.SsdError) as e:
            fn()
        return e.value.code

    assert code(lambda: p.ctx.verify_tree([1, 2], [0, 0], p.kv, buf.data_ptr())) == ssd.SSD_ERR_INVALID_TREE
    assert code(lambda: p.ctx.verify_tree([1, 2, 3], [-1, 2, 0], p.kv, buf.data_ptr())) == ssd.SSD_ERR_INVALID_TREE
    assert code(lambda: p.ctx.verify_tree([1, p.V], [-1, 0], p.kv, buf.data_ptr())) == ssd.SSD_ERR_BAD_ARG
    assert code(lambda: p.ctx.verify_tree([1, -1], [-1, 0], p.kv, buf.data_ptr())) == ssd.SSD_ERR_BAD_ARG
    assert code(lambda: p.ctx.verify_tree([], [], p.kv, buf.data_ptr())) == ssd.SSD_ERR_INVALID_TREE
    assert code(lambda: p.ctx.verify_tree([1] * 257, [-1] + list(range(256)), p.kv, buf.data_ptr())) == ssd.SSD_ERR_INVALID_TREE
    assert code(lambda: p.ctx.verify_tree([1], [-1], p.kv, 0)) == ssd.SSD_ERR_BAD_ARG
    assert code(lambda: p.ctx.kv_commit(p.kv, [0])) == ssd.SSD_ERR_BAD_PATH  # nothing verified yet
    p.ctx.verify_tree([1, 2, 3, 4], [-1, 0, 0, 1], p.kv, buf.data_ptr())
    for bad in ([1], [0, 3], [0, 2, 3], [0, 0]):
        assert code(lambda: p.ctx.kv_commit(p.kv, bad)) == ssd.SSD_ERR_BAD_PATH
    p.ctx.kv_commit(p.kv, [0, 1, 3])
    assert code(lambda: p.ctx.kv_commit(p.kv, [0])) == ssd.SSD_ERR_BAD_PATH  # one commit per verify
    assert code(lambda: p.kv.rollback(10)) == ssd.SSD_ERR_BAD_ARG
    # context overflow: a prefix that leaves no room for the tree's depth
    small = ssd.Context(ssd_synth.config("tiny", n_ctx=8))
    try:
        assert code(lambda: small.verify_tree([1], [-1], small.new_kv(), buf.data_ptr())) == ssd.SSD_ERR_NOT_LOADED
    finally:
        small.close()
    assert p.ctx.device_status() == 0


def test_context_overflow(util, ssd):
    p = util.Pair("tiny", seed=0, n_ctx=16)
    try:
        p.prefill(ssd_synth.uniform_tokens(12, p.V, np.random.default_rng(0)))
        buf = torch.empty((8, p.V), dtype=torch.float32, device="cuda")
        with pytest.raises(ssd.SsdError) as e:
            p.ctx.verify_tree([1] * 5, ssd_synth.tree_chain(5), p.kv, buf.data_ptr())  # 12 + 4 >= 16
        assert e.value.code == ssd.SSD_ERR_CTX_OVERFLOW
        with pytest.raises(ssd_oracle.OracleError) as e2:
            p.okv.verify_tree([1] * 5, ssd_synth.tree_chain(5))
        assert e2.value.code == ssd_oracle.ORC_CTX_OVERFLOW
        p.ctx.verify_tree([1] * 4, ssd_synth.tree_chain(4), p.kv, buf.data_ptr())
        p.ctx.kv_commit(p.kv, [0, 1, 2, 3])
        assert len(p.kv) == 16
    finally:
        p.close()


# --------------------------------------------------------------------------- bf16 tensor-core path, more shapes
@pytest.mark.parametrize("n", [1, 15, 16, 17, 48, 64, 100, 256])
def test_bf16_tree_sizes(n, util):
    """Tree sizes around the 16-row operand boxes and up to the maximum; chain prefill uses n = 64 too."""
    p = util.Pair("tiny_bf16", seed=5, qk_gain=4.0)
    try:
        rng = np.random.default_rng(n)
        p.prefill(ssd_synth.uniform_tokens(100, p.V, rng))
        parent = ssd_synth.tree_random(n, 8, rng)
        tokens = ssd_synth.uniform_tokens(n, p.V, rng)
        got, want, _ = p.verify(tokens, parent)
        assert np.isfinite(got).all()
        assert np.abs(got - want).max() <= TOL_BF16
        assert p.ctx.device_status() == 0
    finally:
        p.close()


@pytest.mark.parametrize("prefix", [0, 1, 15, 16, 17, 31, 143])
def test_bf16_prefix_lengths_around_key_blocks(prefix, util):
    """The attention kernel cuts the keys in blocks of 16 and keeps the partly filled last block of the prefix in shared
    memory with the tree's own keys: prefixes of every residue, the empty one included, with an odd tree size (so that
    the last pair of transposed V stores is a single key)."""
    p = util.Pair("ragged_bf16", seed=3, qk_gain=4.0)
    try:
        rng = np.random.default_rng(500 + prefix)
        if prefix:
            p.prefill(ssd_synth.uniform_tokens(prefix, p.V, rng), chunk=48)
        for n in (21, 32):
            parent = ssd_synth.tree_random(n, 6, rng)
            tokens = ssd_synth.uniform_tokens(n, p.V, rng)
            got, want, _ = p.verify(tokens, parent)
            assert np.isfinite(got).all()
            assert np.abs(got - want).max() <= TOL_BF16
        assert p.ctx.device_status() == 0
    finally:
        p.close()


def test_bf16_last_step_that_fits_the_context(util):
    """A tree verified and committed right up to the end of the context (ragged_bf16: 256 positions): the step whose
    commit fills the cache exactly, then the refusal of one more node."""
    import paper_2308_04623_b200 as ssd
    p = util.Pair("ragged_bf16", seed=6, qk_gain=3.0)
    try:
        rng = np.random.default_rng(77)
        n_ctx = p.cfg["n_ctx"]
        chain = 9
        p.prefill(ssd_synth.uniform_tokens(n_ctx - chain, p.V, rng), chunk=64)
        parent = ssd_synth.tree_chain(chain)
        tokens = ssd_synth.uniform_tokens(chain, p.V, rng)
        got, want, _ = p.verify(tokens, parent)
        assert np.abs(got - want).max() <= TOL_BF16
        p.commit(list(range(chain)))                      # the cache is now full
        with pytest.raises(ssd.SsdError) as e:
            p.verify(tokens[:1], parent[:1])
        assert e.value.code == ssd.SSD_ERR_CTX_OVERFLOW
        assert p.ctx.device_status() == 0
    finally:
        p.close()


def test_bf16_steps_with_commit(util):
    import paper_2308_04623_b200 as ssd
    p = util.Pair("ragged_bf16", seed=2)
    try:
        p.ctx.set_tuning(ssd.SSD_TUNE_HEAD_STATS, 1)  # (the LM head with complete sums and row statistics; the default head is tested everywhere else)
        rng = np.random.default_rng(3)
        p.prefill(ssd_synth.uniform_tokens(33, p.V, rng))
        root = 5
        for step in range(4):
            parent = ssd_synth.tree_random(int(rng.integers(3, 40)), 5, rng)
            tokens = ssd_synth.uniform_tokens(len(parent), p.V, rng)
            tokens[0] = root
            got, want, buf = p.verify(tokens, parent)
            assert np.abs(got - want).max() <= TOL_BF16
            for c in range(1, len(parent)):
                if rng.random() < 0.6:
                    tokens[c] = int(np.argmax(got[parent[c]]))
            got, want, buf = p.verify(tokens, parent)
            launches = p.ctx.kernel_launches()
            path, nxt = p.ctx.accept_tree(buf.data_ptr(), None, tokens, parent, mode=ssd.SSD_GREEDY)
            assert p.ctx.kernel_launches() - launches == 1    # the walk alone: the LM head left the rows' statistics per vocabulary tile
            opath, onxt, _ = ssd_oracle.accept_tree(got.astype(np.float32), None, tokens, parent, mode=0)
            assert (path, nxt) == (opath, onxt)
            other = buf.clone()                               # the same logits in another buffer: the arg-max pass runs, same result
            launches = p.ctx.kernel_launches()
            assert p.ctx.accept_tree(other.data_ptr(), None, tokens, parent, mode=ssd.SSD_GREEDY) == (path, nxt)
            assert p.ctx.kernel_launches() - launches == 2
            p.commit(path)
            root = nxt
            # committed rows: bf16 storage of the fp32 projections, compared with the oracle's exact rows
            for l in range(p.cfg["n_layer"]):
                for which_kv in (0, 1):
                    a = p.ctx.kv_read(p.kv, l, which_kv, 0, len(p.kv))
                    b = p.okv.read(l, which_kv, 0, len(p.kv))
                    assert np.abs(a - b).max() <= 3e-2
    finally:
        p.close()


# --------------------------------------------------------------------------- cluster-reduced projections, CTA counts
@pytest.mark.parametrize("name,n,cmax", [("tiny_bf16", 1, 8), ("tiny_bf16", 7, 1), ("tiny_bf16", 16, 2), ("tiny_bf16", 40, 8), ("ragged_bf16", 33, 3),
                                         ("tiny_bf16", 64, 4), ("ragged_bf16", 48, 5), ("tiny_bf16", 31, 16), ("ragged_bf16", 17, 7)])
def test_cluster_reduced_path_cluster_sizes_and_steps(name, n, cmax, util, ssd):
    """Five launches per layer: split-K partial sums reduced inside a thread-block cluster, LayerNorms folded, GELU and
    the residual additions in the epilogues.  Every cluster size (1 = no split, odd sizes with uneven column chunks, the
    non-portable 16) gives logits within the bf16 tolerance, bit-identical from run to run, over two committed steps; the
    launch count shows that the path ran; the 8-launch path gives the same logits within twice the tolerance's noise."""
    p = util.Pair(name, seed=9, qk_gain=3.0)
    try:
        p.ctx.set_tuning(ssd.SSD_TUNE_CLUSTER_REDUCE, 1)
        p.ctx.set_tuning(ssd.SSD_TUNE_CLUSTER_MAX, cmax)
        rng = np.random.default_rng(300 + n)
        p.prefill(ssd_synth.uniform_tokens(37, p.V, rng), chunk=32)
        for step in range(2):
            parent = ssd_synth.tree_random(n, 6, rng)
            tokens = ssd_synth.uniform_tokens(n, p.V, rng)
            before = p.ctx.kernel_launches()
            got, want, buf = p.verify(tokens, parent)
            assert p.ctx.kernel_launches() - before == 3 + 5 * p.cfg["n_layer"] + 2
            assert np.isfinite(got).all()
            assert np.abs(got - want).max() <= TOL_BF16
            if step == 0:
                again, _, _ = p.verify(tokens, parent)
                # the layers are reproducible bit for bit; the LM head still adds its stream-K partial sums at L2
                assert np.abs(again - got).max() <= 1e-5, np.abs(again - got).max()
                p.ctx.set_tuning(ssd.SSD_TUNE_CLUSTER_REDUCE, 0)
                before = p.ctx.kernel_launches()
                plain, _, _ = p.verify(tokens, parent)
                assert p.ctx.kernel_launches() - before == 3 + 8 * p.cfg["n_layer"] + 2
                assert np.abs(plain - want).max() <= TOL_BF16
                p.ctx.set_tuning(ssd.SSD_TUNE_CLUSTER_REDUCE, 1)
                got, want, buf = p.verify(tokens, parent)
            path, nxt = p.ctx.accept_tree(buf.data_ptr(), None, tokens, parent)
            p.commit(path)
            for l in range(p.cfg["n_layer"]):
                for which_kv in (0, 1):
                    a = p.ctx.kv_read(p.kv, l, which_kv, 0, len(p.kv))
                    assert np.abs(a - p.okv.read(l, which_kv, 0, len(p.kv))).max() <= 3e-2
        assert p.ctx.device_status() == 0
    finally:
        p.close()


@pytest.mark.parametrize("ctas", [1, 37, 148, 296, 500])
def test_projection_cta_counts_give_the_same_logits(ctas, util, ssd):
    """The (output tile, k tile) units of a projection are cut into one contiguous range per CTA, whatever the CTA
    count (one CTA, fewer CTAs than SMs, one or two per SM, more CTAs than units for the small matrices); on the
    cluster-reduced path the count bounds the clusters' sizes instead."""
    p = util.Pair("ragged_bf16", seed=4, qk_gain=3.0)
    try:
        p.ctx.set_tuning(ssd.SSD_TUNE_CLUSTER_REDUCE, ctas % 2)
        p.ctx.set_tuning(ssd.SSD_TUNE_GEMM_CTAS, ctas)
        p.ctx.set_tuning(ssd.SSD_TUNE_HEAD_CTAS, max(1, ctas // 2))
        rng = np.random.default_rng(77)
        p.prefill(ssd_synth.uniform_tokens(21, p.V, rng), chunk=16)
        parent = ssd_synth.tree_random(29, 5, rng)
        tokens = ssd_synth.uniform_tokens(29, p.V, rng)
        got, want, _ = p.verify(tokens, parent)
        assert np.abs(got - want).max() <= TOL_BF16
        assert p.ctx.device_status() == 0
    finally:
        p.close()


@pytest.mark.parametrize("name,n", [("ragged_bf16", 29), ("tiny_bf16", 100)])
def test_head_with_row_statistics_and_stream_k_head_give_the_same_logits(name, n, util, ssd):
    """SSD_TUNE_HEAD_STATS = 1: the LM head with complete sums per CTA (plain stores, no clearing launch, per-tile row
    maxima that the greedy walk reads instead of the logits) against the default stream-K head adding partial sums into
    cleared logits, greedy acceptance with its own arg-max pass; same logits within reduction-order noise, same paths."""
    p = util.Pair(name, seed=4, qk_gain=3.0)
    try:
        p.ctx.set_tuning(ssd.SSD_TUNE_HEAD_STATS, 1)
        rng = np.random.default_rng(5)
        p.prefill(ssd_synth.uniform_tokens(21, p.V, rng), chunk=16)
        parent = ssd_synth.tree_random(n, 5, rng)
        tokens = ssd_synth.uniform_tokens(n, p.V, rng)
        got, want, buf = p.verify(tokens, parent)
        assert np.abs(got - want).max() <= TOL_BF16
        before = p.ctx.kernel_launches()
        first = p.ctx.accept_tree(buf.data_ptr(), None, tokens, parent)
        assert p.ctx.kernel_launches() - before == 1
        p.ctx.set_tuning(ssd.SSD_TUNE_HEAD_STATS, 0)
        before = p.ctx.kernel_launches()
        plain, _, buf2 = p.verify(tokens, parent)
        assert p.ctx.kernel_launches() - before == forward_launches(p.cfg["n_layer"], n)
        assert np.abs(plain - got).max() <= 1e-3 and np.abs(plain - want).max() <= TOL_BF16
        before = p.ctx.kernel_launches()
        opath, onxt, _ = ssd_oracle.accept_tree(plain.astype(np.float32), None, tokens, parent, mode=0)
        assert p.ctx.accept_tree(buf2.data_ptr(), None, tokens, parent) == (opath, onxt)
        assert p.ctx.kernel_launches() - before == 2
        assert first == ssd_oracle.accept_tree(got.astype(np.float32), None, tokens, parent, mode=0)[:2]
        assert p.ctx.device_status() == 0
    finally:
        p.close()


def test_kernel_timeline_has_eight_ordered_stamps_per_launch(util, ssd):
    """SSD_TUNE_KERNEL_TRACE: eight values per kernel of the last forward; entry <= dependencies met <= end for every
    traced kernel, kernels in launch order, and the logits are unchanged by tracing (up to reduction order)."""
    p = util.Pair("tiny_bf16", seed=5, qk_gain=3.0)
    try:
        rng = np.random.default_rng(11)
        p.prefill(ssd_synth.uniform_tokens(19, p.V, rng), chunk=16)
        parent = ssd_synth.tree_random(21, 4, rng)
        tokens = ssd_synth.uniform_tokens(21, p.V, rng)
        base, want, _ = p.verify(tokens, parent)
        p.ctx.set_tuning(ssd.SSD_TUNE_KERNEL_TRACE, 1)
        before = p.ctx.kernel_launches()
        got, _, _ = p.verify(tokens, parent)
        kernels = p.ctx.kernel_launches() - before
        # (the order of the fp32 reductions at L2 differs from run to run, and a last-bit difference can move a query or a
        #  softmax weight across a bf16 rounding boundary inside the attention kernel)
        assert np.abs(got - base).max() <= 1e-3
        t = p.ctx.phase_trace().astype(np.int64)
        assert len(t) == 8 * kernels
        t = t.reshape(kernels, 8)[3:]          # (the three set-up kernels are not traced)
        assert (t[:, 0] > 0).all() and (t[:, 0] <= t[:, 1]).all() and (t[:, 1] <= t[:, 2]).all() and (t[:, 2] <= t[:, 6]).all()
        assert (np.diff(t[:, 1]) >= 0).all()   # dependencies are met in launch order
        p.ctx.set_tuning(ssd.SSD_TUNE_KERNEL_TRACE, 0)
        assert p.ctx.device_status() == 0
    finally:
        p.close()


# --------------------------------------------------------------------------- failure path (a wait that runs out, made safely)
def test_expired_device_wait_surfaces_as_timeout_and_can_be_reset(util, ssd):
    """A bounded device-side wait that expires must reach the caller: the test hook makes one warp wait 10 us on an
    mbarrier nobody arrives at (nothing else in flight), which records the error word.  The next accept returns
    SSD_ERR_TIMEOUT, a verify enqueued while the word is set leaves its projections undone, and after a reset the
    context computes the right logits again."""
    p = util.Pair("tiny_bf16", seed=5, qk_gain=3.0)
    try:
        rng = np.random.default_rng(21)
        p.prefill(ssd_synth.uniform_tokens(19, p.V, rng), chunk=16)
        parent = ssd_synth.tree_random(12, 4, rng)
        tokens = ssd_synth.uniform_tokens(12, p.V, rng)
        good, want, buf = p.verify(tokens, parent)
        assert np.abs(good - want).max() <= TOL_BF16 and p.ctx.device_status() == 0
        p.ctx.debug_expire_wait(10)
        assert p.ctx.device_status() == 0xE00
        with pytest.raises(ssd.SsdError) as e:
            p.ctx.accept_tree(buf.data_ptr(), None, tokens, parent)
        assert e.value.code == ssd.SSD_ERR_TIMEOUT
        stale = torch.full((12, p.V), 7.0, dtype=torch.float32, device="cuda")
        p.ctx.verify_tree(tokens, parent, p.kv, stale.data_ptr())   # projections are no-ops while the word is set
        torch.cuda.synchronize()
        assert float(stale.abs().max()) == 0.0                      # cleared at the start of the forward, never accumulated into
        assert p.ctx.device_status() == 0xE00
        p.ctx.reset_device_status()
        assert p.ctx.device_status() == 0
        again, _, buf = p.verify(tokens, parent)
        assert np.abs(again - want).max() <= TOL_BF16
        path, nxt = p.ctx.accept_tree(buf.data_ptr(), None, tokens, parent)
        opath, onxt, _ = ssd_oracle.accept_tree(again.astype(np.float32), None, tokens, parent, mode=0)
        assert (path, nxt) == (opath, onxt)
    finally:
        p.close()


# --------------------------------------------------------------------------- proposal rows as lists, proposals of a stage
def test_sparse_proposal_rows_give_the_dense_rule_on_the_trigram_tree(ssd):
    """ssd_accept_tree_sparse on the stage-two tree: the four-entry trigram rows and one-entry (deterministic) rows walk exactly
    as the oracle's dense rule does on the same rows written out densely, at the full vocabulary."""
    cfg = ssd_synth.config("gpt2_small")
    V = cfg["vocab"]
    ctx = ssd.Context(cfg, device=0, stream=torch.cuda.current_stream().cuda_stream)
    try:
        rng = np.random.default_rng(33)
        tokens, parent, dense = ssd_synth.trigram_tree(11, 22, 33, V)
        n = len(parent)
        logits = rng.normal(0.0, 1.5, size=(n, V)).astype(np.float32)
        for c in range(1, n):                       # make the proposed tokens plausible under the verifier
            logits[parent[c], tokens[c]] += 6.0
        idx = np.full((n, 4), -1, dtype=np.int32)
        val = np.zeros((n, 4), dtype=np.float32)
        for c in range(1, n):
            nz = np.nonzero(dense[c])[0]
            idx[c, :len(nz)], val[c, :len(nz)] = nz, dense[c, nz]
        onehot = np.zeros((n, V), dtype=np.float32)
        onehot[np.arange(1, n), tokens[1:]] = 1.0
        lg = torch.from_numpy(logits).cuda()
        deep = 0
        for step in range(40):
            for rows_dense, i_, v_ in ((dense, idx, val), (onehot, np.concatenate([[-1], tokens[1:]]).reshape(-1, 1), np.ones((n, 1), dtype=np.float32))):
                for top_k in (0, 50):
                    got = ctx.accept_tree_sparse(lg.data_ptr(), i_, v_, tokens, parent, mode=ssd.SSD_SAMPLING, top_k=top_k, rng=ssd.binding.ssd_rng(3, step))
                    opath, onxt, margin = ssd_oracle.accept_tree(logits, rows_dense, tokens, parent, mode=1, top_k=top_k, seed=3, step=step)
                    assert got == (opath, onxt), (step, top_k, margin)
                    deep += len(opath) > 1
        assert deep > 20
    finally:
        ctx.close()


def test_proposed_children_follow_the_nodes_laws(ssd):
    """ssd_propose_children: the rows are the nodes' target laws (fp64 softmax, temperature, top-k cut) to fp32 rounding, the
    deterministic picks are the most probable tokens in order, the sampled picks are the inverse-CDF draws of the same uniforms."""
    from oracle import staged_oracle
    cfg = ssd_synth.config("tiny", vocab=5000)
    V = cfg["vocab"]
    ctx = ssd.Context(cfg, device=0, stream=torch.cuda.current_stream().cuda_stream)
    try:
        rng = np.random.default_rng(8)
        logits = rng.normal(0.0, 2.0, size=(12, V)).astype(np.float32)
        logits[3, [7, 9]] = 11.0                         # a tie at the top: the lower id comes first
        lg = torch.from_numpy(logits).cuda()
        nodes = [0, 3, 11, 5]
        rows = torch.zeros((len(nodes), V), dtype=torch.float32, device="cuda")
        for T, k in ((1.0, 0), (0.7, 50)):
            srng = ssd.binding.ssd_rng(21, 4)
            got = ctx.propose_children(lg.data_ptr(), nodes, 4, mode=ssd.SSD_GREEDY, temperature=T, top_k=k, rng=srng, rows_out_ptr=rows.data_ptr())
            assert srng.step == 5
            r = rows.cpu().numpy()
            for j, node in enumerate(nodes):
                p = staged_oracle.law(logits[node], float(np.float32(T)), k)
                assert np.abs(r[j].astype(np.float64) - p).max() <= 1e-7 * max(1.0, p.max())
                assert got[j].tolist() == staged_oracle.most_probable(p, 4)
            assert got[1, :2].tolist() == [7, 9]
            got = ctx.propose_children(lg.data_ptr(), nodes, 8, mode=ssd.SSD_SAMPLING, temperature=T, top_k=k, rng=ssd.binding.ssd_rng(21, 9))
            for j, node in enumerate(nodes):
                p = staged_oracle.law(logits[node], float(np.float32(T)), k)
                assert got[j].tolist() == [staged_oracle.draw(p, ssd_oracle.uniform(21, 9, 1024 + 16 * node + t)) for t in range(8)]
        bad = lg.clone()
        bad[5, 100] = float("inf")
        with pytest.raises(ssd.SsdError) as e:
            ctx.propose_children(bad.data_ptr(), nodes, 2)
        assert e.value.code == ssd.SSD_ERR_BAD_ARG
    finally:
        ctx.close()


# ---------------------------------------------------------------------------
# 8-bit weight streaming (Section 4, closing list of next steps)
# ---------------------------------------------------------------------------
def test_w8_device_encoding_matches_the_oracle_encoding(ssd):
    """Arbitrary bf16 matrices: the codes and scales the library holds are, bit for bit, those of the encoding's definition."""
    from oracle import w8_oracle
    cfg = ssd_synth.config("ragged_bf16", dtype="bf16_w8")
    w = ssd_synth.make_weights(cfg, seed=21)
    w["w_fc"][1][5, :] = 0.0                     # a row of zeros
    w["w_o"][0][7, 3] = ssd_synth.round_to_bf16(np.float32([3.7]))[0]   # a row with one dominant entry: the others fall into the sub-normal codes
    ctx = ssd.Context(cfg, device=0, stream=torch.cuda.current_stream().cuda_stream)
    ctx.load_weights(ssd_synth.bf16_bits(w))
    for which, name in enumerate(w8_oracle.MATRICES):
        for l in range(cfg["n_layer"]):
            codes, scales = ctx.w8_read(which, l)
            want_c, want_s = w8_oracle.quantise_rows(w[name][l])
            assert np.array_equal(scales, want_s), (name, l)
            assert np.array_equal(codes & 0x7F, want_c & 0x7F) and np.array_equal((codes >> 7)[(codes & 0x7F) != 0], (want_c >> 7)[(want_c & 0x7F) != 0]), (name, l)
    codes, scales = ctx.w8_read(4)
    want_c, want_s = w8_oracle.quantise_rows(w["wte"])
    assert np.array_equal(scales, want_s) and np.array_equal(codes & 0x7F, want_c & 0x7F)
    sub = (codes & 0x7F) < 8
    assert sub.any()                              # sub-normal codes occur in these matrices
    # another dtype has nothing to read
    with pytest.raises(ssd.SsdError):
        ssd.Context(ssd_synth.config("ragged_bf16")).w8_read(0, 0)
    ctx.close()


@pytest.mark.parametrize("cfg_name,qk_gain", [("ragged_bf16", 1.0), ("tiny_bf16", 1.0), ("tiny_bf16", 4.0)])
def test_w8_logits_against_the_oracle_and_the_bf16_path(ssd, util, cfg_name, qk_gain):
    """The model on the code grid held three ways - by the oracle (fp64), by the library as bf16 and by the library as 8-bit
    codes: 8-bit against the oracle within the bf16 tolerance over trees that span the single- and two-instruction operand
    layouts and ragged tails, with commits in between; 8-bit against bf16 to summation-order noise (same numbers, same
    products; only the order of the fp32 additions differs); same number of launches."""
    rng = np.random.default_rng(31)
    # (qk_gain > 1: sharpened attention, so that a wrong key, mask or plane shows in the logits)
    p8 = util.Pair(cfg_name, seed=4, qk_gain=qk_gain, on_grid=True, dtype="bf16_w8")
    p16 = util.Pair(cfg_name, seed=4, qk_gain=qk_gain, on_grid=True)
    V = p8.V
    prefix = ssd_synth.uniform_tokens(70, V, rng)
    p8.prefill(prefix); p16.prefill(prefix)
    L = p8.cfg["n_layer"]
    for n in (1, 5, 29, 64, 100, 256):
        par = ssd_synth.tree_random(n, 8, rng)
        tok = ssd_synth.uniform_tokens(n, V, rng)
        before = p8.ctx.kernel_launches()
        got8, want, buf8 = p8.verify(tok, par)
        assert p8.ctx.kernel_launches() - before == forward_launches(L, n, w8=True)
        got16, _, _ = p16.verify(tok, par)
        assert np.isfinite(got8).all()
        assert np.abs(got8 - want).max() <= TOL_BF16, n
        # (sharpened attention magnifies a last-bit difference that moves a K / V value across a bf16 rounding boundary of the cache)
        assert np.abs(got8 - got16).max() <= (1e-3 if qk_gain == 1.0 else 5e-3), n
        path, nxt = p8.ctx.accept_tree(buf8.data_ptr(), None, tok, par)
        opath, onext, margin = ssd_oracle.accept_tree(want.astype(np.float32), None, tok, par)
        if margin > 4 * TOL_BF16:
            assert list(path) == list(opath) and nxt == onext
        p8.commit(opath[:3]); p16.commit(opath[:3])
    assert p8.ctx.device_status() == 0
    p8.close(); p16.close()


@pytest.mark.parametrize("ctas", [1, 2, 5])
def test_w8_with_few_ctas_gives_the_same_logits(ssd, util, ctas):
    """With few CTAs each one streams many (output tile, k tile) units through its stage ring and runs several epilogues over
    its accumulator buffers (at full size only the LM head does): same logits as the oracle, over several steps."""
    rng = np.random.default_rng(41 + ctas)
    p8 = util.Pair("ragged_bf16", seed=6, on_grid=True, dtype="bf16_w8")
    p8.ctx.set_tuning(ssd.SSD_TUNE_GEMM_CTAS, ctas)
    p8.ctx.set_tuning(ssd.SSD_TUNE_HEAD_CTAS, ctas)
    V = p8.V
    p8.prefill(ssd_synth.uniform_tokens(37, V, rng))
    for n in (3, 40, 130):
        par = ssd_synth.tree_random(n, 6, rng)
        tok = ssd_synth.uniform_tokens(n, V, rng)
        got8, want, _ = p8.verify(tok, par)
        assert np.abs(got8 - want).max() <= TOL_BF16, (ctas, n)
        p8.commit([0])
    assert p8.ctx.device_status() == 0
    p8.close()


def test_w8_plane_count(ssd, util):
    """Three of the four activation planes (12 significant bits) still meet the bf16 tolerance; two (what a single bf16 plane
    carries) stay finite and close; the knob belongs to 8-bit contexts only."""
    rng = np.random.default_rng(51)
    p8 = util.Pair("tiny_bf16", seed=8, on_grid=True, dtype="bf16_w8")
    V = p8.V
    p8.prefill(ssd_synth.uniform_tokens(50, V, rng))
    par = ssd_synth.tree_random(48, 6, rng)
    tok = ssd_synth.uniform_tokens(48, V, rng)
    errs = {}
    for planes in (4, 3, 2):
        p8.ctx.set_tuning(ssd.SSD_TUNE_W8_PLANES, planes)
        got, want, _ = p8.verify(tok, par)
        errs[planes] = np.abs(got - want).max()
    assert errs[4] <= TOL_BF16 and errs[3] <= TOL_BF16 and errs[2] <= 4 * TOL_BF16 and errs[4] <= errs[2]
    for bad in (1, 5):
        with pytest.raises(ssd.SsdError):
            p8.ctx.set_tuning(ssd.SSD_TUNE_W8_PLANES, bad)
    p8.close()
    p16 = util.Pair("tiny_bf16", seed=8)
    with pytest.raises(ssd.SsdError):
        p16.ctx.set_tuning(ssd.SSD_TUNE_W8_PLANES, 3)
    p16.close()


@pytest.mark.parametrize("prefix,warps", [(0, 4), (5, 8), (16, 4), (37, 8), (37, 4), (16, 8)])
def test_tree_rows_read_from_the_cache_give_the_same_logits(ssd, util, prefix, warps):
    """Large trees: a kernel of its own writes the tree's K / V rows to the cache's scratch slots (and zeroes the rest of the last
    16-key block) and the attention reads every block from the cache.  Against the oracle and against the path in which every
    node tile stages the tree's keys itself, for prefixes that end on and off a 16-key boundary, with commits in between (the
    scratch rows then become committed ones); forcing the path on a small tree covers the case of a single partial block.  Both
    shapes of the cache-reading CTA: four warps, and eight (the choice depends on how many (head, tile) items the GPU holds)."""
    rng = np.random.default_rng(61 + prefix)
    p = util.Pair("ragged_bf16", seed=3, qk_gain=3.0)
    p.ctx.set_tuning(ssd.SSD_TUNE_ATTN_STAGED_WARPS, warps)
    V, L = p.V, p.cfg["n_layer"]
    if prefix:
        p.prefill(ssd_synth.uniform_tokens(prefix, V, rng))
    for n in (70, 131, 256, 9):
        par = ssd_synth.tree_random(n, 7, rng)
        tok = ssd_synth.uniform_tokens(n, V, rng)
        p.ctx.set_tuning(ssd.SSD_TUNE_STAGE_KV_FROM, 1)
        before = p.ctx.kernel_launches()
        got, want, _ = p.verify(tok, par)
        assert p.ctx.kernel_launches() - before == 3 + 9 * L + 2
        p.ctx.set_tuning(ssd.SSD_TUNE_STAGE_KV_FROM, 0)
        before = p.ctx.kernel_launches()
        plain, _, _ = p.verify(tok, par)
        assert p.ctx.kernel_launches() - before == 3 + 8 * L + 2
        assert np.abs(got - want).max() <= TOL_BF16, (prefix, n)
        assert np.abs(got - plain).max() <= 1e-3, (prefix, n)
        path = ssd_synth.path_to(par, int(rng.integers(0, n)))
        p.commit(path)
    assert p.ctx.device_status() == 0
    p.close()


@pytest.mark.parametrize("splits", [2, 4])
def test_attention_key_splits_merged_in_a_cluster(ssd, util, splits):
    """Several CTAs - one thread-block cluster - share a (head, node tile), each with a part of the key blocks, merged in the first
    one's shared memory.  Forced on short prefixes too (some splits then hold no block at all, or only masked keys) and compared with
    the oracle and with the single-CTA path; commits in between check that the tree's K / V rows still reach the cache (the
    last split of tile 0 writes them); then with the split count chosen from the prefix length."""
    rng = np.random.default_rng(71 + splits)
    p = util.Pair("ragged_bf16", seed=5, qk_gain=3.0)
    V, L = p.V, p.cfg["n_layer"]
    for prefix_add, n in ((0, 1), (3, 9), (13, 40), (16, 64), (60, 21), (90, 100)):
        par = ssd_synth.tree_random(n, 6, rng)
        tok = ssd_synth.uniform_tokens(n, V, rng)
        p.ctx.set_tuning(ssd.SSD_TUNE_ATTN_SPLITS, splits)
        got, want, _ = p.verify(tok, par)
        p.ctx.set_tuning(ssd.SSD_TUNE_ATTN_SPLITS, 1)
        plain, _, _ = p.verify(tok, par)
        assert np.isfinite(got).all()
        assert np.abs(got - want).max() <= TOL_BF16, (splits, n)
        assert np.abs(got - plain).max() <= 2e-3, (splits, n)
        p.ctx.set_tuning(ssd.SSD_TUNE_ATTN_SPLITS, splits)
        got2, _, _ = p.verify(tok, par)                      # (the scratch rows the commit below moves come from this forward)
        path = ssd_synth.path_to(par, int(rng.integers(0, n)))
        p.commit(path)
        extra = int(prefix_add)
        for _ in range(extra):                                  # grow the prefix one committed root at a time, splits still forced
            t1 = ssd_synth.uniform_tokens(1, V, rng)
            p.verify(t1, np.array([-1], dtype=np.int32))
            p.commit([0])
    p.ctx.set_tuning(ssd.SSD_TUNE_ATTN_SPLITS, 0)
    assert len(p.kv) > 150                                      # long enough for the automatic choice to split
    par = ssd_synth.tree_random(12, 5, rng)
    tok = ssd_synth.uniform_tokens(12, V, rng)
    got, want, _ = p.verify(tok, par)
    assert np.abs(got - want).max() <= TOL_BF16
    assert p.ctx.device_status() == 0
    p.close()


def test_back_projection_applies_the_gelu_itself(ssd, util):
    """SSD_TUNE_FUSED_GELU = 1: the feed-forward block's back-projection reads the first projection's fp32 sums and writes its
    gelu(.) hi / lo operand planes into shared memory itself, against the default, a separate element-wise kernel (same arithmetic,
    so the logits differ by the order of the fp32 reductions only), and against the oracle; one launch fewer per layer where it
    applies (at most 64 rows per CTA: trees of up to 64 nodes, node groups beyond 128).  Tree sizes with one to four 16-row chunks
    per thread, ragged ones, and node groups with a ragged last group."""
    rng = np.random.default_rng(97)
    p = util.Pair("ragged_bf16", seed=9, qk_gain=3.0)
    V, L = p.V, p.cfg["n_layer"]
    p.prefill(ssd_synth.uniform_tokens(23, V, rng))
    for n in (1, 16, 17, 33, 48, 64, 100, 150, 256):
        par = ssd_synth.tree_random(n, 5, rng)
        tok = ssd_synth.uniform_tokens(n, V, rng)
        p.ctx.set_tuning(ssd.SSD_TUNE_FUSED_GELU, 0)
        before = p.ctx.kernel_launches()
        plain, want, _ = p.verify(tok, par)
        separate = p.ctx.kernel_launches() - before
        p.ctx.set_tuning(ssd.SSD_TUNE_FUSED_GELU, 1)
        before = p.ctx.kernel_launches()
        got, _, _ = p.verify(tok, par)
        assert separate == forward_launches(L, n) and p.ctx.kernel_launches() - before == separate - (0 if 64 < n <= 128 else L), n
        assert np.isfinite(got).all()
        assert np.abs(got - want).max() <= TOL_BF16, n
        assert np.abs(got - plain).max() <= 1e-3, n
        p.commit(ssd_synth.path_to(par, n - 1))
    # without the low plane the projection keeps reading prepared planes
    p.ctx.set_tuning(ssd.SSD_TUNE_LOW_PLANE, 0)
    before = p.ctx.kernel_launches()
    p.verify(tok[:20], ssd_synth.tree_random(20, 5, rng))
    assert p.ctx.kernel_launches() - before == forward_launches(L, 20)
    assert p.ctx.device_status() == 0
    p.close()


def test_projections_on_node_groups_give_the_same_logits(ssd, util):
    """Trees of more than 128 nodes: the layers' projections run as one copy of a 64-node CTA arrangement per group of 64 nodes
    (ragged last group included).  Against the oracle and against the whole-batch projections, with a commit in between."""
    rng = np.random.default_rng(83)
    p = util.Pair("ragged_bf16", seed=7, qk_gain=3.0)
    V = p.V
    p.prefill(ssd_synth.uniform_tokens(19, V, rng))
    for n in (129, 200, 256, 193):
        par = ssd_synth.tree_random(n, 7, rng)
        tok = ssd_synth.uniform_tokens(n, V, rng)
        p.ctx.set_tuning(ssd.SSD_TUNE_NODE_GROUPS, 1)
        got, want, _ = p.verify(tok, par)
        p.ctx.set_tuning(ssd.SSD_TUNE_NODE_GROUPS, 0)
        plain, _, _ = p.verify(tok, par)
        assert np.isfinite(got).all()
        assert np.abs(got - want).max() <= TOL_BF16, n
        assert np.abs(got - plain).max() <= 2e-3, n
        p.ctx.set_tuning(ssd.SSD_TUNE_NODE_GROUPS, 1)
        p.verify(tok, par)
        p.commit(ssd_synth.path_to(par, n - 1))
    assert p.ctx.device_status() == 0
    p.close()
