"""Full-size parity at the benchmark's configurations (GPU + CPU oracle on the same seeded inputs).

These are the shapes bench.py times: the GPT-2-Large-shaped verifier with a 256-token prefix and
the 32-node tree, the GPT-2-small-shaped draft verified in the second stage with a 512-token prefix
and the eight-node trigram tree, and a GPT-2-XL-shaped case.  The whole logits matrix is compared.
"""
import numpy as np
import pytest
import torch

import ssd_synth
from oracle import ssd_oracle

pytestmark = pytest.mark.gpu
TOL_BF16 = 3e-2


def _run(name, P, trees, seed=0, chunk=256, **pair_args):
    from tests import gpu_util
    import paper_2308_04623_b200 as ssd
    p = gpu_util.Pair(name, seed=seed, **pair_args)
    worst = {}
    fragile = 0
    try:
        rng = np.random.default_rng(1002)
        p.prefill(ssd_synth.uniform_tokens(P, p.V, rng), chunk=chunk)
        for label, tokens, parent in trees(p, rng):
            got, want, buf = p.verify(tokens, parent)
            assert np.isfinite(got).all(), label
            err = float(np.abs(got - want).max())
            worst[label] = err
            assert err <= TOL_BF16, (label, err)
            # greedy acceptance on the GPU's own logits, compared with the oracle's walk on the same logits
            path, nxt = p.ctx.accept_tree(buf.data_ptr(), None, tokens, parent)
            opath, onxt, _ = ssd_oracle.accept_tree(got.astype(np.float32), None, tokens, parent, mode=0)
            assert (path, nxt) == (opath, onxt), label
            # sampling acceptance at the full vocabulary (dense rule, then with the top-k cut), same logits on both sides
            draft = ssd_synth.draft_rows_gamma(len(tokens), p.V, rng)
            dbuf = torch.from_numpy(draft).cuda()
            for top_k in (0, 50):
                srng = ssd.binding.ssd_rng(11, 5)
                path, nxt = p.ctx.accept_tree(buf.data_ptr(), dbuf.data_ptr(), tokens, parent, mode=ssd.SSD_SAMPLING, temperature=1.0,
                                              top_k=top_k, rng=srng)
                opath, onxt, margin = ssd_oracle.accept_tree(got.astype(np.float32), draft, tokens, parent, mode=1, temperature=1.0,
                                                             top_k=top_k, seed=11, step=5)
                if (path, nxt) != (opath, onxt):
                    assert margin < 1e-9, (label, top_k, margin)
                    fragile += 1
            # the same with proposal rows as four-entry lists (what a trigram stage hands over): the kernels read the lists, the
            # oracle the dense rows they stand for; several steps, so that chains of refusals occur
            n = len(tokens)
            idx = np.argsort(-draft, axis=1)[:, :4].astype(np.int32)
            idx[1:, 0] = tokens[1:]                      # (the proposed token is in its row's list, as a real proposal's is)
            for c in range(1, n):                        # distinct indices per row
                seen = set()
                for e in range(4):
                    while int(idx[c, e]) in seen:
                        idx[c, e] = (idx[c, e] + 1) % p.V
                    seen.add(int(idx[c, e]))
            val = rng.dirichlet(np.ones(4), size=n).astype(np.float32)
            dense = np.zeros((n, p.V), dtype=np.float32)
            np.put_along_axis(dense, idx.astype(np.int64), val, axis=1)
            for step in range(6):
                for top_k in (0, 50):
                    srng = ssd.binding.ssd_rng(23, step)
                    path, nxt = p.ctx.accept_tree_sparse(buf.data_ptr(), idx, val, tokens, parent, mode=ssd.SSD_SAMPLING, temperature=1.0,
                                                         top_k=top_k, rng=srng)
                    opath, onxt, margin = ssd_oracle.accept_tree(got.astype(np.float32), dense, tokens, parent, mode=1, temperature=1.0,
                                                                 top_k=top_k, seed=23, step=step)
                    if (path, nxt) != (opath, onxt):
                        assert margin < 1e-9, (label, "lists", top_k, step, margin)
                        fragile += 1
        print("draws forgiven for a margin below 1e-9:", fragile)
        assert fragile == 0
        assert p.ctx.device_status() == 0
    finally:
        p.close()
    print(name, worst)
    return worst


def test_gpt2_large_shape_256_prefix_trees_16_32_64():
    def trees(p, rng):
        for n, br in ((32, (4, 2, 2, 1, 1)), (16, (4, 2, 2, 1, 1)), (64, (4, 2, 2, 2, 1, 1))):
            yield "n=%d" % n, ssd_synth.uniform_tokens(n, p.V, rng), ssd_synth.tree_branching(n, br)
    _run("gpt2_large", 256, trees)


def test_gpt2_small_shape_stage_two_trigram_tree():
    def trees(p, rng):
        tokens, parent, rows = ssd_synth.trigram_tree(11, 22, 33, p.V)
        yield "trigram8", tokens, parent
        yield "n=32", ssd_synth.uniform_tokens(32, p.V, rng), ssd_synth.tree_branching(32)
    _run("gpt2_small", 512, trees)


def test_gpt2_xl_shape_random_trees():
    def trees(p, rng):
        for n in (8, 128):
            yield "n=%d" % n, ssd_synth.uniform_tokens(n, p.V, rng), ssd_synth.tree_random(n, 8, rng)
    _run("gpt2_xl", 128, trees, chunk=128)


def test_gpt2_large_shape_8bit_weights():
    """The benchmark's shape with the streamed matrices as 8-bit codes (model on the code grid, so that the oracle holds the same
    numbers): the 32-node tree bench.py times and a 160-node tree, whose projections run on node groups of 64."""
    def trees(p, rng):
        yield "n=32", ssd_synth.uniform_tokens(32, p.V, rng), ssd_synth.tree_branching(32, (4, 2, 2, 1, 1))
        yield "n=160", ssd_synth.uniform_tokens(160, p.V, rng), ssd_synth.tree_random(160, 8, rng)
    _run("gpt2_large", 256, trees, on_grid=True, dtype="bf16_w8")
