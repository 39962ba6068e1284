"""The Katz back-off trigram stage: pins of the CPU oracle (no GPU) and parity of the CUDA table and lookup kernels."""
from fractions import Fraction as Fr

import numpy as np
import pytest

import ssd_synth
from oracle.trigram_oracle import DISCOUNT, KatzTrigram


def zipf_stream(n, vocab, seed):
    """A token stream with repeated structure: a first-order chain whose rows are Zipf-weighted over a few successors."""
    rng = np.random.default_rng(seed)
    succ = rng.integers(0, vocab, size=(vocab, 6))
    w = np.arange(1, 7, dtype=np.float64) ** -1.1
    w /= w.sum()
    out = np.zeros(n, dtype=np.int32)
    out[0] = rng.integers(vocab)
    for i in range(1, n):
        out[i] = succ[out[i - 1], rng.choice(6, p=w)] if rng.random() < 0.9 else rng.integers(vocab)
    return out


# ------------------------------------------------------------------------------------------ oracle pins (CPU)
def test_hand_counted_corpus_closed_form_probabilities():
    """Stream 0 1 2 0 1 3 0 1 2 over a vocabulary of 5, every value worked out by hand with rationals.
    c1 = (3, 3, 2, 1, 0), N = 9.  After (0, 1): token 2 twice, token 3 once.  After 1: 2 twice, 3 once."""
    m = KatzTrigram([0, 1, 2, 0, 1, 3, 0, 1, 2], vocab=5)
    D = Fr(1, 2)
    p1 = [Fr(3, 9), Fr(3, 9), Fr(2, 9), Fr(1, 9), Fr(0)]
    assert np.allclose(m.p1(), [float(x) for x in p1], atol=0, rtol=1e-15)
    # bigram level after 1: seen {2: 2, 3: 1}, total 3
    a2 = (D * 2 / 3) / (1 - (p1[2] + p1[3]))
    p2 = [a2 * p1[0], a2 * p1[1], (2 - D) / 3, (1 - D) / 3, a2 * p1[4]]
    assert sum(p2) == 1
    assert np.allclose(m.p2(1), [float(x) for x in p2], atol=1e-15)
    # trigram level after (0, 1): the same seen set; unseen tokens back off to the bigram level
    a3 = (D * 2 / 3) / (1 - (p2[2] + p2[3]))
    p3 = [a3 * p2[0], a3 * p2[1], (2 - D) / 3, (1 - D) / 3, a3 * p2[4]]
    assert sum(p3) == 1
    assert np.allclose(m.p3(0, 1), [float(x) for x in p3], atol=1e-15)
    ids, pr = m.top_next(0, 1)
    assert ids.tolist() == [2, 3, 0, 1]              # 1/2, 1/6, then the tie between tokens 0 and 1 goes to the lower id
    assert np.allclose(pr, [0.5, 1 / 6, float(p3[0]), float(p3[1])], atol=1e-15)
    # a context never seen backs off entirely; a token never seen as a context backs off to the unigram law
    assert np.array_equal(m.p3(4, 1), m.p2(1))
    assert np.array_equal(m.p3(1, 4), m.p1())
    assert m.top_next(3, 4)[0].tolist() == [0, 1, 2, 3]


@pytest.mark.parametrize("seed", [0, 1])
def test_every_level_is_a_probability_law(seed):
    s = zipf_stream(3000, 40, seed)
    m = KatzTrigram(s, 40)
    rng = np.random.default_rng(seed)
    for _ in range(40):
        i = int(rng.integers(2, len(s)))
        for a, b in ((s[i - 2], s[i - 1]), (int(rng.integers(40)), s[i - 1]), (s[i - 2], int(rng.integers(40)))):
            p = m.p3(int(a), int(b))
            assert abs(p.sum() - 1.0) < 1e-12 and (p >= 0).all()
    # the discounted probabilities of seen continuations are below their relative frequencies by exactly D / total
    a, b = int(s[10]), int(s[11])
    seen = m.c3[(a, b)]
    tot = sum(seen.values())
    p = m.p3(a, b)
    for w, c in seen.items():
        assert abs(p[w] - (c - DISCOUNT) / tot) < 1e-15


def test_proposal_tree_follows_the_best_continuations():
    s = zipf_stream(4000, 30, 3)
    m = KatzTrigram(s, 30)
    parent = ssd_synth.tree_chain_plus_branch()
    tok, pr = m.propose_tree(int(s[100]), int(s[101]), parent)
    ids, p = m.top_next(int(s[100]), int(s[101]))
    assert tok[0] == s[101] and tok[1:4].tolist() == ids[:3].tolist()    # nodes 1, 2, 3: first, second, third continuation
    ids2, _ = m.top_next(int(tok[0]), int(tok[1]))
    assert tok[4:6].tolist() == ids2[:2].tolist()                        # nodes 4, 5 hang off node 1
    assert np.allclose(pr[1:4], p[:3])


# ------------------------------------------------------------------------------------------ GPU parity
@pytest.mark.gpu
@pytest.mark.parametrize("vocab,n", [(50, 5000), (1000, 60000), (50257, 40000)])
def test_device_table_answers_equal_the_oracle(vocab, n):
    import paper_2308_04623_b200 as ssd
    s = zipf_stream(n, vocab, 11)
    m = KatzTrigram(s, vocab)
    t = ssd.Trigram(s, vocab)
    try:
        assert t.contexts() == len(m.c3)
        rng = np.random.default_rng(5)
        ctx = []
        for _ in range(60 if vocab > 2000 else 200):                     # (the oracle ranks the whole vocabulary per query)
            i = int(rng.integers(2, n))
            ctx += [(s[i - 2], s[i - 1]), (int(rng.integers(vocab)), s[i - 1]), (s[i - 2], int(rng.integers(vocab)))]
        ctx.append((vocab - 1, vocab - 1))
        tok, pr = t.lookup(np.asarray(ctx, dtype=np.int32))
        for q, (a, b) in enumerate(ctx):
            ids, p = m.top_next(int(a), int(b))
            assert tok[q].tolist() == ids.tolist(), (q, a, b)            # integer results: exact
            assert np.abs(pr[q].astype(np.float64) - p).max() <= 1e-7    # fp32 storage of the fp64 values
        parent = ssd_synth.tree_chain_plus_branch()
        for i in (2, 77, n - 1):
            gt, gp = t.propose(int(s[i - 1]), int(s[i]), parent)
            ot, op = m.propose_tree(int(s[i - 1]), int(s[i]), parent)
            assert gt.tolist() == ot.tolist()
            assert np.abs(gp.astype(np.float64) - op).max() <= 1e-7
        with pytest.raises(ssd.SsdError) as e:
            t.propose(1, 2, np.array([-1, 0, 0, 0, 0, 0], dtype=np.int32))   # five children: more than a context stores
        assert e.value.code == ssd.SSD_ERR_INVALID_TREE
    finally:
        t.close()
