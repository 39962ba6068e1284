"""The full staged loop (oracle <- draft <- trigram): pins of the CPU loop, and the device loop against it."""
import numpy as np
import pytest

import ssd_synth
from oracle import ssd_oracle, staged_oracle
from oracle.trigram_oracle import KatzTrigram


def models(draft_same=False):
    cfg0 = ssd_synth.config("tiny")
    w0 = ssd_synth.make_weights(cfg0, seed=0, qk_gain=4.0)
    cfg1 = cfg0 if draft_same else ssd_synth.config("tiny", n_layer=2)
    w1 = w0 if draft_same else ssd_synth.make_weights(cfg1, seed=5, qk_gain=4.0)
    return (cfg0, w0), (cfg1, w1)


def draft_stream(cfg1, w1, prompt, n):
    """A token stream for the trigram table: the draft's own greedy continuation (so that the table often proposes what
    the draft would emit) followed by uniform noise."""
    m1 = ssd_oracle.Model(cfg1, w1)
    out = list(prompt) + staged_oracle.greedy_autoregressive(m1, prompt, n)
    rng = np.random.default_rng(3)
    return np.asarray(out + rng.integers(0, cfg1["vocab"], size=200).tolist(), dtype=np.int32)


PROMPT = [5, 17, 400, 9, 33, 801, 2]


def test_law_is_the_acceptance_rules_target():
    """A child proposed from q = law(z) with q <= p everywhere is never refused: u q[x] < p[x] for every u < 1.  So the law used
    for proposal rows is the target law of the C acceptance rule (temperature and top-k cut included)."""
    rng = np.random.default_rng(0)
    z = (rng.normal(size=(2, 64)) * 3).astype(np.float32)
    for T, k in ((1.0, 0), (0.7, 0), (1.0, 5), (1.3, 17)):
        q = staged_oracle.law(z[0], T, k)
        assert abs(q.sum() - 1) < 1e-12 and (np.count_nonzero(q) == (k or 64))
        rows = np.zeros((2, 64), dtype=np.float64)
        rows[1] = q * (1 - 1e-9)                      # just below the target everywhere
        for x in np.nonzero(q)[0][:8]:
            for step in range(40):
                path, _, _ = ssd_oracle.accept_tree(z, rows.astype(np.float32), [0, int(x)], [-1, 0], mode=1, temperature=T, top_k=k, seed=1, step=step)
                assert path == [0, 1]
    assert staged_oracle.most_probable(np.array([0.2, 0.3, 0.3, 0.2]), 3) == [1, 2, 0]
    assert staged_oracle.draw(np.array([0.0, 0.5, 0.0, 0.5]), 0.49) == 1 and staged_oracle.draw(np.array([0.0, 0.5, 0.0, 0.5]), 0.5) == 3


@pytest.mark.parametrize("draft_same,n_tokens", [(False, 256), (True, 96)])
def test_greedy_staged_decoding_equals_greedy_autoregressive_decoding(draft_same, n_tokens):
    """Deterministic staged decoding emits exactly the oracle model's greedy continuation, whatever the trigram table and
    the draft propose: 256 tokens with an unrelated draft (few acceptances), and with the oracle as its own draft (every
    chain accepted, the two-token stem of the next step exercised)."""
    (cfg0, w0), (cfg1, w1) = models(draft_same)
    tri = KatzTrigram(draft_stream(cfg1, w1, PROMPT, 300), cfg0["vocab"])
    loop = staged_oracle.StagedOracle(ssd_oracle.Model(cfg0, w0), ssd_oracle.Model(cfg1, w1), tri, mode=0, rounds=2, siblings=1)
    loop.prefill(PROMPT)
    got = loop.generate(n_tokens)
    want = staged_oracle.greedy_autoregressive(ssd_oracle.Model(cfg0, w0), PROMPT, n_tokens)
    assert got == want
    st = loop.stats
    assert st["emitted"] >= n_tokens and st["draft_forwards"] == 2 * st["target_steps"]
    assert sum(st["origin"].values()) == st["emitted"] and st["origin"]["target"] == st["target_steps"]
    if draft_same:   # the draft is the oracle: every chain token is accepted, several tokens per step
        assert st["emitted"] / st["target_steps"] >= 3.0 and st["origin"]["trigram"] > 0 and st["origin"]["draft"] > 0
    assert len(loop.kv0) == len(loop.seq) - 1 and 1 <= len(loop.seq) - len(loop.kv1) <= 2


def test_sampled_staged_decoding_is_reproducible_and_keeps_both_caches_consistent():
    (cfg0, w0), (cfg1, w1) = models(True)
    tri = KatzTrigram(draft_stream(cfg1, w1, PROMPT, 200), cfg0["vocab"])
    runs = []
    for _ in range(2):
        loop = staged_oracle.StagedOracle(ssd_oracle.Model(cfg0, w0), ssd_oracle.Model(cfg1, w1), tri, mode=1, temperature=0.8, top_k=20, rounds=2,
                                          siblings=2, seed=11)
        loop.prefill(PROMPT)
        runs.append(loop.generate(60))
        assert all(0 <= t < cfg0["vocab"] for t in runs[-1])
        assert loop.stats["emitted"] / loop.stats["target_steps"] > 1.2      # the oracle as its own draft: chains are accepted under sampling too
        # the oracle's cache equals the cache of decoding the emitted sequence token by token
        ref = ssd_oracle.Model(cfg0, w0).new_kv()
        ref.prefill(np.asarray(loop.seq[:-1], dtype=np.int32), chunk=64)
        for l in range(cfg0["n_layer"]):
            assert np.abs(loop.kv0.read(l, 0, 0, len(ref)) - ref.read(l, 0, 0, len(ref))).max() <= 1e-9
    assert runs[0] == runs[1]


# ------------------------------------------------------------------------------------------ device loop
@pytest.mark.gpu
@pytest.mark.parametrize("mode,draft_same", [(0, False), (0, True), (1, True), (1, False)])
def test_device_loop_emits_the_oracle_loops_tokens(mode, draft_same):
    """The same loop through the C ABI (fp32 models, so logits agree to 1e-6): the same tokens as the CPU loop under
    deterministic decoding, and under sampling with the same seed - both sides draw the same counter-based uniforms."""
    import torch
    import paper_2308_04623_b200 as ssd
    from paper_2308_04623_b200.staged import StagedDecoder
    (cfg0, w0), (cfg1, w1) = models(draft_same)
    stream = draft_stream(cfg1, w1, PROMPT, 300)
    kw = dict(mode=mode, temperature=0.8 if mode else 1.0, top_k=20 if mode else 0, rounds=2, siblings=2 if mode else 1, seed=7)
    cpu = staged_oracle.StagedOracle(ssd_oracle.Model(cfg0, w0), ssd_oracle.Model(cfg1, w1), KatzTrigram(stream, cfg0["vocab"]), **kw)
    cpu.prefill(PROMPT)
    stream_h = torch.cuda.current_stream().cuda_stream
    c0, c1 = ssd.Context(cfg0, device=0, stream=stream_h), ssd.Context(cfg1, device=0, stream=stream_h)
    c0.load_weights(w0)
    c1.load_weights(w1)
    tri = ssd.Trigram(stream, cfg0["vocab"], stream=stream_h)
    gpu = StagedDecoder(c0, c1, tri, **kw)
    try:
        gpu.prefill(PROMPT)
        n = 120 if mode == 0 else 80
        want = cpu.generate(n)
        got = gpu.generate(n)
        if got != want:   # a decision closer to its threshold than the two sides' logits agree may fall either way
            assert cpu.min_margin < 1e-5, (cpu.min_margin, got[:20], want[:20])
            pytest.fail("fragile draw (margin %.3g): choose another seed" % cpu.min_margin)
        assert gpu.stats == cpu.stats
        assert c0.device_status() == 0 and c1.device_status() == 0
    finally:
        gpu.close()
        tri.close()
        c0.close()
        c1.close()
