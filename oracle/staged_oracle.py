"""CPU oracle of the full staged decoding loop (test infrastructure; only tests and the benchmark's CPU leg import it).

Section 3 of the paper in the order it states it.  Three models: the oracle M0, a small draft M1 and a
trigram model M2 (Section 4).  One step of the loop:

  stage 2 -> 1 (Section 3.2, "speculatively decode the draft model, too"), `rounds` times:
      M2 proposes a small tree below the last token the draft has not cached; M1 scores the whole tree in ONE
      tree-batched forward (Section 3.1) and the acceptance rule (Section 2.3) walks it with M1 as the verifier.
      The accepted tokens and the extra token M1 emits at the stop node continue the draft's chain; under
      sampling they are distributed exactly as draws from M1's own law (that is what the rule guarantees), so
      M1's law at a chain token's parent is that token's proposal row for the next stage.  The draft appends the
      accepted slices to its cache speculatively.
  stage 1 -> 0 (Section 3.1): the oracle's tree is the draft's chain plus, at every level, `siblings` extra
      leaves from the same law of M1 - its next most likely tokens ("the second or third most likely tokens")
      when decoding deterministically, independent draws when sampling.  Leaves cost no draft forward.  M0
      scores the tree in one forward, the rule walks it, the accepted slices are appended to M0's cache, and
      M1's cache is rolled back to the tokens both models have accepted.

The paper leaves open: the trigram's tree (the eight-node chain-plus-branch tree of the stage-two
configuration is used), its proposal rows (its proposals are its most probable continuations, so each row
is one-hot on the proposed token: the rule then accepts x iff u < r[x]), the number of rounds and of
siblings, and the uniform generator (the counter-based one of the acceptance oracle; every call of the
rule or of a sibling draw takes the next value of a step counter, in program order).

Deterministic decoding must emit exactly the oracle's greedy continuation whatever the lower stages
propose (Sections 1, 2.3); a test pins that for 256 tokens.
"""
from __future__ import annotations

import numpy as np

from oracle import ssd_oracle

TRI_PARENT = np.array([-1, 0, 0, 0, 1, 1, 4, 6], dtype=np.int32)  # chain 0-1-4-6-7, second / third choices at depth 1, second at depth 2


def law(z, temperature: float = 1.0, top_k: int = 0) -> np.ndarray:
    """Next-token law of a node: softmax(z / T) over the entries whose logit is >= the k-th largest (ties kept)."""
    z = np.asarray(z, dtype=np.float32).astype(np.float64)
    keep = np.ones(len(z), dtype=bool)
    if 0 < top_k < len(z):
        keep = z >= np.sort(z)[::-1][top_k - 1]
    zt = z / float(temperature)
    p = np.where(keep, np.exp(zt - zt[keep].max()), 0.0)
    return p / p.sum()


def most_probable(p, k: int):
    """The k most probable tokens in order, ties towards the lower id."""
    return sorted(range(len(p)), key=lambda v: (-p[v], v))[:k]


def draw(p, u: float) -> int:
    """Inverse CDF: the smallest v whose running sum exceeds u * sum(p); if rounding leaves none, the largest v with p[v] > 0."""
    target = u * float(np.sum(p))
    run = 0.0
    last = -1
    for v, pv in enumerate(p):
        if pv > 0.0:
            last = v
        run += pv
        if run > target:
            return v
    return last


class StagedOracle:
    def __init__(self, oracle_model, draft_model, trigram, mode: int = 0, temperature: float = 1.0, top_k: int = 0, rounds: int = 2,
                 siblings: int = 1, seed: int = 0):
        self.m0, self.m1, self.tri = oracle_model, draft_model, trigram
        self.kv0, self.kv1 = oracle_model.new_kv(), draft_model.new_kv()
        self.mode, self.T, self.top_k, self.rounds, self.siblings, self.seed = mode, float(np.float32(temperature)), top_k, rounds, siblings, seed
        self.V = oracle_model.cfg["vocab"]
        self.rng_step = 0
        self.seq = []
        self.min_margin = float("inf")
        self.stats = {"target_steps": 0, "draft_forwards": 0, "emitted": 0, "origin": {"trigram": 0, "draft": 0, "target": 0}}

    def next_step(self) -> int:
        s = self.rng_step
        self.rng_step += 1
        return s

    def prefill(self, prompt):
        """Both caches take every prompt token but the last, which becomes the first root."""
        prompt = [int(t) for t in prompt]
        assert len(prompt) >= 2
        self.kv0.prefill(np.asarray(prompt[:-1], dtype=np.int32), chunk=64)
        self.kv1.prefill(np.asarray(prompt[:-1], dtype=np.int32), chunk=64)
        self.seq = list(prompt)

    def step(self):
        V, seq_old = self.V, list(self.seq)
        chain, chain_rows, sibs = [], [], []          # (token, origin); M1's law at its parent; extra leaves of that level
        # ---------------- stage 2 -> 1
        for _ in range(self.rounds):
            ctx = seq_old + [t for t, _ in chain]
            stem = ctx[len(self.kv1):]
            s = len(stem)
            assert 1 <= s <= 2
            prev1 = ctx[-2] if len(ctx) >= 2 else ctx[-1]
            ttok, _ = self.tri.propose_tree(int(prev1), int(stem[-1]), TRI_PARENT)
            tokens2 = np.asarray(stem[:-1] + [int(t) for t in ttok], dtype=np.int32)
            parent2 = np.asarray(list(range(-1, s - 1)) + [(s - 1) + int(p) for p in TRI_PARENT[1:]], dtype=np.int32)
            logits1 = self.kv1.verify_tree(tokens2, parent2)
            self.stats["draft_forwards"] += 1
            sub_tokens, sub_logits = tokens2[s - 1:], np.ascontiguousarray(logits1[s - 1:], dtype=np.float32)
            rows = None
            if self.mode == 1:  # the trigram's proposals are deterministic: one-hot rows
                rows = np.zeros((len(sub_tokens), V), dtype=np.float32)
                rows[np.arange(1, len(sub_tokens)), sub_tokens[1:]] = 1.0
            path1, bonus1, margin = ssd_oracle.accept_tree(sub_logits, rows, sub_tokens, TRI_PARENT, mode=self.mode, temperature=self.T,
                                                           top_k=self.top_k, seed=self.seed, step=self.next_step())
            self.min_margin = min(self.min_margin, margin)
            new_chain = [(int(sub_tokens[c]), "trigram") for c in path1[1:]] + [(int(bonus1), "draft")]
            sib_step = self.next_step()
            for j, (tok, _) in enumerate(new_chain):
                node = path1[j]                                            # the chain token's parent, a node M1 has scored
                p = law(sub_logits[node], self.T, self.top_k)
                chain_rows.append(p.astype(np.float32))
                if self.mode == 0:
                    best = most_probable(p, self.siblings + 1)
                    assert best[0] == tok                                  # deterministic decoding: the chain is M1's first choice
                    sibs.append(best[1:])
                else:
                    sibs.append([draw(p, ssd_oracle.uniform(self.seed, sib_step, 1024 + 16 * node + t)) for t in range(self.siblings)])
            self.kv1.commit(list(range(s - 1)) + [(s - 1) + c for c in path1])
            chain += new_chain
        # ---------------- stage 1 -> 0
        m = len(chain)
        tokens1 = [seq_old[-1]] + [t for t, _ in chain]
        parent1 = [-1] + list(range(m))
        origin1 = ["root"] + [o for _, o in chain]
        row_of = list(range(-1, m))                                        # node j (1..m) was proposed from chain_rows[j - 1]
        for level, extra in enumerate(sibs):
            for t in extra:
                tokens1.append(int(t)); parent1.append(level); origin1.append("draft"); row_of.append(level)
        tokens1, parent1 = np.asarray(tokens1, dtype=np.int32), np.asarray(parent1, dtype=np.int32)
        rows1 = None
        if self.mode == 1:
            rows1 = np.zeros((len(tokens1), V), dtype=np.float32)
            for c in range(1, len(tokens1)):
                rows1[c] = chain_rows[row_of[c]]
        logits0 = np.ascontiguousarray(self.kv0.verify_tree(tokens1, parent1), dtype=np.float32)
        path0, next0, margin = ssd_oracle.accept_tree(logits0, rows1, tokens1, parent1, mode=self.mode, temperature=self.T, top_k=self.top_k,
                                                      seed=self.seed, step=self.next_step())
        self.min_margin = min(self.min_margin, margin)
        self.kv0.commit(path0)
        emitted = [int(tokens1[c]) for c in path0[1:]] + [int(next0)]
        origins = [origin1[c] for c in path0[1:]] + ["target"]
        k = sum(1 for j, c in enumerate(path0[1:], start=1) if c == j)     # chain tokens the oracle accepted
        self.kv1.rollback(len(seq_old) + min(k, m - 1))
        self.seq = seq_old + emitted
        self.stats["target_steps"] += 1
        self.stats["emitted"] += len(emitted)
        for o in origins:
            self.stats["origin"][o] += 1
        return emitted, origins

    def generate(self, n_tokens: int):
        out = []
        while len(out) < n_tokens:
            out += self.step()[0]
        return out[:n_tokens]


def greedy_autoregressive(model, prompt, n_tokens: int):
    """Plain token-by-token greedy decoding with the same model (Section 2.1): the sequence deterministic staged decoding must reproduce."""
    kv = model.new_kv()
    prompt = [int(t) for t in prompt]
    kv.prefill(np.asarray(prompt[:-1], dtype=np.int32), chunk=64)
    last, out = prompt[-1], []
    for _ in range(n_tokens):
        logits = np.asarray(kv.verify_tree(np.asarray([last], dtype=np.int32), np.asarray([-1], dtype=np.int32)), dtype=np.float32)
        kv.commit([0])
        last = int(np.argmax(logits[0]))
        out.append(last)
    return out
