"""The full staged decoding loop on the device (Section 3 of the paper), sequenced through the C ABI.

Three stages: the large model whose output the method preserves (the paper's top-level model, called the target here), a small draft model and a trigram table (Section 4).  This module holds
no arithmetic: every forward, every acceptance decision, every proposal law, every draw and every table
look-up is a kernel of libssd reached through `binding`; what is left here is the bookkeeping of which node
hangs under which (lists of small integers) and the order of the calls.  torch is used for device buffers
and for copying proposal rows between them.

One step:
  stage 2 -> 1 (Section 3.2), `rounds` times: ssd_trigram_propose fills the eight-node tree below the last
      token the draft has not cached; the draft scores it with ssd_verify_tree; ssd_accept_tree_sparse walks
      it (the trigram's proposals are its most probable continuations, so their rows are one-hot);
      ssd_propose_children returns the draft's law at every node of the accepted path - the proposal rows of
      the chain for the next stage - and the sibling leaves of each level; ssd_kv_commit appends the accepted
      slices to the draft's cache speculatively.
  stage 1 -> 0 (Section 3.1): the target model scores the chain plus its sibling leaves in one ssd_verify_tree,
      ssd_accept_tree walks it, ssd_kv_commit appends the accepted slices, and ssd_kv_rollback takes the
      draft's cache back to what both models accepted.
"""
from __future__ import annotations

import numpy as np

from . import binding as B

TRI_PARENT = np.array([-1, 0, 0, 0, 1, 1, 4, 6], dtype=np.int32)


class StagedDecoder:
    def __init__(self, target_ctx: B.Context, draft_ctx: B.Context, trigram: B.Trigram, mode: int = B.SSD_GREEDY, temperature: float = 1.0,
                 top_k: int = 0, rounds: int = 2, siblings: int = 1, seed: int = 0):
        import torch
        self.torch = torch
        self.c0, self.c1, self.tri = target_ctx, draft_ctx, trigram
        self.kv0, self.kv1 = target_ctx.new_kv(), draft_ctx.new_kv()
        self.mode, self.T, self.top_k, self.rounds, self.siblings = mode, float(np.float32(temperature)), top_k, rounds, siblings
        self.V = target_ctx.cfg["vocab"]
        self.rng = B.ssd_rng(seed, 0)
        self.seq = []
        max_chain = rounds * len(TRI_PARENT)
        self.logits0 = torch.empty((max_chain * (1 + siblings) + 1, self.V), dtype=torch.float32, device="cuda")
        self.logits1 = torch.empty((len(TRI_PARENT) + 1, self.V), dtype=torch.float32, device="cuda")
        self.chain_rows = torch.zeros((max_chain + 1, self.V), dtype=torch.float32, device="cuda")   # row j: the law chain token j was proposed from
        self.rows1 = torch.zeros_like(self.logits0)
        self.stats = {"target_steps": 0, "draft_forwards": 0, "emitted": 0, "origin": {"trigram": 0, "draft": 0, "target": 0}}

    def prefill(self, prompt):
        """Both caches take every prompt token but the last, which becomes the first root (hot-path calls only)."""
        prompt = [int(t) for t in prompt]
        assert len(prompt) >= 2
        body = np.asarray(prompt[:-1], dtype=np.int32)
        for ctx, kv in ((self.c0, self.kv0), (self.c1, self.kv1)):
            buf = self.torch.empty((64, self.V), dtype=self.torch.float32, device="cuda")
            for s in range(0, len(body), 64):
                t = body[s:s + 64]
                ctx.verify_tree(t, np.arange(-1, len(t) - 1, dtype=np.int32), kv, buf.data_ptr())
                ctx.kv_commit(kv, np.arange(len(t), dtype=np.int32))
        self.seq = list(prompt)

    def step(self):
        V, seq_old = self.V, list(self.seq)
        row_bytes = 4 * V
        chain, sibs = [], []
        # ---------------- stage 2 -> 1
        for _ in range(self.rounds):
            ctx = seq_old + [t for t, _ in chain]
            stem = ctx[len(self.kv1):]
            s = len(stem)
            assert 1 <= s <= 2
            prev1 = ctx[-2] if len(ctx) >= 2 else ctx[-1]
            ttok, _ = self.tri.propose(prev1, stem[-1], TRI_PARENT)
            tokens2 = np.asarray(stem[:-1] + [int(t) for t in ttok], dtype=np.int32)
            parent2 = np.asarray(list(range(-1, s - 1)) + [(s - 1) + int(p) for p in TRI_PARENT[1:]], dtype=np.int32)
            self.c1.verify_tree(tokens2, parent2, self.kv1, self.logits1.data_ptr())
            self.stats["draft_forwards"] += 1
            sub_tokens, sub_ptr = tokens2[s - 1:], self.logits1.data_ptr() + (s - 1) * row_bytes
            if self.mode == B.SSD_SAMPLING:   # one-hot rows as one-entry lists
                idx = np.concatenate([[-1], sub_tokens[1:]]).astype(np.int32).reshape(-1, 1)
                val = np.ones((len(sub_tokens), 1), dtype=np.float32)
                path1, bonus1 = self.c1.accept_tree_sparse(sub_ptr, idx, val, sub_tokens, TRI_PARENT, mode=self.mode, temperature=self.T,
                                                           top_k=self.top_k, rng=self.rng)
            else:
                path1, bonus1 = self.c1.accept_tree(sub_ptr, None, sub_tokens, TRI_PARENT, mode=self.mode, rng=self.rng)
            new_chain = [(int(sub_tokens[c]), "trigram") for c in path1[1:]] + [(int(bonus1), "draft")]
            at = len(chain)
            picks = self.siblings + 1 if self.mode == B.SSD_GREEDY else self.siblings
            got = self.c1.propose_children(sub_ptr, path1, picks, mode=self.mode, temperature=self.T, top_k=self.top_k, rng=self.rng,
                                           rows_out_ptr=self.chain_rows.data_ptr() + at * row_bytes)
            for j, (tok, _) in enumerate(new_chain):
                if self.mode == B.SSD_GREEDY:
                    assert int(got[j, 0]) == tok   # deterministic decoding: the chain is the draft's first choice
                    sibs.append([int(v) for v in got[j, 1:]])
                else:
                    sibs.append([int(v) for v in got[j]])
            self.c1.kv_commit(self.kv1, list(range(s - 1)) + [(s - 1) + c for c in path1])
            chain += new_chain
        # ---------------- stage 1 -> 0
        m = len(chain)
        tokens1 = [seq_old[-1]] + [t for t, _ in chain]
        parent1 = [-1] + list(range(m))
        origin1 = ["root"] + [o for _, o in chain]
        row_of = list(range(-1, m))
        for level, extra in enumerate(sibs):
            for t in extra:
                tokens1.append(t); parent1.append(level); origin1.append("draft"); row_of.append(level)
        n1 = len(tokens1)
        self.c0.verify_tree(tokens1, parent1, self.kv0, self.logits0.data_ptr())
        rows_ptr = None
        if self.mode == B.SSD_SAMPLING:     # every node's proposal row: the law of its level (a copy between device buffers)
            self.rows1[1:n1] = self.chain_rows[self.torch.as_tensor(row_of[1:], device="cuda")]
            rows_ptr = self.rows1.data_ptr()
        path0, next0 = self.c0.accept_tree(self.logits0.data_ptr(), rows_ptr, tokens1, parent1, mode=self.mode, temperature=self.T,
                                           top_k=self.top_k, rng=self.rng)
        self.c0.kv_commit(self.kv0, path0)
        emitted = [int(tokens1[c]) for c in path0[1:]] + [int(next0)]
        origins = [origin1[c] for c in path0[1:]] + ["target"]
        k = sum(1 for j, c in enumerate(path0[1:], start=1) if c == j)
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

    def close(self):
        self.kv0.close()
        self.kv1.close()
