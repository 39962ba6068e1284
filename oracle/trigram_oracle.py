"""CPU oracle of the lowest speculation stage: a Katz back-off trigram model (test infrastructure).

Section 4 of the paper names the third model of its staged pipeline: a Katz back-off trigram model
that proposes tokens for the small draft model (Section 3.2).  The paper gives neither the discount
nor how the proposals are read off the model, so this file fixes one plain reading and states it:

  * counts c3(a, b, w), c2(b, w), c1(w) over every position of a token stream of length N;
  * absolute discount D = 0.5 (Katz's back-off with a fixed discount instead of Good-Turing counts):
        P1(w)       = c1(w) / N
        P2(w | b)   = (c2(b, w) - D) / c2(b, .)                     if c2(b, w) > 0
                    = alpha2(b) * P1(w)                             otherwise
        P3(w | a,b) = (c3(a, b, w) - D) / c3(a, b, .)               if c3(a, b, w) > 0
                    = alpha3(a, b) * P2(w | b)                      otherwise
    with the back-off weights that make each level sum to one:
        alpha2(b)    = (D * types2(b) / c2(b, .))       / (1 - sum of P1(w)     over the w seen after b)
        alpha3(a, b) = (D * types3(a, b) / c3(a, b, .)) / (1 - sum of P2(w | b) over the w seen after (a, b));
    a context never seen backs off entirely: P3(. | a, b) = P2(. | b), P2(. | b) = P1;
  * the proposals for a context are the K = 4 most probable next tokens under P3, ties broken towards
    the lower token id.

Everything is plain Python over dictionaries and a loop over the whole vocabulary (the definition
written out, fp64); only tests and the benchmark's CPU leg may import it.  It shares no code with the
CUDA library.
"""
from __future__ import annotations

from collections import defaultdict

import numpy as np

DISCOUNT = 0.5
TOP = 4


class KatzTrigram:
    def __init__(self, stream, vocab: int):
        s = [int(t) for t in stream]
        self.V, self.N = int(vocab), len(s)
        self.c1 = np.zeros(self.V, dtype=np.int64)
        self.c2 = defaultdict(lambda: defaultdict(int))
        self.c3 = defaultdict(lambda: defaultdict(int))
        for t in s:
            self.c1[t] += 1
        for i in range(1, len(s)):
            self.c2[s[i - 1]][s[i]] += 1
        for i in range(2, len(s)):
            self.c3[(s[i - 2], s[i - 1])][s[i]] += 1

    def p1(self) -> np.ndarray:
        return self.c1.astype(np.float64) / self.N

    def p2(self, b: int) -> np.ndarray:
        p1 = self.p1()
        seen = self.c2.get(b)
        if not seen:
            return p1
        tot = sum(seen.values())
        out = np.zeros(self.V)
        mass_seen_lower = 0.0
        for w, c in sorted(seen.items()):  # (sums in ascending token order)
            out[w] = (c - DISCOUNT) / tot
            mass_seen_lower += p1[w]
        alpha = (DISCOUNT * len(seen) / tot) / (1.0 - mass_seen_lower) if mass_seen_lower < 1.0 else 0.0
        for w in range(self.V):
            if w not in seen:
                out[w] = alpha * p1[w]
        return out

    def p3(self, a: int, b: int) -> np.ndarray:
        p2 = self.p2(b)
        seen = self.c3.get((a, b))
        if not seen:
            return p2
        tot = sum(seen.values())
        out = np.zeros(self.V)
        mass_seen_lower = 0.0
        for w, c in sorted(seen.items()):
            out[w] = (c - DISCOUNT) / tot
            mass_seen_lower += p2[w]
        alpha = (DISCOUNT * len(seen) / tot) / (1.0 - mass_seen_lower) if mass_seen_lower < 1.0 else 0.0
        for w in range(self.V):
            if w not in seen:
                out[w] = alpha * p2[w]
        return out

    def top_next(self, a: int, b: int, k: int = TOP):
        """The k most probable next tokens after (a, b) and their probabilities; ties go to the lower id."""
        p = self.p3(a, b)
        order = sorted(range(self.V), key=lambda w: (-p[w], w))[:k]
        return np.asarray(order, dtype=np.int32), np.asarray([p[w] for w in order], dtype=np.float64)

    def propose_tree(self, prev1: int, root: int, parent):
        """Fills a tree whose node 0 holds `root` (preceded by `prev1`): the children of a node, in index order, get the
        most probable next tokens of the node's context (its parent's token, its own token).  Returns tokens, probabilities."""
        n = len(parent)
        tokens = np.zeros(n, dtype=np.int32)
        probs = np.zeros(n, dtype=np.float64)
        tokens[0] = root
        before = {0: prev1}
        kids = defaultdict(list)
        for i in range(1, n):
            kids[int(parent[i])].append(i)
        for p in range(n):
            if not kids[p]:
                continue
            assert len(kids[p]) <= TOP
            ids, pr = self.top_next(before[p], int(tokens[p]), TOP)
            for rank, c in enumerate(kids[p]):
                tokens[c], probs[c] = ids[rank], pr[rank]
                before[c] = int(tokens[p])
        return tokens, probs
