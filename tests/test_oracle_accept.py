"""Pins of the oracle's acceptance walk (no GPU).

The paper states the property (Sections 1 and 2.3: speculation keeps the model's
distribution exactly) but not the rule.  Two things are therefore checked:
 (1) the sibling-wise residual rejection rule, written here with exact rationals,
     has output law == the target law for every way a proposer may build the
     tree (exhaustive enumeration on a small vocabulary);
 (2) the oracle's C implementation of that rule reproduces the target law
     (chi-square on a 16-token vocabulary, trees re-drawn from the draft in every
     trial) and its deterministic special cases.
"""
import itertools
from fractions import Fraction as Fr

import numpy as np
import pytest
from scipy.stats import chi2

import ssd_synth
from oracle import ssd_oracle


# ---------------------------------------------------------------------------
# (1) exactness of the rule by enumeration with rationals
# ---------------------------------------------------------------------------
def first_token_law(p, rows, xs):
    """Exact law of the first emitted token for fixed sibling tokens xs, rows[i] the
    proposal row of sibling i: accept x with probability min(1, r[x]/q[x]) (always if
    q[x] == 0 < r[x]), on refusal r <- normalised positive part of r - q."""
    V = len(p)
    out, alive, r = [Fr(0)] * V, Fr(1), list(p)
    for x, q in zip(xs, rows):
        if q[x] == 0:
            a = Fr(1) if r[x] > 0 else Fr(0)
        else:
            a = min(Fr(1), r[x] / q[x])
        out[x] += alive * a
        alive *= 1 - a
        t = [max(Fr(0), rv - qv) for rv, qv in zip(r, q)]
        Z = sum(t)
        if Z > 0:
            r = [tv / Z for tv in t]
    return [o + alive * rv for o, rv in zip(out, r)]


def rational_dist(rng, V, denom=60, zeros=0):
    cuts = sorted(rng.choice(np.arange(1, denom), size=V - 1 - zeros, replace=False))
    parts = np.diff([0] + list(cuts) + [denom]).tolist() + [0] * zeros
    rng.shuffle(parts)
    return [Fr(int(a), denom) for a in parts]


@pytest.mark.parametrize("k", [1, 2, 3])
def test_rule_exact_for_iid_siblings(k):
    rng = np.random.default_rng(k)
    V = 5
    p, q = rational_dist(rng, V, zeros=1), rational_dist(rng, V)
    law = [Fr(0)] * V
    for xs in itertools.product(range(V), repeat=k):
        wt = Fr(1)
        for x in xs:
            wt *= q[x]
        if wt:
            law = [a + wt * b for a, b in zip(law, first_token_law(p, [q] * k, xs))]
    assert law == p


@pytest.mark.parametrize("k", [2, 3])
def test_rule_exact_for_siblings_without_replacement(k):
    rng = np.random.default_rng(10 + k)
    V = 5
    p, q = rational_dist(rng, V), rational_dist(rng, V)
    law = [Fr(0)] * V
    for xs in itertools.permutations(range(V), k):
        wt, rows, rem = Fr(1), [], list(q)
        for x in xs:
            s = sum(rem)
            row = [a / s for a in rem]
            rows.append(row)
            wt *= row[x]
            rem[x] = Fr(0)
        law = [a + wt * b for a, b in zip(law, first_token_law(p, rows, xs))]
    assert law == p


def test_rule_exact_for_deterministic_top_children():
    rng = np.random.default_rng(4)
    V = 5
    p, q = rational_dist(rng, V), rational_dist(rng, V)
    xs = sorted(range(V), key=lambda v: -q[v])[:3]
    rows = [[Fr(int(v == x)) for v in range(V)] for x in xs]
    assert first_token_law(p, rows, xs) == p


def test_rule_exact_two_levels():
    """Joint law of the first two tokens on a depth-2 tree with 2 i.i.d. children per node."""
    rng = np.random.default_rng(9)
    V = 3
    p1, q1 = rational_dist(rng, V, denom=12), rational_dist(rng, V, denom=12)
    p2 = [rational_dist(rng, V, denom=12) for _ in range(V)]
    q2 = [rational_dist(rng, V, denom=12) for _ in range(V)]
    joint = {}
    # level 1: children (a, b) ~ q1 x q1; level 2 under an accepted child with token x: (c, d) ~ q2[x] x q2[x]
    for a, b in itertools.product(range(V), repeat=2):
        w1 = q1[a] * q1[b]
        if not w1:
            continue
        law1 = first_token_law(p1, [q1, q1], (a, b))
        # the first token is x1 with law1[x1]; if x1 came from an accepted child the second token is
        # decided in the same step from that child's subtree, else in the next step; both have law p2[x1]
        for x1 in range(V):
            for c, d in itertools.product(range(V), repeat=2):
                w2 = q2[x1][c] * q2[x1][d]
                if not w2:
                    continue
                law2 = first_token_law(p2[x1], [q2[x1], q2[x1]], (c, d))
                for x2 in range(V):
                    joint[(x1, x2)] = joint.get((x1, x2), Fr(0)) + w1 * law1[x1] * w2 * law2[x2]
    for x1 in range(V):
        for x2 in range(V):
            assert joint[(x1, x2)] == p1[x1] * p2[x1][x2]


def test_reusing_one_row_for_dependent_siblings_is_wrong():
    """Why each child carries its own proposal row: with siblings drawn without
    replacement, testing all of them against the parent's single row changes the law."""
    rng = np.random.default_rng(12)
    V = 5
    p, q = rational_dist(rng, V), rational_dist(rng, V)
    law = [Fr(0)] * V
    for xs in itertools.permutations(range(V), 2):
        wt, rem = Fr(1), list(q)
        for x in xs:
            s = sum(rem)
            wt *= rem[x] / s
            rem[x] = Fr(0)
        law = [a + wt * b for a, b in zip(law, first_token_law(p, [q, q], xs))]
    assert max(abs(a - b) for a, b in zip(law, p)) > Fr(1, 100)


# ---------------------------------------------------------------------------
# (2) the C implementation: statistical law, special cases, deterministic mode
# ---------------------------------------------------------------------------
def logits_of(p):
    with np.errstate(divide="ignore"):
        return np.maximum(np.log(np.asarray(p, dtype=np.float64)), -80.0).astype(np.float32)


def chi_square(counts, probs, min_expected=10.0):
    """Pearson statistic after merging cells with a small expected count; returns (stat, dof)."""
    N = counts.sum()
    order = np.argsort(probs)
    c, e = counts[order].astype(float), probs[order] * N
    cells_c, cells_e, ac, ae = [], [], 0.0, 0.0
    for ci, ei in zip(c, e):
        ac += ci
        ae += ei
        if ae >= min_expected:
            cells_c.append(ac)
            cells_e.append(ae)
            ac = ae = 0.0
    if ae > 0:
        cells_c[-1] += ac
        cells_e[-1] += ae
    cc, ee = np.array(cells_c), np.array(cells_e)
    return float(((cc - ee) ** 2 / ee).sum()), len(cc) - 1


def test_chi_square_first_token_law_16_vocab():
    V, N, k = 16, 200_000, 3
    rng = np.random.default_rng(16)
    p = rng.dirichlet(np.full(V, 0.5))
    q = rng.dirichlet(np.full(V, 0.5)).astype(np.float32)
    p32 = np.exp(logits_of(p).astype(np.float64))
    p32 /= p32.sum()  # the law the fp32 logits actually encode
    parent = np.array([-1] + [0] * k, dtype=np.int32)
    logits = np.tile(logits_of(p), (k + 1, 1))
    rows = np.tile(q, (k + 1, 1))
    kids = rng.choice(V, size=(N, k), p=q.astype(np.float64) / q.astype(np.float64).sum())
    counts = np.zeros(V, dtype=np.int64)
    tokens = np.zeros(k + 1, dtype=np.int32)
    for t in range(N):
        tokens[1:] = kids[t]
        path, nxt, _ = ssd_oracle.accept_tree(logits, rows, tokens, parent, mode=1, seed=123, step=t)
        counts[tokens[path[1]] if len(path) > 1 else nxt] += 1
    stat, dof = chi_square(counts, p32)
    assert stat < chi2.ppf(0.999, dof), (stat, dof)
    # power of the test: the same counts do NOT fit the draft's law
    stat_q, dof_q = chi_square(counts, q.astype(np.float64) / q.sum())
    assert stat_q > 10 * chi2.ppf(0.999, dof_q)


def test_chi_square_joint_of_two_tokens_16_vocab():
    """Two emitted tokens through a depth-2 tree (2 children per node, drawn from the
    draft) and, when the first step stops at the root, a second step."""
    V, N = 16, 120_000
    rng = np.random.default_rng(17)
    p1 = rng.dirichlet(np.full(V, 0.5))
    p2 = rng.dirichlet(np.full(V, 0.5), size=V)
    q1 = rng.dirichlet(np.full(V, 0.5)).astype(np.float32)
    q2 = rng.dirichlet(np.full(V, 0.5), size=V).astype(np.float32)
    enc = lambda p: (lambda e: e / e.sum())(np.exp(logits_of(p).astype(np.float64)))
    joint = (enc(p1)[:, None] * np.stack([enc(p2[x]) for x in range(V)])).ravel()
    l1, l2 = logits_of(p1), np.stack([logits_of(p2[x]) for x in range(V)])
    parent = np.array([-1, 0, 0, 1, 1, 2, 2], dtype=np.int32)
    nq1 = q1.astype(np.float64) / q1.astype(np.float64).sum()
    nq2 = q2.astype(np.float64) / q2.astype(np.float64).sum(axis=1, keepdims=True)
    counts = np.zeros(V * V, dtype=np.int64)
    for t in range(N):
        tokens = np.zeros(7, dtype=np.int32)
        tokens[1:3] = rng.choice(V, size=2, p=nq1)
        tokens[3:5] = rng.choice(V, size=2, p=nq2[tokens[1]])
        tokens[5:7] = rng.choice(V, size=2, p=nq2[tokens[2]])
        logits = np.stack([l1, l2[tokens[1]], l2[tokens[2]], l1, l1, l1, l1])
        rows = np.stack([q1, q1, q1, q2[tokens[1]], q2[tokens[1]], q2[tokens[2]], q2[tokens[2]]])
        path, nxt, _ = ssd_oracle.accept_tree(logits, rows, tokens, parent, mode=1, seed=77, step=2 * t)
        out = [int(tokens[c]) for c in path[1:]] + [nxt]
        if len(out) < 2:  # next step: new root = the emitted token, fresh tree below it
            tk = np.zeros(3, dtype=np.int32)
            tk[0] = out[0]
            tk[1:] = rng.choice(V, size=2, p=nq2[out[0]])
            lg = np.stack([l2[out[0]], l1, l1])
            rw = np.stack([q1, q2[out[0]], q2[out[0]]])
            path, nxt, _ = ssd_oracle.accept_tree(lg, rw, tk, [-1, 0, 0], mode=1, seed=77, step=2 * t + 1)
            out += [int(tk[c]) for c in path[1:]] + [nxt]
        counts[out[0] * V + out[1]] += 1
    stat, dof = chi_square(counts, joint)
    assert stat < chi2.ppf(0.999, dof), (stat, dof)


def test_identical_draft_always_accepts_first_child():
    V = 16
    rng = np.random.default_rng(1)
    p = rng.dirichlet(np.full(V, 0.5))
    lg = logits_of(p)
    p32 = np.exp(lg.astype(np.float64))
    q = (p32 / p32.sum()).astype(np.float32) * np.float32(0.999)  # q <= p everywhere => ratio >= 1
    for t in range(300):
        x = int(rng.choice(V, p=p))
        path, nxt, _ = ssd_oracle.accept_tree(np.stack([lg, lg]), np.stack([q, q]), [0, x], [-1, 0], mode=1, seed=5, step=t)
        assert path == [0, 1]


def test_disjoint_supports_always_reject_and_bonus_follows_target():
    V, N = 16, 40_000
    rng = np.random.default_rng(2)
    p = np.zeros(V)
    p[:8] = rng.dirichlet(np.full(8, 0.5))
    q = np.zeros(V, dtype=np.float32)
    q[8:] = rng.dirichlet(np.full(8, 0.5))
    lg = np.where(p > 0, np.log(np.maximum(p, 1e-300)), -np.inf)
    lg = np.where(np.isfinite(lg), lg, -1e4).astype(np.float32)  # finite logits, zero mass after exp
    counts = np.zeros(V, dtype=np.int64)
    for t in range(N):
        x = 8 + int(rng.integers(8))
        path, nxt, _ = ssd_oracle.accept_tree(np.stack([lg, lg, lg]), np.stack([q, q, q]), [0, x, x], [-1, 0, 0],
                                              mode=1, seed=6, step=t)
        assert path == [0]
        counts[nxt] += 1
    assert counts[8:].sum() == 0
    enc = np.exp(lg[:8].astype(np.float64))
    stat, dof = chi_square(counts[:8], enc / enc.sum())
    assert stat < chi2.ppf(0.999, dof)


def test_one_hot_draft_accepts_with_target_probability():
    V, N = 16, 40_000
    rng = np.random.default_rng(3)
    p = rng.dirichlet(np.full(V, 2.0))
    lg = logits_of(p)
    enc = np.exp(lg.astype(np.float64))
    enc /= enc.sum()
    x = 5
    q = np.zeros(V, dtype=np.float32)
    q[x] = 1.0
    acc = 0
    for t in range(N):
        path, nxt, _ = ssd_oracle.accept_tree(np.stack([lg, lg]), np.stack([q, q]), [0, x], [-1, 0], mode=1, seed=8, step=t)
        acc += len(path) == 2
        if len(path) == 1:
            assert nxt != x  # after refusing x the residual has no mass on x
    assert abs(acc / N - enc[x]) < 4 * np.sqrt(enc[x] * (1 - enc[x]) / N)


def test_duplicate_sibling_is_refused_after_first_refusal_and_zero_q_accepts():
    V = 8
    p = np.full(V, 1.0 / V)
    lg = logits_of(p)
    q = np.zeros(V, dtype=np.float32)
    q[3] = 1.0
    # find a step whose first uniform refuses token 3 (u >= 1/8); then the duplicate must be refused as well
    for t in range(50):
        if ssd_oracle.uniform(1, t, 2) >= 0.125 + 1e-6:
            path, nxt, _ = ssd_oracle.accept_tree(np.stack([lg] * 3), np.stack([q] * 3), [0, 3, 3], [-1, 0, 0], mode=1, seed=1, step=t)
            assert path == [0] and nxt != 3
            break
    else:
        raise AssertionError("no refusing draw found")
    # a child whose token has zero proposal mass but positive target mass is accepted (product form u*0 < r)
    path, nxt, _ = ssd_oracle.accept_tree(np.stack([lg] * 2), np.stack([q] * 2), [0, 6], [-1, 0], mode=1, seed=1, step=0)
    assert path == [0, 1]


def test_chain_tree_reduces_to_single_sequence_rule():
    """One child per node: accept x with probability min(1, p/q); stop at the first refusal."""
    V = 16
    rng = np.random.default_rng(40)
    for t in range(200):
        p = rng.dirichlet(np.full(V, 0.5), size=4)
        q = rng.dirichlet(np.full(V, 0.5), size=4).astype(np.float32)
        toks = np.concatenate([[0], rng.integers(0, V, size=3)]).astype(np.int32)
        lg = np.stack([logits_of(r) for r in p])
        path, nxt, _ = ssd_oracle.accept_tree(lg, q, toks, [-1, 0, 1, 2], mode=1, seed=31, step=t)
        want, cur = [0], 0
        for c in (1, 2, 3):
            e = np.exp(lg[cur].astype(np.float64))
            r = e / e.sum()
            if ssd_oracle.uniform(31, t, 2 * c) * float(q[c][toks[c]]) < r[toks[c]]:
                want.append(c)
                cur = c
            else:
                break
        assert path == want


def test_greedy_walk_follows_argmax_children_and_breaks_ties_low():
    V = 10
    lg = np.zeros((6, V), dtype=np.float32)
    lg[0, 4] = 2.0          # root prefers 4
    lg[2, 7] = 1.0          # node 2 prefers 7
    lg[4, [3, 8]] = 5.0     # tie at node 4: lowest index (3) wins
    parent = np.array([-1, 0, 0, 2, 2, 4], dtype=np.int32)
    tokens = np.array([1, 9, 4, 6, 7, 8], dtype=np.int32)
    path, nxt, _ = ssd_oracle.accept_tree(lg, None, tokens, parent, mode=0)
    assert (path, nxt) == ([0, 2, 4], 3)
    tokens[5] = 3
    path, nxt, _ = ssd_oracle.accept_tree(lg, None, tokens, parent, mode=0)
    assert path == [0, 2, 4, 5] and nxt == 0  # leaf row is all zeros: argmax = lowest index
    # duplicate sibling tokens: the first one is taken
    path, nxt, _ = ssd_oracle.accept_tree(lg[:3], None, [1, 4, 4], [-1, 0, 0], mode=0)
    assert path == [0, 1]


def test_top_k_and_temperature_warp():
    V, N = 16, 30_000
    rng = np.random.default_rng(50)
    z = rng.normal(size=V).astype(np.float32) * 2
    z[3] = z[9]  # a tie inside the row
    k, T = 5, 0.7
    kth = np.sort(z)[::-1][k - 1]
    e = np.where(z >= kth, np.exp(z.astype(np.float64) / T), 0.0)
    want = e / e.sum()
    q = np.full(V, 1.0 / V, dtype=np.float32)
    counts = np.zeros(V, dtype=np.int64)
    for t in range(N):
        x = int(rng.integers(V))
        path, nxt, _ = ssd_oracle.accept_tree(np.stack([z, z]), np.stack([q, q]), [0, x], [-1, 0], mode=1, temperature=T,
                                              top_k=k, seed=9, step=t)
        counts[x if len(path) == 2 else nxt] += 1
    assert counts[want == 0].sum() == 0
    stat, dof = chi_square(counts[want > 0], want[want > 0])
    assert stat < chi2.ppf(0.999, dof)


def test_non_finite_logits_are_reported():
    lg = np.zeros((2, 8), dtype=np.float32)
    lg[0, 2] = np.nan
    with pytest.raises(ssd_oracle.OracleError) as e:
        ssd_oracle.accept_tree(lg, None, [0, 1], [-1, 0], mode=0)
    assert e.value.code == ssd_oracle.ORC_BAD_ARG


def test_min_margin_closed_form_on_four_word_vocabulary():
    """The margin the oracle reports (how close the nearest decision came to flipping) on a hand-made case
    where every quantity is a dyadic rational, so the expected value is exact in fp64.

    Vocabulary of 4, all logits zero: every node's target law is (1/4, 1/4, 1/4, 1/4).  One child c = 1 of
    the root with token 0, proposed from q = (1/2, 1/2, 0, 0).  With u = u(seed, step, 2c):
      accept test   u / 2 < 1 / 4, relative distance |u / 2 - 1 / 4| / (1 / 4) = |2 u - 1|;
      accepted      the extra token is drawn at the leaf from the uniform law with u' = u(seed, step, 2 c + 1):
                    cell v = floor(4 u'), distance to the nearer cell edge over the cell's mass
                    = min(4 u' - v, v + 1 - 4 u');
      refused       residual = positive part of p - q = (0, 0, 1/4, 1/4), renormalised (0, 0, 1/2, 1/2); the
                    extra token is drawn at the root with u' = u(seed, step, 1): token 2 if u' < 1 / 2 else 3,
                    distance min(2 u' - (v - 2), (v - 1) - 2 u').
    The reported margin is the smaller of the two distances."""
    V = 4
    logits = np.zeros((2, V), dtype=np.float32)
    draft = np.zeros((2, V), dtype=np.float32)
    draft[1] = [0.5, 0.5, 0.0, 0.0]
    tokens, parent = [3, 0], [-1, 0]
    seen = {"accepted": 0, "refused": 0}
    for step in range(64):
        u = ssd_oracle.uniform(123, step, 2)
        path, nxt, margin = ssd_oracle.accept_tree(logits, draft, tokens, parent, mode=1, seed=123, step=step)
        m1 = abs(2.0 * u - 1.0)
        if u < 0.5:
            u2 = ssd_oracle.uniform(123, step, 3)
            v = int(np.floor(4.0 * u2))
            m2 = min(4.0 * u2 - v, v + 1 - 4.0 * u2)
            assert (path, nxt) == ([0, 1], v)
            seen["accepted"] += 1
        else:
            u2 = ssd_oracle.uniform(123, step, 1)
            v = 2 if u2 < 0.5 else 3
            m2 = min(2.0 * u2 - (v - 2), (v - 1) - 2.0 * u2)
            assert (path, nxt) == ([0], v)
            seen["refused"] += 1
        assert abs(margin - min(m1, m2)) <= 1e-12, (step, margin, m1, m2)
        assert margin > 1e-6  # none of these 24-bit draws sits on a threshold
    assert seen["accepted"] >= 10 and seen["refused"] >= 10


def test_min_margin_shrinks_to_the_distance_of_a_near_threshold_draw():
    """A proposal probability chosen so that u * q[x] misses r[x] by a known relative amount: the oracle must
    report exactly that amount (a margin that came out too small would make the parity tests forgive real
    mismatches, one that came out too large would hide fragile draws)."""
    V = 4
    logits = np.zeros((2, V), dtype=np.float32)
    tokens, parent = [3, 0], [-1, 0]
    for step, eps in ((0, 2.0 ** -20), (1, -2.0 ** -20), (2, 2.0 ** -12)):
        u = ssd_oracle.uniform(9, step, 2)
        q0 = np.float32(0.25 * (1.0 + eps) / u)          # u * q0 = (1 + eps) / 4 up to the rounding of q0 to fp32
        if not (0.0 < q0 <= 1.0):
            continue
        draft = np.zeros((2, V), dtype=np.float32)
        draft[1] = [q0, 1.0 - q0, 0.0, 0.0]
        path, nxt, margin = ssd_oracle.accept_tree(logits, draft, tokens, parent, mode=1, seed=9, step=step)
        rel = abs(u * float(q0) - 0.25) / 0.25           # with the fp32 value of q0 the oracle was given
        assert len(path) == (2 if u * float(q0) < 0.25 else 1)
        assert margin <= rel + 1e-15
        if margin < rel - 1e-15:                          # then the extra draw was the closer call
            assert margin >= 0.0
        else:
            assert abs(margin - rel) <= 1e-15
