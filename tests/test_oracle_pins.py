"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle.

P1  losslessness (Definition 3.2 and Section 5: OT-based traversal and delayed trees preserve the
    target law; Traversal Verification is lossless too) by exact enumeration on tiny vocabularies
P3  one-path Traversal == block verification (Section 3.2), which beats naive (Section 3.1)
P4  depth-1 Traversal == SpecInfer decisions
P5  k = 1 SpecInfer == naive speculative sampling; acceptance = sum min(p,q) = 1 - L1/2 (Section 5)
P6  SpecInfer acceptance rate == Algorithm 9
P7  SpecInfer branching with uniform child choice == Algorithm 14
P8  invariants
plus a coarse brute-force grid over the uniforms themselves, and a negative control showing that
the enumeration rejects a verifier with a dropped residual.
"""
import itertools
import math

import numpy as np
import pytest

import oracle
from oracle import TreeInputs
from paper_2602_16994_b200.synth import delayed_tree, children_lists
from tests.exact_law import (ContextModel, emitted_law, target_law, outcomes, softmax64,
                             ACCEPT_U, REJECT_U)


def tree_inputs(logits_p, logits_q, token, u_accept, u_bonus=None, parent=None, T=1.0, top_k=0, top_p=1.0):
    B, N, V = logits_p.shape
    if u_bonus is None:
        u_bonus = np.full((B, N), 0.5, np.float32)
    return TreeInputs(np.asarray(logits_p, np.float32), np.asarray(logits_q, np.float32), parent,
                      np.asarray(token, np.int32), np.asarray(u_accept, np.float32),
                      np.asarray(u_bonus, np.float32), temperature=T, top_k=top_k, top_p=top_p)


VERIFIERS = {"specinfer": oracle.verify_specinfer, "traversal": oracle.verify_traversal}


# ---------------------------------------------------------------------------------------------
# P1 losslessness
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("algo", ["specinfer", "traversal"])
@pytest.mark.parametrize("V,K,L1,L2,T", [
    (2, 1, 0, 3, 1.0),     # one path
    (3, 2, 0, 2, 1.0),     # root-branched
    (2, 3, 0, 2, 1.0),     # three paths, many duplicate siblings
    (3, 2, 1, 1, 1.0),     # delayed: trunk then branches
    (2, 2, 1, 2, 1.0),     # delayed, deeper branches
    (2, 2, 2, 1, 0.7),     # delayed, temperature != 1
    (3, 3, 0, 1, 1.3),     # wide and flat
])
def test_p1_output_law_is_target_law(algo, V, K, L1, L2, T):
    parent, depth = delayed_tree(K, L1, L2)
    D = int(depth.max())
    model = ContextModel(V, D, seed=100 * V + 10 * K + L1 + L2, temperature=T)
    mk = lambda lp, lq, tok, u: tree_inputs(lp, lq, tok, u, parent=parent, T=T)
    law = emitted_law(VERIFIERS[algo], mk, model, parent, D + 1)
    ref = target_law(model, D + 1)
    assert abs(sum(law.values()) - 1.0) < 1e-9
    worst = max(abs(law.get(s, 0.0) - ref[s]) for s in ref)
    assert worst < 2e-7, worst          # float32 uniforms cap the forced-reject branch at 6e-8


@pytest.mark.parametrize("algo", ["specinfer", "traversal"])
@pytest.mark.parametrize("top_k,top_p", [(2, 1.0), (0, 0.7)])
def test_p1_lossless_under_truncation(algo, top_k, top_p):
    """With top-k / top-p applied to both models the verifiers reproduce the truncated target law;
    draft tokens outside the target's support and target mass outside the draft's are exercised.
    (The truncated row law itself is pinned in test_oracle_rows.)"""
    V, K, L1, L2, T = 4, 2, 1, 1, 0.9
    parent, depth = delayed_tree(K, L1, L2)
    D = int(depth.max())
    trunc = lambda z, temp: oracle.row_probs(z, temp, top_k, top_p)[0]
    model = ContextModel(V, D, seed=77, temperature=np.float32(T), truncate=trunc)
    mk = lambda lp, lq, tok, u: tree_inputs(lp, lq, tok, u, parent=parent, T=T, top_k=top_k, top_p=top_p)
    law = emitted_law(VERIFIERS[algo], mk, model, parent, D + 1)
    ref = target_law(model, D + 1)
    assert min(ref.values()) == 0.0                  # truncation really removes strings
    assert max(abs(law.get(s, 0.0) - ref[s]) for s in ref) < 2e-7


def test_p1_negative_control_dropped_residual_is_caught():
    """The enumeration has teeth: a verifier that draws the correction from p instead of the
    residual (a dropped term) does not reproduce the target law."""
    V, K, L = 3, 1, 2
    parent, depth = delayed_tree(K, 0, L)
    model = ContextModel(V, L, seed=5)

    def broken(inp, want_residual=True):
        good = oracle.verify_specinfer(inp, want_residual=True)
        node = int(good.accepted_node[0])
        z = inp.target_logits[0, node].astype(np.float64)
        good.residual[0] = softmax64(z)        # forget (p - q)+
        return good

    mk = lambda lp, lq, tok, u: tree_inputs(lp, lq, tok, u, parent=parent)
    law = emitted_law(broken, mk, model, parent, L + 1)
    ref = target_law(model, L + 1)
    assert max(abs(law.get(s, 0.0) - ref[s]) for s in ref) > 1e-3


# ---------------------------------------------------------------------------------------------
# brute force over the uniforms themselves (coarse grid), tying the trace-driven law to how the
# uniforms are really consumed, bonus uniform of the stop node included
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("algo", ["specinfer", "traversal"])
def test_uniform_grid_matches_exact_law(algo):
    V, M = 3, 40
    parent, _ = delayed_tree(2, 0, 1)               # root with two leaf children
    rng = np.random.default_rng(3)
    lp = rng.standard_normal((1, 3, V)).astype(np.float32)
    lq = rng.standard_normal((1, 3, V)).astype(np.float32)
    token = np.array([[0, 1, 2]], np.int32)
    grid = (np.arange(M, dtype=np.float64) + 0.5) / M
    g = np.array(list(itertools.product(grid, repeat=3)), np.float32)        # u1, u2, u_bonus
    B = g.shape[0]
    ua = np.zeros((B, 3), np.float32); ua[:, 1] = g[:, 0]; ua[:, 2] = g[:, 1]
    ub = np.repeat(g[:, 2:3], 3, axis=1)
    inp = tree_inputs(np.repeat(lp, B, 0), np.repeat(lq, B, 0), np.repeat(token, B, 0), ua, ub, parent)
    res = VERIFIERS[algo](inp)
    emp = {}
    for b in range(B):
        key = (int(res.accepted_node[b]), int(res.bonus_token[b]))
        emp[key] = emp.get(key, 0.0) + 1.0 / B
    exact = {}
    mk = lambda u: tree_inputs(lp, lq, token, u, parent=parent)
    for prob, node, residual, _ in outcomes(VERIFIERS[algo], mk, 3):
        for y in range(V):
            exact[(node, y)] = exact.get((node, y), 0.0) + prob * residual[y]
    for key in set(emp) | set(exact):
        assert abs(emp.get(key, 0.0) - exact.get(key, 0.0)) < 4.0 / M


# ---------------------------------------------------------------------------------------------
# P5: k = 1 SpecInfer is naive speculative sampling
# ---------------------------------------------------------------------------------------------
def test_p5_single_path_specinfer_is_naive():
    V, L = 7, 4
    rng = np.random.default_rng(11)
    parent, _ = delayed_tree(1, 0, L)
    N = L + 1
    lp = rng.standard_normal((1, N, V)).astype(np.float32) * 1.5
    lq = rng.standard_normal((1, N, V)).astype(np.float32) * 1.5
    p, q = softmax64(lp[0]), softmax64(lq[0])
    token = np.array([[0] + list(rng.integers(0, V, L))], np.int32)
    mk = lambda u: tree_inputs(lp, lq, token, u, parent=parent)
    outs = outcomes(oracle.verify_specinfer, mk, N)
    surv = 1.0
    by_node = {node: (prob, res) for prob, node, res, _ in outs}
    assert len(by_node) == len(outs)
    for a in range(N):
        if a < L:
            x = token[0, a + 1]
            r = min(1.0, p[a, x] / q[a, x])
            resid = np.maximum(p[a] - q[a], 0.0); resid /= resid.sum()
            if r < 1.0:
                assert by_node[a][0] == pytest.approx(surv * (1 - r), abs=1e-12)
                np.testing.assert_allclose(by_node[a][1], resid, atol=1e-12)
            else:
                assert a not in by_node          # a ratio of 1 cannot be rejected
            surv *= r
        else:
            assert by_node[a][0] == pytest.approx(surv, abs=1e-12)
            np.testing.assert_allclose(by_node[a][1], p[a], atol=1e-12)
    # acceptance rate over the draft token: sum_x q(x) min(1, p/q) = sum min(p,q) = 1 - L1/2
    for a in range(L):
        acc = 0.0
        for x in range(V):
            tok = token.copy(); tok[0, a + 1] = x
            res = oracle.verify_specinfer(tree_inputs(lp, lq, tok, np.zeros((1, N), np.float32), parent=parent))
            thr = dict((n, t) for n, t, _ in res.trace[0])
            # with u = 0 the walk reaches node a+1 only if the earlier nodes accept; read the table instead
            ratio, _, _, _ = oracle.specinfer_tables(tree_inputs(lp, lq, tok, np.zeros((1, N), np.float32), parent=parent))
            acc += q[a, x] * ratio[0, a + 1]
            if a + 1 in thr:
                assert thr[a + 1] == pytest.approx(ratio[0, a + 1], abs=0)
        assert acc == pytest.approx(np.minimum(p[a], q[a]).sum(), abs=1e-12)
        assert acc == pytest.approx(1.0 - 0.5 * np.abs(p[a] - q[a]).sum(), abs=1e-12)


# ---------------------------------------------------------------------------------------------
# P6: SpecInfer acceptance rate against Algorithm 9
# ---------------------------------------------------------------------------------------------
def algorithm9_acceptance(p, q, k):
    """SpecInfer acceptance rate, closed form of Algorithm 9 (appendix on OTLP acceptances)."""
    p = p.copy()
    p_rej, m = 1.0, np.ones_like(p)
    for _ in range(k):
        r = np.minimum(p, q).sum()
        p_rej *= (1.0 - r)
        if r < 1.0:
            m = m * (1.0 - np.maximum(q - p, 0.0) / (1.0 - r))
        res = np.maximum(p - q, 0.0)
        if res.sum() > 0:
            p = res / res.sum()
    return (1.0 - p_rej) + p_rej * float((p * (1.0 - m)).sum())


@pytest.mark.parametrize("V,k", [(3, 1), (3, 2), (4, 3), (5, 2)])
def test_p6_specinfer_acceptance_rate_matches_algorithm9(V, k):
    rng = np.random.default_rng(40 + V + k)
    parent, _ = delayed_tree(k, 0, 1)
    N = k + 1
    lp = rng.standard_normal((1, N, V)).astype(np.float32) * 1.2
    lq = rng.standard_normal((1, N, V)).astype(np.float32) * 1.2
    p, q = softmax64(lp[0, 0]), softmax64(lq[0, 0])
    alpha = 0.0
    for xs in itertools.product(range(V), repeat=k):
        token = np.array([(0,) + xs], np.int32)
        w = float(np.prod([q[x] for x in xs]))
        mk = lambda u: tree_inputs(lp, lq, token, u, parent=parent)
        for prob, node, residual, _ in outcomes(oracle.verify_specinfer, mk, N):
            if node != 0:
                alpha += w * prob
            else:
                alpha += w * prob * sum(residual[y] for y in set(xs))
    assert alpha == pytest.approx(algorithm9_acceptance(p, q, k), abs=1e-12)


# ---------------------------------------------------------------------------------------------
# P7: branching probabilities against Algorithm 14 (uniform child selection = random order)
# ---------------------------------------------------------------------------------------------
def algorithm14_branching(p, q, xs):
    """B(f, xs, t) for every distinct child token t: the DP of Algorithm 14 over sub-multisets.
    After i rejections the next test uses p_i, i.e. the ratio min(1, p_i / q)."""
    k = len(xs)
    ps = [p.copy()]
    for _ in range(k):
        res = np.maximum(ps[-1] - q, 0.0)
        ps.append(res / res.sum() if res.sum() > 0 else ps[-1].copy())
    a = [np.minimum(1.0, np.where(q > 0, ps[i] / np.where(q > 0, q, 1.0), 1.0)) for i in range(k)]

    from functools import lru_cache

    @lru_cache(None)
    def B(S, x):                      # S: sorted tuple of remaining child tokens
        i = k - len(S)
        if not S:
            return float(ps[k][x])
        tot = 0.0
        for j, t in enumerate(S):
            rest = S[:j] + S[j + 1:]
            tot += a[i][t] * (1.0 if t == x else 0.0) + (1.0 - a[i][t]) * B(rest, x)
        return tot / len(S)

    return {x: B(tuple(sorted(xs)), x) for x in set(xs)}


@pytest.mark.parametrize("xs", [(0, 1), (2, 2), (0, 1, 2), (1, 1, 3), (3, 0, 3)])
def test_p7_branching_matches_algorithm14(xs):
    V, k = 4, len(xs)
    rng = np.random.default_rng(70 + sum(xs))
    parent, _ = delayed_tree(k, 0, 1)
    N = k + 1
    lp = rng.standard_normal((1, N, V)).astype(np.float32)
    lq = rng.standard_normal((1, N, V)).astype(np.float32)
    p, q = softmax64(lp[0, 0]), softmax64(lq[0, 0])
    perms = list(itertools.permutations(range(k)))
    got = {x: 0.0 for x in set(xs)}
    for perm in perms:
        order = [xs[i] for i in perm]
        token = np.array([[0] + order], np.int32)
        mk = lambda u: tree_inputs(lp, lq, token, u, parent=parent)
        for prob, node, residual, _ in outcomes(oracle.verify_specinfer, mk, N):
            for x in got:
                if node != 0:
                    got[x] += prob * (1.0 if order[node - 1] == x else 0.0) / len(perms)
                else:
                    got[x] += prob * residual[x] / len(perms)
    want = algorithm14_branching(p, q, xs)
    for x in got:
        assert got[x] == pytest.approx(want[x], abs=1e-12)


# ---------------------------------------------------------------------------------------------
# P3: one-path Traversal is block verification, and block verification beats naive
# ---------------------------------------------------------------------------------------------
def block_verification_reference(p, q, xs):
    """Block verification on one path, written from its definition: weights
    w_i = min(1, w_{i-1} p_i(x_i)/q_i(x_i)); test the leaf with w_L; a node reached after its
    child was rejected is tested with S/(S + 1 - w), S = sum (w p - q)+; correction from
    norm((w p - q)+).  Returns P(tau = i) for i = 0..L and the correction laws."""
    L = len(xs)
    w = [1.0]
    for i in range(L):
        w.append(min(1.0, w[i] * p[i, xs[i]] / q[i, xs[i]]))
    prob_tau, laws = np.zeros(L + 1), [None] * (L + 1)
    reach = 1.0
    prob_tau[L] = reach * w[L]; laws[L] = p[L]; reach *= 1 - w[L]
    for i in range(L - 1, -1, -1):
        r = np.maximum(w[i] * p[i] - q[i], 0.0)
        S = r.sum()
        h = S / (S + 1.0 - w[i]) if S > 0 else (1.0 if w[i] >= 1 else 0.0)
        prob_tau[i] = reach * h
        laws[i] = r / S if S > 0 else p[i]
        reach *= 1 - h
    return prob_tau, laws


def test_p3_single_path_traversal_is_block_verification_and_beats_naive():
    """Per path: Traversal == block verification.  Over paths drawn from q: E[tau] of block
    verification is at least that of naive speculative sampling (Section 3.1)."""
    V, L = 4, 3
    rng = np.random.default_rng(21)
    parent, _ = delayed_tree(1, 0, L)
    N = L + 1
    strictly = 0
    for trial in range(6):
        lp = rng.standard_normal((1, N, V)).astype(np.float32) * 1.5
        lq = rng.standard_normal((1, N, V)).astype(np.float32) * 1.5
        p, q = softmax64(lp[0]), softmax64(lq[0])
        e_bv = e_naive = 0.0
        for xs in itertools.product(range(V), repeat=L):
            token = np.array([(0,) + xs], np.int32)
            w_path = float(np.prod([q[i, xs[i]] for i in range(L)]))
            mk = lambda u: tree_inputs(lp, lq, token, u, parent=parent)
            got = np.zeros(N)
            want, laws = block_verification_reference(p, q, xs)
            for prob, node, residual, _ in outcomes(oracle.verify_traversal, mk, N):
                got[node] += prob
                np.testing.assert_allclose(residual, laws[node], atol=1e-12)
            np.testing.assert_allclose(got, want, atol=1e-12)
            naive = np.zeros(N)
            for prob, node, _, _ in outcomes(oracle.verify_specinfer, mk, N):
                naive[node] += prob
            e_bv += w_path * (got * np.arange(N)).sum()
            e_naive += w_path * (naive * np.arange(N)).sum()
        assert e_bv >= e_naive - 1e-12
        strictly += e_bv > e_naive + 1e-9
    assert strictly > 0


def test_p3_negative_control_literal_reading_of_block_verification_is_not_lossless():
    """Section 3.1's paragraph read literally -- accept every node independently with probability w_i,
    return the deepest accepted node, correct from norm((w p - q)+) -- does not reproduce the target
    law; the enumeration tells the two readings apart (the oracle's reading passes P1 above)."""
    V, L = 3, 2
    model = ContextModel(V, L, seed=8)
    law = {}
    for xs in itertools.product(range(V), repeat=L):
        ctx = [tuple(xs[:i]) for i in range(L + 1)]
        p = [model.p(c) for c in ctx]; q = [model.q(c) for c in ctx]
        w_path = float(np.prod([q[i][xs[i]] for i in range(L)]))
        w = [1.0]
        for i in range(L):
            w.append(min(1.0, w[i] * p[i][xs[i]] / q[i][xs[i]]))
        for tau in range(L, -1, -1):
            # tau = deepest accepted node: node tau accepted (the root always), all deeper ones not
            pr = (w[tau] if tau > 0 else 1.0) * float(np.prod([1 - w[j] for j in range(tau + 1, L + 1)]))
            if tau == L:
                corr = p[L]
            else:
                r = np.maximum(w[tau] * p[tau] - q[tau], 0.0)
                corr = r / r.sum() if r.sum() > 0 else p[tau]
            for y in range(V):
                s = tuple(xs[:tau]) + (y,)
                mass = w_path * pr * corr[y]
                # continue from p up to length L + 1
                def ext(s, m):
                    if len(s) == L + 1:
                        law[s] = law.get(s, 0.0) + m
                        return
                    pn = model.p(s)
                    for z in range(V):
                        ext(s + (z,), m * pn[z])
                ext(s, mass)
    ref = target_law(model, L + 1)
    assert abs(sum(law.values()) - 1.0) < 1e-9
    assert max(abs(law.get(s, 0.0) - ref[s]) for s in ref) > 1e-3


def test_traversal_tables_incoming_weights_on_paths_and_leaves():
    """w_in of oracle.traversal_tables: on a path it is block verification's weight list
    w_i = min(1, w_{i-1} p(x_i)/q(x_i)) (Section 3.1); at any leaf, reached after its earlier siblings'
    subtrees were rejected, it is the threshold the leaf is tested with in the enumerated decision
    tree of the sampling-mode verifier (a leaf's final weight is the weight it was handed)."""
    V, L = 4, 3
    rng = np.random.default_rng(61)
    parent, _ = delayed_tree(1, 0, L)
    N = L + 1
    lp = rng.standard_normal((1, N, V)).astype(np.float32) * 1.5
    lq = rng.standard_normal((1, N, V)).astype(np.float32) * 1.5
    p, q = softmax64(lp[0]), softmax64(lq[0])
    for xs in itertools.product(range(V), repeat=L):
        token = np.array([(0,) + xs], np.int32)
        w = [1.0]
        for i in range(L):
            w.append(min(1.0, w[i] * p[i, xs[i]] / q[i, xs[i]]))
        w_in, w_fin, _, st = oracle.traversal_tables(tree_inputs(lp, lq, token, np.zeros((1, N), np.float32), parent=parent))
        np.testing.assert_allclose(w_in[0], w, atol=1e-13)
        assert w_fin[0, L] == pytest.approx(w[L], abs=1e-13)
    # branched trees: every leaf's incoming weight against the decision tree of the sampling mode
    for K, L1, L2, seed in [(3, 0, 1, 1), (2, 1, 1, 2), (2, 0, 2, 3), (3, 1, 1, 4)]:
        parent, depth = delayed_tree(K, L1, L2)
        N = len(parent)
        rng = np.random.default_rng(200 + seed)
        lp = rng.standard_normal((1, N, V)).astype(np.float32) * 1.2
        lq = rng.standard_normal((1, N, V)).astype(np.float32) * 1.2
        token = np.concatenate([[0], rng.integers(0, V, N - 1)]).astype(np.int32)[None]
        mk = lambda u: tree_inputs(lp, lq, token, u, parent=parent)
        w_in, w_fin, _, _ = oracle.traversal_tables(mk(np.zeros((1, N), np.float32)))
        leaves = [a for a in range(1, N) if a not in set(parent[1:].tolist())]
        seen = {}
        for prob, node, residual, trace in outcomes(oracle.verify_traversal, mk, N):
            for tn, thr, _ in trace:
                seen.setdefault(tn, thr)
                assert seen[tn] == pytest.approx(thr, abs=1e-13)      # weights do not depend on the decisions
        for a in leaves:
            if a in seen:
                assert w_in[0, a] == pytest.approx(seen[a], abs=1e-13)
                assert w_fin[0, a] == pytest.approx(seen[a], abs=1e-13)
        assert any(a in seen for a in leaves)
        for a in range(1, N):
            if a in seen:
                assert w_fin[0, a] == pytest.approx(seen[a], abs=1e-13)


def test_traversal_weight_one_is_stable_under_small_residual_masses():
    """A node of weight exactly 1 keeps weight exactly 1 through every rejected child subtree, however
    small the residual masses are: w' = S / (S + 1 - w) = 1 (Section 3.1's recursion at w = 1).
    Four children with the same dominant token in a near-greedy law: S is about 1e-5 at every step."""
    V = 64
    rng = np.random.default_rng(4)
    parent, _ = delayed_tree(4, 0, 1)
    N = 5
    base = rng.standard_normal(V).astype(np.float32)
    base[7] += 12.0                                     # one dominant token in both laws
    lq = np.repeat(base[None, None], N, 1).astype(np.float32)
    lp = lq.copy(); lp[0, 0, 7] += 1.5                  # p even more peaked: p(7) > q(7), ratio clipped to 1
    token = np.array([[0, 7, 7, 7, 7]], np.int32)
    w_in, w_fin, _, st = oracle.traversal_tables(tree_inputs(lp, lq, token, np.zeros((1, N), np.float32), parent=parent))
    assert st[0] == 0
    assert w_fin[0, 0] == 1.0                           # exactly
    assert w_in[0, 1] == 1.0


# ---------------------------------------------------------------------------------------------
# P4: on a depth-1 tree Traversal and SpecInfer take the same decisions
# ---------------------------------------------------------------------------------------------
def test_p4_depth_one_traversal_equals_specinfer():
    V, k, B = 9, 4, 500
    rng = np.random.default_rng(31)
    parent, _ = delayed_tree(k, 0, 1)
    N = k + 1
    lp = rng.standard_normal((B, N, V)).astype(np.float32) * 2
    lq = rng.standard_normal((B, N, V)).astype(np.float32) * 2
    token = np.concatenate([np.zeros((B, 1), np.int32), rng.integers(0, V, (B, k)).astype(np.int32)], 1)
    ua = rng.random((B, N), dtype=np.float32); ub = rng.random((B, N), dtype=np.float32)
    inp = tree_inputs(lp, lq, token, ua, ub, parent)
    a, b = oracle.verify_specinfer(inp, True), oracle.verify_traversal(inp, True)
    np.testing.assert_array_equal(a.accepted_node, b.accepted_node)
    np.testing.assert_array_equal(a.bonus_token, b.bonus_token)
    np.testing.assert_allclose(a.residual, b.residual, atol=1e-12)
    assert (a.accepted_node > 0).any() and (a.accepted_node == 0).any()


# ---------------------------------------------------------------------------------------------
# P8: invariants on random inputs
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("algo", ["specinfer", "traversal"])
@pytest.mark.parametrize("K,L1,L2", [(2, 0, 3), (4, 2, 4), (3, 1, 2)])
def test_p8_invariants(algo, K, L1, L2):
    V, B = 50, 64
    rng = np.random.default_rng(K * 100 + L1 * 10 + L2)
    parent, depth = delayed_tree(K, L1, L2)
    N = len(parent)
    lq = (3 * rng.standard_normal((B, N, V))).astype(np.float32)
    lp = (lq + rng.standard_normal((B, N, V))).astype(np.float32)
    q = softmax64(lq)
    token = np.zeros((B, N), np.int32)
    for b in range(B):
        for c in range(1, N):
            token[b, c] = rng.choice(V, p=q[b, parent[c]])
    ua = rng.random((B, N), dtype=np.float32); ub = rng.random((B, N), dtype=np.float32)
    inp = tree_inputs(lp, lq, token, ua, ub, parent)
    res = VERIFIERS[algo](inp, True)
    assert (res.status == 0).all()
    assert (res.residual >= 0).all()
    np.testing.assert_allclose(res.residual.sum(1), 1.0, atol=1e-12)
    for b in range(B):
        a = int(res.accepted_node[b])
        assert res.accept_len[b] == depth[a]
        path = []
        while a != 0:
            path.append(int(token[b, a])); a = int(parent[a])
        path.reverse()
        assert list(res.out_tokens[b, :len(path)]) == path
        assert res.out_tokens[b, len(path)] == res.bonus_token[b]
        assert (res.out_tokens[b, len(path) + 1:] == -1).all()
        assert res.residual[b, res.bonus_token[b]] > 0        # zero-probability tokens never emitted
        for node, thr, acc in res.trace[b]:
            assert 0.0 <= thr <= 1.0 + 1e-12       # S/(S+1-w) may round a hair above 1
            assert acc == (ua[b, node] < thr)
    if algo == "traversal":
        w_in, w_fin, bonus_all, st = oracle.traversal_tables(inp)
        assert (st == 0).all()
        assert ((w_in >= 0) & (w_in <= 1 + 1e-12)).all() and ((w_fin >= 0) & (w_fin <= 1 + 1e-12)).all()
        np.testing.assert_allclose(w_fin[:, 0], 1.0, atol=1e-12)      # the root is always accepted
        # the accepted node is the first in DFS post-order whose uniform is below its final weight
        ch = children_lists(parent)
        order = []
        def post(a):
            for c in ch[a]:
                post(c)
            order.append(a)
        post(0)
        for b in range(B):
            first = next(a for a in order if a == 0 or ua[b, a] < w_fin[b, a])
            assert first == res.accepted_node[b]
            assert bonus_all[b, first] == res.bonus_token[b]
    else:
        ratio, nxt, bonus_all, st = oracle.specinfer_tables(inp)
        assert (st == 0).all()
        for b in range(B):
            a = 0
            while nxt[b, a] >= 0:
                a = int(nxt[b, a])
            assert a == res.accepted_node[b]
            assert bonus_all[b, a] == res.bonus_token[b]
            for node, thr, acc in res.trace[b]:
                assert ratio[b, node] == thr


def test_bad_inputs_are_reported_per_sequence():
    V = 5
    parent, _ = delayed_tree(1, 0, 2)
    lp = np.zeros((2, 3, V), np.float32); lq = np.zeros((2, 3, V), np.float32)
    token = np.array([[0, 1, 2], [0, 7, 2]], np.int32)           # second sequence: token >= V
    u = np.full((2, 3), 0.5, np.float32)
    res = oracle.verify_specinfer(tree_inputs(lp, lq, token, u, u, parent))
    assert res.status[0] == 0 and res.status[1] != 0
    bad_parent = np.array([-1, 2, 1], np.int32)                  # parent[i] >= i
    res = oracle.verify_traversal(tree_inputs(lp[:1], lq[:1], token[:1], u[:1], u[:1], bad_parent))
    assert res.status[0] != 0
