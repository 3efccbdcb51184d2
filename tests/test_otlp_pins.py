"""Pins for the second oracle file (otlp_oracle.c): the other OTLP solvers, acceptance rates,
branching probabilities, the block-efficiency sum, divergences and the latency model -- each against
what the paper and the mathematics fix, not against the oracle's own formulas.

S1  every solver is an OTLP solver (Definition 3.2): for i.i.d. children ~ q its output follows p --
    brute force over all child tuples and all uniform outcomes on a grid-free exact enumeration
S2  acceptance rates (Algorithms 6-9) = P(output among the children), from the same enumeration
S3  branching probabilities (Algorithms 11-14) = P(output = token | child list), from the enumeration;
    the uniform-order SpecInfer variant against the average over all child orders
S4  k = 1: SpecTr, SpecInfer and Naive coincide; rho* = 1; NSS acceptance = sum p q
S5  block-efficiency sum = exact E[tau + 1] of the verifier on given tiny trees
S6  divergences against scipy; latency model against a hand-worked case
S7  the top-down walk with NSS / Naive / SpecTr is lossless on a tiny tree (grid over the uniforms)
"""
import itertools

import numpy as np
import pytest
from scipy.special import rel_entr

import oracle
from oracle import TreeInputs
from paper_2602_16994_b200.synth import delayed_tree
from tests.exact_law import ACCEPT_U, REJECT_U, softmax64, outcomes


def random_laws(V, seed, sharp=1.0):
    rng = np.random.default_rng(seed)
    return rng.dirichlet(np.full(V, sharp)), rng.dirichlet(np.full(V, sharp))


# ---------------------------------------------------------------------------------------------
# exact output law of one solver call, written from the solvers' definitions (Appendix B) as a
# decision tree over the uniforms: independent of the oracle's code
# ---------------------------------------------------------------------------------------------
def solver_output_law(solver, p, q, xs):
    """P(output = t | children xs) for t in range(V), straight from Algorithms 1-4."""
    V, k = len(p), len(xs)
    out = np.zeros(V)
    ratio = lambda P, Q: 0.0 if P <= 0 else (1.0 if Q <= 0 else min(1.0, P / Q))
    if solver == "nss":
        return p.copy()
    if solver == "naive":
        a = ratio(p[xs[0]], q[xs[0]])
        res = np.maximum(p - q, 0); res = res / res.sum() if res.sum() > 0 else p
        out[xs[0]] += a
        return out + (1 - a) * res
    if solver == "spectr":
        rho = spectr_rho_reference(p, q, k)
        beta = np.minimum(p / rho, q).sum()
        pacc = 1 - (1 - beta) ** k
        gamma = pacc / beta
        res = np.maximum(p - np.minimum(p / rho, q) * gamma, 0); res = res / res.sum()
        alive = 1.0
        for x in xs:
            a = min(1.0, (p[x] / q[x]) / rho) if q[x] > 0 else (1.0 if p[x] > 0 else 0.0)
            out[x] += alive * a
            alive *= 1 - a
        return out + alive * res
    if solver in ("specinfer", "specinfer_uniform"):
        orders = [tuple(range(k))] if solver == "specinfer" else list(itertools.permutations(range(k)))
        for order in orders:
            P, alive = p.copy(), 1.0 / len(orders)
            for i in order:
                a = ratio(P[xs[i]], q[xs[i]])
                out[xs[i]] += alive * a
                alive *= 1 - a
                R = np.maximum(P - q, 0)
                if R.sum() > 0:
                    P = R / R.sum()
            out += alive * P
        return out
    raise ValueError(solver)


def spectr_rho_reference(p, q, k):
    """rho*: root of 1 - (1 - beta)^k - rho beta on [1, k] by scipy's brentq (another root finder)."""
    from scipy.optimize import brentq
    if k == 1:
        return 1.0
    f = lambda r: 1 - (1 - np.minimum(p / r, q).sum()) ** k - r * np.minimum(p / r, q).sum()
    if f(1.0) <= 0:
        return 1.0
    if f(float(k)) >= 0:
        return float(k)
    return brentq(f, 1.0, float(k), xtol=1e-15, rtol=1e-15)


SOLVERS = ["nss", "naive", "spectr", "specinfer", "specinfer_uniform"]


# ---------------------------------------------------------------------------------------------
# S1: the OTLP property
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("solver", SOLVERS)
@pytest.mark.parametrize("V,k", [(3, 1), (3, 2), (4, 3)])
def test_s1_output_follows_p_for_iid_children(solver, V, k):
    p, q = random_laws(V, 10 * V + k)
    law = np.zeros(V)
    for xs in itertools.product(range(V), repeat=k):
        law += np.prod([q[x] for x in xs]) * solver_output_law(solver, p, q, list(xs))
    np.testing.assert_allclose(law, p, atol=1e-9)       # the reference itself is lossless ...
    # ... and the oracle's branching probabilities agree with it token by token
    for xs in itertools.product(range(V), repeat=k):
        got = oracle.branching(solver, p, q, list(xs))
        want = solver_output_law(solver, p, q, list(xs))
        np.testing.assert_allclose(got, [want[x] for x in xs], atol=1e-10)


def test_s1_spectr_rho_against_another_root_finder():
    for seed in range(20):
        V, k = 5 + seed % 4, 2 + seed % 4
        p, q = random_laws(V, 100 + seed, sharp=0.5)
        assert oracle.spectr_rho(p, q, k) == pytest.approx(spectr_rho_reference(p, q, k), abs=1e-12)
    assert oracle.spectr_rho(p, q, 1) == 1.0


# ---------------------------------------------------------------------------------------------
# S2: acceptance rates = P(output among the children) over i.i.d. children
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("V,k", [(3, 1), (3, 2), (4, 3), (5, 2)])
def test_s2_acceptance_rates_against_enumeration(V, k):
    p, q = random_laws(V, 7 * V + k)
    want = {s: 0.0 for s in ("nss", "naive", "spectr", "specinfer")}
    for xs in itertools.product(range(V), repeat=k):
        w = np.prod([q[x] for x in xs])
        for s in want:
            law = solver_output_law(s, p, q, list(xs))
            want[s] += w * sum(law[t] for t in set(xs))
    got = oracle.acceptance(p, q, k)
    for i, s in enumerate(("nss", "naive", "spectr", "specinfer")):
        assert got[i] == pytest.approx(want[s], abs=1e-10), s
    # closed forms the paper states: Naive at k = 1 is sum min(p,q) = 1 - L1/2 (Section 5)
    a1 = oracle.acceptance(p, q, 1)
    assert a1[1] == pytest.approx(np.minimum(p, q).sum(), abs=1e-14)
    assert a1[1] == pytest.approx(1 - 0.5 * oracle.divergences(p, q)[0], abs=1e-14)
    assert a1[0] == pytest.approx((p * q).sum(), abs=1e-14)


# ---------------------------------------------------------------------------------------------
# S3: uniform-order SpecInfer branching = Algorithm 14, and covers-the-vocabulary sums
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("xs", [(0, 1), (2, 2), (0, 1, 2), (1, 1, 3), (3, 0, 3), (0, 1, 2, 3)])
def test_s3_branching_sums(xs):
    V = 4
    p, q = random_laws(V, 50 + sum(xs))
    for s in SOLVERS:
        b = oracle.branching(s, p, q, list(xs))
        per_token = {x: b[i] for i, x in enumerate(xs)}          # duplicates carry the same value
        for i, x in enumerate(xs):
            assert b[i] == pytest.approx(per_token[x], abs=1e-14)
        total = sum(per_token.values())
        assert total <= 1 + 1e-12
        if set(xs) == set(range(V)):
            assert total == pytest.approx(1.0, abs=1e-10), s     # the children cover the vocabulary


# ---------------------------------------------------------------------------------------------
# S4: k = 1 reductions
# ---------------------------------------------------------------------------------------------
def test_s4_single_child_reductions():
    p, q = random_laws(6, 3)
    for x in range(6):
        b = {s: oracle.branching(s, p, q, [x])[0] for s in SOLVERS}
        assert b["spectr"] == pytest.approx(b["naive"], abs=1e-14)
        assert b["specinfer"] == pytest.approx(b["naive"], abs=1e-14)
        assert b["specinfer_uniform"] == pytest.approx(b["naive"], abs=1e-14)
        assert b["nss"] == pytest.approx(p[x], abs=0)
    a = oracle.acceptance(p, q, 1)
    assert a[2] == pytest.approx(a[1], abs=1e-14) and a[3] == pytest.approx(a[1], abs=1e-14)


# ---------------------------------------------------------------------------------------------
# S5: block-efficiency sum = exact E[tau + 1] of the verifier on a given tree
# ---------------------------------------------------------------------------------------------
def _tree_inputs(lp, lq, token, ua, ub, parent):
    return TreeInputs(np.asarray(lp, np.float32), np.asarray(lq, np.float32), parent, np.asarray(token, np.int32),
                      np.asarray(ua, np.float32), np.asarray(ub, np.float32))


@pytest.mark.parametrize("K,L1,L2", [(2, 0, 2), (2, 1, 1), (3, 0, 1), (1, 0, 3)])
def test_s5_block_efficiency_is_the_verifiers_expected_length(K, L1, L2):
    V = 3
    parent, depth = delayed_tree(K, L1, L2)
    N = len(parent)
    rng = np.random.default_rng(1000 + 100 * K + 10 * L1 + L2)
    for trial in range(4):
        lp = rng.standard_normal((1, N, V)).astype(np.float32) * 1.3
        lq = rng.standard_normal((1, N, V)).astype(np.float32) * 1.3
        token = np.concatenate([[0], rng.integers(0, V, N - 1)]).astype(np.int32)[None]
        ub = np.full((1, N), 0.5, np.float32)
        mk = lambda u: _tree_inputs(lp, lq, token, u, ub, parent)
        inp = mk(np.zeros((1, N), np.float32))
        # SpecInfer (list order): exact law of the oracle verifier pinned in test_oracle_pins
        e_tau = 0.0
        for prob, node, residual, _ in outcomes(oracle.verify_specinfer, mk, N):
            e_tau += prob * depth[node]
        be, reach, br, st = oracle.block_efficiency(inp, "specinfer")
        assert st[0] == 0
        assert be[0] == pytest.approx(1.0 + e_tau, abs=1e-10)
        assert reach[0, 0] == 1.0 and be[0] == pytest.approx(reach[0].sum(), abs=1e-12)
        # the other solvers: expected length from the reference output laws, node by node
        for s in ("nss", "naive", "spectr"):
            be_s, reach_s, _, _ = oracle.block_efficiency(inp, s)
            want = np.zeros(N); want[0] = 1.0
            for a in range(N):
                ch = [c for c in range(a + 1, N) if parent[c] == a]
                if not ch:
                    continue
                p = softmax64(lp[0, a]); q = softmax64(lq[0, a])
                law = solver_output_law(s, p, q, [int(token[0, c]) for c in ch])
                seen = set()
                for c in ch:
                    t = int(token[0, c])
                    want[c] = 0.0 if t in seen else want[a] * law[t]
                    seen.add(t)
            np.testing.assert_allclose(reach_s[0], want, atol=1e-10)
            assert be_s[0] == pytest.approx(want.sum(), abs=1e-10)


# ---------------------------------------------------------------------------------------------
# S6: divergences and the latency model
# ---------------------------------------------------------------------------------------------
def test_s6_divergences_against_scipy():
    p, q = random_laws(50, 9)
    d = oracle.divergences(p, q)
    assert d[0] == pytest.approx(np.abs(p - q).sum(), abs=1e-14)
    assert d[1] == pytest.approx(rel_entr(p, q).sum(), abs=1e-12)
    assert d[2] == pytest.approx(rel_entr(q, p).sum(), abs=1e-12)
    p2 = p.copy(); p2[3] = 0; p2 /= p2.sum()
    d2 = oracle.divergences(p2, q)
    assert np.isfinite(d2[1]) and np.isinf(d2[2])


def test_s6_latency_model_hand_worked():
    # t_q(l) = 1 + l/100, t_p(l) = 10 + l/10; action K=3, L1=2, L2=2 at context 100:
    # trunk t_q(100) + t_q(101); branches t_q(102) + t_q(105); target t_p(100 + 2 + 6)
    t_q = 1 + np.arange(400) / 100.0
    t_p = 10 + np.arange(400) / 10.0
    T = oracle.latency_model(t_q, t_p, 100, [[3, 2, 2], [1, 0, 0], [4, 8, 8]])
    assert T[0] == pytest.approx((2.00 + 2.01) + (2.02 + 2.05) + 20.8, abs=1e-12)
    assert T[1] == pytest.approx(20.0, abs=1e-12)
    want = sum(t_q[100 + j] for j in range(8)) + sum(t_q[108 + 4 * j] for j in range(8)) + t_p[140]
    assert T[2] == pytest.approx(want, abs=1e-12)
    pi = np.array([0.5, 0.25, 0.25]); E = np.array([3.0, 1.0, 5.0])
    assert oracle.tps_estimate(pi, E, T) == pytest.approx((pi * E).sum() / (pi * T).sum(), abs=1e-15)


# ---------------------------------------------------------------------------------------------
# S7: the top-down walk with each solver consumes the uniforms as specified and is lossless
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("solver", ["nss", "naive", "spectr"])
def test_s7_walk_on_a_grid_of_uniforms(solver):
    """Root with two leaf children: a fine grid over (u_1, u_2, u_bonus[root]) must reproduce the
    reference output law of the solver at the root, and a landed child must be moved to."""
    V, M = 3, 24
    parent, _ = delayed_tree(2, 0, 1)
    rng = np.random.default_rng(5)
    lp = rng.standard_normal((1, 3, V)).astype(np.float32)
    lq = rng.standard_normal((1, 3, V)).astype(np.float32)
    token = np.array([[0, 1, 2]], np.int32)
    grid = (np.arange(M, dtype=np.float64) + 0.5) / M
    g = np.array(list(itertools.product(grid, repeat=3)), np.float32)
    B = g.shape[0]
    ua = np.zeros((B, 3), np.float32); ua[:, 1] = g[:, 0]; ua[:, 2] = g[:, 1]
    ub = np.full((B, 3), 0.5, np.float32); ub[:, 0] = g[:, 2]
    inp = TreeInputs(np.repeat(lp, B, 0), np.repeat(lq, B, 0), parent, np.repeat(token, B, 0), ua, ub)
    res = oracle.verify_otlp(inp, solver)
    assert (res.status == 0).all()
    p, q = softmax64(lp[0, 0]), softmax64(lq[0, 0])
    law = solver_output_law(solver, p, q, [1, 2])
    first = res.out_tokens[:, 0]
    for t in range(V):
        assert (first == t).mean() == pytest.approx(law[t], abs=3.0 / M)
    moved = res.accepted_node > 0
    assert (res.accept_len[moved] == 1).all() and (res.accept_len[~moved] == 0).all()
    assert ((first == 1) == (res.accepted_node == 1)).all() and ((first == 2) == (res.accepted_node == 2)).all()
    # at a leaf the walk emits one more token from p(.|leaf) with the leaf's bonus uniform (0.5 here)
    for c in (1, 2):
        sel = res.accepted_node == c
        want, _ = oracle.inverse_cdf(softmax64(lp[0, c]), 0.5)
        assert (res.bonus_token[sel] == want).all() and (res.out_tokens[sel, 1] == want).all()
