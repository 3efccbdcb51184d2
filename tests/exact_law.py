"""Exact output law of a verifier, obtained by driving its sampling mode through every decision.

A verifier consumes one acceptance uniform per tested node and compares it with a threshold
(``u < thr``).  Its outcome is therefore a decision tree over the uniforms.  ``outcomes`` walks
that tree: it forces a prefix of decisions by setting the consumed uniforms to 0 (accept) or to
the largest float below 1 (reject), reads the verifier's own trace to learn which node is
consulted next and with which threshold, and branches with probabilities thr and 1 - thr.  The
leaves carry the accepted node and the distribution the bonus token is drawn from, so the full
law of the emitted tokens follows without Monte Carlo.
"""
from __future__ import annotations

import itertools

import numpy as np

ACCEPT_U = np.float32(0.0)
REJECT_U = np.nextafter(np.float32(1.0), np.float32(0.0))


def outcomes(verify, make_inputs, N):
    """verify(inp, want_residual=True) -> result with .trace/.accepted_node/.residual (B=1).
    make_inputs(u_accept[1,N]) -> inputs.  Yields (probability, accepted_node, residual[V], trace)."""
    out = []

    def rec(prefix, prob):
        u = np.full((1, N), ACCEPT_U, np.float32)
        for node, acc in prefix:
            u[0, node] = ACCEPT_U if acc else REJECT_U
        res = verify(make_inputs(u), want_residual=True)
        assert res.status[0] == 0
        tr = res.trace[0]
        for (node, acc), (tn, thr, tacc) in zip(prefix, tr):
            assert tn == node
            if tacc != acc:      # a forced decision the threshold does not allow (mass < 6e-8)
                return
        if len(tr) > len(prefix):
            node, thr, _ = tr[len(prefix)]
            if thr > 0.0:
                rec(prefix + [(node, True)], prob * min(thr, 1.0))
            if thr < 1.0:
                rec(prefix + [(node, False)], prob * (1.0 - thr))
            return
        out.append((prob, int(res.accepted_node[0]), res.residual[0].copy(), list(tr)))

    rec([], 1.0)
    return out


def softmax64(z):
    z = np.asarray(z, np.float64)
    e = np.exp(z - z.max(-1, keepdims=True))
    return e / e.sum(-1, keepdims=True)


class ContextModel:
    """Context-dependent toy target / draft models on a tiny vocabulary.

    Logits are float32 so that the verifier and this table see the same numbers; the law of a
    context is the float64 softmax of its float32 logits divided by the temperature."""

    def __init__(self, V, max_len, seed, temperature=1.0, spread=1.5, truncate=None):
        rng = np.random.default_rng(seed)
        self.V, self.T = V, float(temperature)
        self.truncate = truncate      # optional callable(z float64[V], T) -> law, for top-k / top-p
        self.zp, self.zq = {}, {}
        for L in range(max_len + 1):
            for ctx in itertools.product(range(V), repeat=L):
                zq = (spread * rng.standard_normal(V)).astype(np.float32)
                self.zq[ctx] = zq
                self.zp[ctx] = (zq + rng.standard_normal(V).astype(np.float32)).astype(np.float32)

    def _law(self, z):
        if self.truncate is not None:
            return self.truncate(z.astype(np.float64), self.T)
        return softmax64(z.astype(np.float64) / self.T)

    def p(self, ctx):
        return self._law(self.zp[tuple(ctx)])

    def q(self, ctx):
        return self._law(self.zq[tuple(ctx)])


def node_contexts(parent, token):
    ctx = [()]
    for i in range(1, len(parent)):
        ctx.append(ctx[int(parent[i])] + (int(token[i]),))
    return ctx


def emitted_law(verify, make_tree_inputs, model: ContextModel, parent, total_len):
    """Law of the first ``total_len`` tokens produced by: draft a random tree from q, verify it,
    emit path + bonus, then continue sampling from p.  Returns {string: probability}."""
    N, V = len(parent), model.V
    law = {}
    for toks in itertools.product(range(V), repeat=N - 1):
        token = np.array((0,) + toks, np.int32)
        ctx = node_contexts(parent, token)
        p_tree = 1.0
        for i in range(1, N):
            p_tree *= model.q(ctx[int(parent[i])])[token[i]]
        if p_tree == 0.0:
            continue
        logits_p = np.stack([model.zp[c] for c in ctx])[None]
        logits_q = np.stack([model.zq[c] for c in ctx])[None]
        mk = lambda u: make_tree_inputs(logits_p, logits_q, token[None], u)
        for prob, node, residual, _ in outcomes(verify, mk, N):
            base = ctx[node]
            for y in range(V):
                if residual[y] == 0.0:
                    continue
                _extend(law, model, base + (y,), p_tree * prob * residual[y], total_len)
    return law


def _extend(law, model, s, mass, total_len):
    if len(s) == total_len:
        law[s] = law.get(s, 0.0) + mass
        return
    pn = model.p(s)
    for y in range(model.V):
        _extend(law, model, s + (y,), mass * pn[y], total_len)


def target_law(model: ContextModel, total_len):
    law = {}
    _extend(law, model, (), 1.0, total_len)
    return law
