"""Shared helpers of the GPU parity tests: run the oracle and the CUDA library on the same seeded
batch and compare them under the stated rules.

Rules.  Integer outputs (accepted node, path tokens, bonus token) must be identical, except where
the oracle itself says the decision was closer than 1e-6 to its threshold (|u - thr| for an
acceptance test, distance to the CDF boundary as a fraction of the total mass for the bonus draw);
such differences are counted and reported, anything else fails.  Probabilities, residuals, per-node
thresholds, weights and margins must agree within 1e-5 absolute, every entry.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

import oracle
from oracle import TreeInputs
from paper_2602_16994_b200 import binding

MARGIN = 1e-6
PROB_TOL = 1e-5


def assert_thresholds(got, ref, what):
    d = np.abs(np.asarray(got, np.float64) - ref)
    assert d.max(initial=0.0) < PROB_TOL, f"{what} differ by {d.max():.3e}"


def oracle_inputs(batch) -> TreeInputs:
    a = batch.numpy()
    w = batch.workload
    return TreeInputs(a["target_logits"], a["draft_logits"], a["parent"], a["token"], a["u_accept"],
                      a["u_bonus"], temperature=w.temperature, top_k=w.top_k, top_p=w.top_p)


def gpu_verify(batch, algo, **opts):
    w = batch.workload
    fn = binding.verify_specinfer if algo == "specinfer" else binding.verify_traversal
    out = fn(batch.target_logits, batch.draft_logits, batch.parent, batch.token, batch.u_accept,
             batch.u_bonus, w.temperature, w.top_k, w.top_p, **opts)
    torch.cuda.synchronize()
    return out


@dataclass
class Tally:
    decisions: int = 0
    near_margin_mismatches: int = 0
    near_margin_decisions: int = 0
    sequences: int = 0
    rows: int = 0                 # logit rows whose cut (top-k / top-p) was compared
    rows_near_boundary: int = 0   # of those: nucleus boundary within 1e-6 of top_p (the oracle's own margin)
    rows_cut_differs: int = 0     # of those: the device kept a different set (tolerated only near the boundary)
    sequences_set_aside: int = 0  # sequences holding such a row: their outputs are not compared

    def add(self, other):
        for k in vars(self):
            setattr(self, k, getattr(self, k) + getattr(other, k))


def settle_cuts(batch, inp, tally: Tally):
    """Truncating workloads: compare the cut (smallest kept logit) the device chose for every row the
    verifiers read with the oracle's.  A different cut is tolerated only where the oracle says the
    nucleus boundary lies within 1e-6 of top_p; the sequences that hold such a row are returned (their
    distributions legitimately differ there) and counted."""
    w = batch.workload
    B, N, V = inp.shape
    parent = batch.parent.cpu().numpy()
    internal = np.zeros(N, bool); internal[parent[1:]] = True
    bad_seq = np.zeros(B, bool)
    for which, rows in ((0, np.ones(N, bool)), (1, internal)):
        logits = batch.target_logits if which == 0 else batch.draft_logits
        _, st = binding.tree_probs(logits, 0, temperature=w.temperature, top_k=w.top_k, top_p=w.top_p,
                                   want_probs=False)
        torch.cuda.synchronize()
        got_cut = st[..., 5].cpu().numpy().astype(np.float32)
        _, ref, _ = oracle.tree_probs(inp, which, want_probs=False)
        ref_cut = ref[..., 6].astype(np.float32)
        differs = (got_cut != ref_cut) & rows[None, :]
        near = (ref[..., 5] < MARGIN) & rows[None, :]
        assert not (differs & ~near).any(), (
            f"{int((differs & ~near).sum())} rows cut at another logit although the nucleus boundary is "
            f"further than 1e-6 from top_p")
        tally.rows += int(rows.sum()) * B
        tally.rows_near_boundary += int(near.sum())
        tally.rows_cut_differs += int(differs.sum())
        bad_seq |= differs.any(1)
    tally.sequences_set_aside += int(bad_seq.sum())
    return bad_seq


def compare_decisions(ref, got, parent) -> Tally:
    """ref: oracle VerifyResult; got: VerifyOutputs (device).  Raises AssertionError on a real mismatch."""
    t = Tally()
    acc = got.accepted_node.cpu().numpy(); alen = got.accept_len.cpu().numpy()
    toks = got.out_tokens.cpu().numpy(); bonus = got.bonus_token.cpu().numpy()
    status = got.status.cpu().numpy()
    B = acc.shape[0]
    for b in range(B):
        assert ref.status[b] == 0, f"oracle status {ref.status[b]} for sequence {b}"
        assert status[b] == 0, f"device status {status[b]} for sequence {b}"
        trace = ref.trace[b]
        t.decisions += len(trace) + 1
        min_margin = min([m for m in ref.trace_margins[b]], default=1.0)
        t.near_margin_decisions += sum(m < MARGIN for m in ref.trace_margins[b]) + (ref.bonus_margin[b] < MARGIN)
        if acc[b] != ref.accepted_node[b]:
            assert min_margin < MARGIN, (f"sequence {b}: accepted node {acc[b]} != oracle {ref.accepted_node[b]} "
                                         f"with smallest decision margin {min_margin:.3e}")
            t.near_margin_mismatches += 1
            continue
        assert alen[b] == ref.accept_len[b]
        if bonus[b] != ref.bonus_token[b]:
            assert ref.bonus_margin[b] < MARGIN, (f"sequence {b}: bonus {bonus[b]} != oracle {ref.bonus_token[b]} "
                                                  f"with CDF margin {ref.bonus_margin[b]:.3e}")
            t.near_margin_mismatches += 1
            assert (toks[b, :alen[b]] == ref.out_tokens[b, :alen[b]]).all()
            continue
        assert (toks[b] == ref.out_tokens[b]).all(), f"sequence {b}: out_tokens differ"
    return t


def run_oracle(batch, algo, want_residual=False):
    inp = oracle_inputs(batch)
    fn = oracle.verify_specinfer if algo == "specinfer" else oracle.verify_traversal
    res = fn(inp, want_residual)
    ua = inp.u_accept
    res.trace_margins = [[abs(float(ua[b, node]) - thr) for node, thr, _ in res.trace[b]]
                         for b in range(len(res.trace))]
    return inp, res


def check_batch(batch, algo, full=True) -> Tally:
    """Plain call (fast path) and, if ``full``, a call with every optional output, both against the oracle.
    With top-k / top-p the rows' cuts are compared first (``settle_cuts``)."""
    w = batch.workload
    pre = Tally()
    if (0 < w.top_k < w.V) or w.top_p < 1.0:
        if getattr(batch, "_settled", None) is None:       # once per batch: both verifiers read the same rows
            t0 = Tally()
            batch._settled = (settle_cuts(batch, oracle_inputs(batch), t0), t0)
            pre.add(t0)
        bad = batch._settled[0]
        if bad.any():
            batch = batch.select([i for i in range(w.B) if not bad[i]])
            if batch.workload.B == 0:
                return pre
    inp, ref = run_oracle(batch, algo, want_residual=full)
    parent = batch.parent.cpu().numpy()
    tally = compare_decisions(ref, gpu_verify(batch, algo), parent)
    tally.add(pre)
    tally.sequences += batch.workload.B
    if not full:
        return tally
    got = gpu_verify(batch, algo, residual=True, node_thr=True, features=True, margin=True,
                     **({"node_w_in": True} if algo == "traversal" else {}))
    t2 = compare_decisions(ref, got, parent)
    assert t2.near_margin_mismatches == tally.near_margin_mismatches
    B, N, V = inp.shape
    acc = got.accepted_node.cpu().numpy()
    same = (acc == ref.accepted_node) & (got.bonus_token.cpu().numpy() == ref.bonus_token)
    res = got.residual.cpu().numpy().astype(np.float64)
    err = np.abs(res - ref.residual)[same]
    assert err.size == 0 or err.max() < PROB_TOL, f"residual differs by {err.max():.3e}"
    assert np.abs(res[same].sum(1) - 1.0).max(initial=0.0) < 1e-4
    thr = got.node_thr.cpu().numpy().astype(np.float64)
    if algo == "specinfer":
        ratio, nxt, bonus_all, st = oracle.specinfer_tables(inp)
        assert_thresholds(thr, ratio, "thresholds")
    else:
        w_in, w_fin, bonus_all, st = oracle.traversal_tables(inp)
        assert_thresholds(thr, w_fin, "final weights")
        gw = got.node_w_in.cpu().numpy().astype(np.float64)
        assert_thresholds(gw, w_in, "incoming weights")
    # selector features: entropies and top-1 probabilities of the sampling distributions
    feats = got.node_features.cpu().numpy().astype(np.float64)
    _, sp, _ = oracle.tree_probs(inp, 0, want_probs=False)
    _, sq, _ = oracle.tree_probs(inp, 1, want_probs=False)
    internal = np.zeros(N, bool); internal[parent[1:]] = True
    assert np.abs(feats[..., 0] - sp[..., 3]).max() < 1e-4
    assert np.abs(feats[..., 2] - sp[..., 4]).max() < PROB_TOL
    assert np.abs(feats[:, internal, 1] - sq[:, internal, 3]).max(initial=0.0) < 1e-4
    assert np.abs(feats[:, internal, 3] - sq[:, internal, 4]).max(initial=0.0) < PROB_TOL
    mg = got.margin.cpu().numpy()
    ua = inp.u_accept.astype(np.float64)
    ref_thr = ratio if algo == "specinfer" else w_fin
    assert np.abs(mg[:, 1:N] - np.abs(ua[:, 1:] - ref_thr[:, 1:])).max(initial=0.0) < PROB_TOL
    return tally
