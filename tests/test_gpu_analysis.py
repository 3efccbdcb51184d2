"""GPU parity of the offline analysis (spec_tree_analysis, spec_latency_model) against the CPU oracle:
acceptance rates (Algorithms 6-9), divergences, branching probabilities (Algorithms 11-14), the
block-efficiency sum of equation (3), and the forward-time model of equation (8)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_16994_b200 import binding
from paper_2602_16994_b200.synth import WORKLOADS, Workload, make_batch
from tests.parity import PROB_TOL, oracle_inputs

pytestmark = pytest.mark.gpu

SHAPES = [
    Workload("an_v1000_f32", 4, 1000, "f32", 3, 0, 2, 1.0),
    Workload("an_v32000_k4", 3, 32000, "bf16", 4, 1, 2, 1.0),
    Workload("an_v50257_k8_T06", 2, 50257, "bf16", 8, 0, 2, 0.7, temperature=0.6),
    Workload("an_v128256_cfg2", 2, 128256, "bf16", 4, 2, 4, 1.0),
    Workload("an_v8192_cold", 4, 8192, "bf16", 4, 1, 2, 0.5, temperature=0.2),
    Workload("an_tinyV_dups", 16, 6, "f32", 3, 1, 2, 1.0),
    Workload("an_v4099_topk", 3, 4099, "bf16", 3, 1, 2, 1.0, temperature=0.7, top_k=40),
    Workload("an_v262144", 1, 262144, "bf16", 4, 1, 2, 0.75),
]


def run(batch):
    w = batch.workload
    out = binding.tree_analysis(batch.target_logits, batch.draft_logits, batch.parent, batch.token, batch.u_accept,
                                batch.u_bonus, w.temperature, w.top_k, w.top_p)
    torch.cuda.synchronize()
    return out


@pytest.mark.parametrize("w", SHAPES, ids=lambda w: w.name)
def test_analysis_against_oracle(w):
    batch = make_batch(w, seed=3, device="cuda")
    got = run(batch)
    inp = oracle_inputs(batch)
    acc, dv, st = oracle.node_analysis(inp)
    assert (st == 0).all()
    parent = batch.parent.cpu().numpy()
    internal = np.zeros(w.N, bool); internal[parent[1:]] = True
    ga = got.acceptance.cpu().numpy().astype(np.float64)
    gd = got.divergence.cpu().numpy().astype(np.float64)
    assert np.isnan(ga[:, ~internal]).all() and np.isnan(gd[:, ~internal]).all()
    err = np.abs(ga[:, internal] - acc[:, internal])
    assert err.max() < PROB_TOL, ("acceptance", err.max(), np.unravel_index(err.argmax(), err.shape))
    assert np.abs(gd[:, internal, 0] - dv[:, internal, 0]).max() < PROB_TOL
    for c in (1, 2):       # KL in nats: can be tens of nats, or +inf under truncation
        a, b = gd[:, internal, c], dv[:, internal, c]
        assert (np.isinf(a) == np.isinf(b)).all()
        fin = np.isfinite(b)
        assert np.abs(a[fin] - b[fin]).max(initial=0.0) < 1e-4 + 1e-5 * np.abs(b[fin]).max(initial=0.0)
    gb = got.branch.cpu().numpy().astype(np.float64)
    gr = got.reach.cpu().numpy().astype(np.float64)
    ge = got.block_eff.cpu().numpy().astype(np.float64)
    for s, name in enumerate(binding.SOLVERS):
        be, reach, br, st = oracle.block_efficiency(inp, name)
        assert (st == 0).all()
        assert np.abs(gb[s] - br).max() < PROB_TOL, (name, "branch", np.abs(gb[s] - br).max())
        assert np.abs(gr[s] - reach).max() < PROB_TOL, (name, "reach")
        assert np.abs(ge[s] - be).max() < 1e-5 * w.N, (name, "block efficiency")


def test_analysis_on_the_benchmark_workload():
    """cfg2 at full size: every node's acceptance rates and SpecInfer's block efficiency."""
    w = WORKLOADS["cfg2_llama3_b8"]
    batch = make_batch(w, seed=0, device="cuda")
    got = run(batch)
    inp = oracle_inputs(batch)
    acc, dv, _ = oracle.node_analysis(inp)
    parent = batch.parent.cpu().numpy()
    internal = np.zeros(w.N, bool); internal[parent[1:]] = True
    assert np.abs(got.acceptance.cpu().numpy()[:, internal] - acc[:, internal]).max() < PROB_TOL
    be, _, _, _ = oracle.block_efficiency(inp, "specinfer")
    assert np.abs(got.block_eff.cpu().numpy()[3] - be).max() < 1e-4


def test_latency_model():
    t_q = 1 + np.arange(400) / 100.0
    t_p = 10 + np.arange(400) / 10.0
    actions = np.array([[K, L1, L2] for K in range(1, 5) for L1 in range(9) for L2 in range(9)], np.int32)
    for ctx in (0, 100, 390):
        got = binding.latency_model(torch.tensor(t_q, device="cuda"), torch.tensor(t_p, device="cuda"), ctx,
                                    torch.tensor(actions, device="cuda"))
        torch.cuda.synchronize()
        want = oracle.latency_model(t_q, t_p, ctx, actions)
        np.testing.assert_allclose(got.cpu().numpy(), want, rtol=0, atol=1e-12)
