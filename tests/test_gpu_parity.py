"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_16994_b200 import binding, synth
from paper_2602_16994_b200.synth import WORKLOADS, Workload, make_batch
from tests.parity import PROB_TOL, Tally, check_batch, gpu_verify, oracle_inputs, run_oracle

pytestmark = pytest.mark.gpu
ALGOS = ["specinfer", "traversal"]


def small(name, V, dtype, K, L1, L2, B, sigma=1.0, T=1.0):
    return Workload(name, B, V, dtype, K, L1, L2, sigma, temperature=T)


@pytest.mark.parametrize("algo", ALGOS)
def test_cfg1_tiny(algo):
    batch = make_batch(WORKLOADS["cfg1_tiny"], seed=0, device="cuda")
    t = check_batch(batch, algo)
    assert t.near_margin_mismatches == 0


SHAPES = [
    small("v5", 5, "f32", 2, 0, 2, 8),                    # vocabulary smaller than a vector
    small("v1000_f32", 1000, "f32", 2, 0, 3, 6),
    small("v1003_bf16_misaligned", 1003, "bf16", 3, 1, 2, 5),   # rows not 16-byte aligned, ragged tail
    small("v4100_f32_T", 4100, "f32", 4, 2, 2, 3, T=0.7),
    small("v32000_bf16", 32000, "bf16", 4, 1, 3, 4, sigma=0.7),
    small("v50257_bf16_odd", 50257, "bf16", 2, 1, 2, 2),
    small("v128256_bf16", 128256, "bf16", 4, 2, 4, 2),    # the headline shape, two sequences
    small("v151936_bf16_T06", 151936, "bf16", 8, 0, 2, 1, sigma=0.7, T=0.6),
    small("v262144_bf16", 262144, "bf16", 4, 1, 2, 1, sigma=0.75),   # 16-CTA clusters
    small("path_only", 2048, "bf16", 1, 0, 6, 4),         # K = 1: naive / block verification
    small("root_only", 3000, "bf16", 1, 0, 0, 3),         # N = 1: just the bonus draw from p
    small("wide", 640, "f32", 16, 0, 1, 3),               # 16 children under one node
    small("cold", 8192, "bf16", 4, 1, 2, 4, sigma=1.2, T=0.3),
    # near-greedy, nothing truncated, several siblings: target and draft put nearly all their mass on
    # the same token, so residual masses are tiny differences of probabilities close to 1
    small("cold_T02", 50000, "bf16", 4, 1, 3, 8, sigma=1.0, T=0.2),
    small("cold_T015", 50000, "bf16", 4, 1, 3, 8, sigma=0.3, T=0.15),
    small("cold_T02_f32", 32000, "f32", 6, 0, 2, 6, sigma=0.5, T=0.2),
    small("cold_T015_v128256", 128256, "bf16", 4, 2, 4, 4, sigma=0.5, T=0.15),
]


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("w", SHAPES, ids=lambda w: w.name)
def test_shapes(algo, w):
    batch = make_batch(w, seed=1, device="cuda")
    check_batch(batch, algo)


@pytest.mark.parametrize("algo", ALGOS)
def test_cfg2_full_size(algo):
    """The bench workload in the bench's launch configuration: every sequence against the oracle."""
    batch = make_batch(WORKLOADS["cfg2_llama3_b8"], seed=0, device="cuda")
    t = check_batch(batch, algo, full=True)
    assert t.near_margin_mismatches == 0


@pytest.mark.parametrize("algo", ALGOS)
def test_many_decisions_mismatch_rate(algo):
    """Tolerated (near-margin) differences stay below 1e-4 of all decisions over a large sample."""
    total = Tally()
    for seed in range(12):
        w = small("rate", 8000, "bf16", 3, 1, 3, 512, sigma=0.8)
        total.add(check_batch(make_batch(w, seed=seed, device="cuda"), algo, full=False))
    assert total.decisions > 20000
    assert total.near_margin_mismatches <= 1e-4 * total.decisions, vars(total)


def test_per_sequence_topology_and_temperature():
    w = small("mixed", 3000, "bf16", 3, 1, 2, 4)
    batch = make_batch(w, seed=3, device="cuda")
    N = w.N
    # sequence-specific trees: same node count, different shapes (all satisfy parent[i] < i)
    shapes = [synth.delayed_tree(3, 1, 2)[0], np.array([-1] + list(range(N - 1)), np.int32),
              np.array([-1] + [0] * (N - 1), np.int32), synth.delayed_tree(3, 1, 2)[0]]
    parent = torch.tensor(np.stack(shapes), dtype=torch.int32, device="cuda")
    temps = torch.tensor([1.0, 0.5, 2.0, 0.9], dtype=torch.float32, device="cuda")
    for algo, fn in (("specinfer", binding.verify_specinfer), ("traversal", binding.verify_traversal)):
        got = fn(batch.target_logits, batch.draft_logits, parent, batch.token, batch.u_accept, batch.u_bonus,
                 temperature=1.0, temperature_per_seq=temps)
        torch.cuda.synchronize()
        a = batch.numpy()
        inp = oracle.TreeInputs(a["target_logits"], a["draft_logits"], parent.cpu().numpy(), a["token"],
                                a["u_accept"], a["u_bonus"], temperature_per_seq=temps.cpu().numpy())
        ref = (oracle.verify_specinfer if algo == "specinfer" else oracle.verify_traversal)(inp)
        assert (got.status.cpu().numpy() == 0).all()
        np.testing.assert_array_equal(got.accepted_node.cpu().numpy(), ref.accepted_node)
        np.testing.assert_array_equal(got.out_tokens.cpu().numpy(), ref.out_tokens)


def test_strided_logits():
    """Rows may sit in a larger buffer: node stride > V, sequence stride > N * node stride."""
    w = small("strided", 2000, "bf16", 2, 1, 2, 3)
    batch = make_batch(w, seed=4, device="cuda")
    B, N, V = batch.target_logits.shape
    big_p = torch.zeros((B, N + 2, V + 24), dtype=torch.bfloat16, device="cuda")
    big_q = torch.zeros_like(big_p)
    big_p[:, :N, :V] = batch.target_logits
    big_q[:, :N, :V] = batch.draft_logits
    got = binding.verify_specinfer(big_p[:, :N, :V], big_q[:, :N, :V], batch.parent, batch.token,
                                   batch.u_accept, batch.u_bonus)
    torch.cuda.synchronize()
    _, ref = run_oracle(batch, "specinfer")
    np.testing.assert_array_equal(got.accepted_node.cpu().numpy(), ref.accepted_node)
    np.testing.assert_array_equal(got.out_tokens.cpu().numpy(), ref.out_tokens)


def test_device_detected_errors_are_reported_not_trapped():
    w = small("bad", 500, "f32", 2, 0, 2, 4)
    batch = make_batch(w, seed=5, device="cuda")
    token = batch.token.clone()
    token[1, 2] = 500                      # token == V
    zp = batch.target_logits.clone()
    zp[2, 0, 17] = float("nan")            # NaN in the root's target row
    zp[3, 1, :] = float("-inf")            # a row with no finite logit
    for fn in (binding.verify_specinfer, binding.verify_traversal):
        got = fn(zp, batch.draft_logits, batch.parent, token, batch.u_accept, batch.u_bonus)
        torch.cuda.synchronize()
        st = got.status.cpu().numpy()
        assert st[0] == 0 and st[1] == 2 and st[2] == 3 and st[3] == 3, st
        assert got.accept_len.cpu().numpy()[1:].tolist() == [-1, -1, -1]
        assert got.accepted_node.cpu().numpy()[0] >= 0
    bad_parent = batch.parent.clone()
    bad_parent[2] = 3                      # parent[i] >= i
    got = binding.verify_specinfer(batch.target_logits, batch.draft_logits, bad_parent, batch.token,
                                   batch.u_accept, batch.u_bonus)
    torch.cuda.synchronize()
    assert (got.status.cpu().numpy() == 1).all()
    many = synth.delayed_tree(17, 0, 1)[0]          # 17 children under the root: above the limit
    wb = small("many", 300, "f32", 17, 0, 1, 2)
    bm = make_batch(wb, seed=6, device="cuda")
    got = binding.verify_traversal(bm.target_logits, bm.draft_logits, bm.parent, bm.token, bm.u_accept, bm.u_bonus)
    torch.cuda.synchronize()
    assert (got.status.cpu().numpy() == 1).all() and len(many) == 18


@pytest.mark.parametrize("V,dtype", [(1000, torch.float32), (4099, torch.bfloat16), (128256, torch.bfloat16),
                                     (262144, torch.bfloat16)])
def test_tree_probs(V, dtype):
    g = torch.Generator(device="cuda").manual_seed(7)
    z = (torch.randn((2, 3, V), generator=g, device="cuda") * 3).to(dtype)
    for T in (1.0, 0.3):
        probs, stats = binding.tree_probs(z, 0, temperature=T)
        torch.cuda.synchronize()
        zb = z.cpu()
        bits = zb.view(torch.int16).numpy().view(np.uint16) if dtype == torch.bfloat16 else zb.numpy()
        inp = oracle.TreeInputs(bits, bits, np.array([-1, 0, 0], np.int32), np.zeros((2, 3), np.int32),
                                np.zeros((2, 3), np.float32), np.zeros((2, 3), np.float32), temperature=T)
        rp, rs, _ = oracle.tree_probs(inp, 0)
        assert np.abs(probs.cpu().numpy() - rp).max() < PROB_TOL
        st = stats.cpu().numpy().astype(np.float64)
        np.testing.assert_allclose(st[..., 0], rs[..., 0], rtol=1e-6)
        np.testing.assert_allclose(st[..., 1], rs[..., 1], rtol=1e-5)
        np.testing.assert_allclose(st[..., 3], rs[..., 3], atol=1e-4)
        np.testing.assert_allclose(st[..., 4], rs[..., 4], atol=PROB_TOL)


@pytest.mark.parametrize("V", [7, 1000, 50001, 128256, 300000])
def test_sample_bonus(V):
    g = torch.Generator(device="cuda").manual_seed(8)
    R = 64
    w = torch.rand((R, V), generator=g, device="cuda")
    w = torch.where(torch.rand((R, V), generator=g, device="cuda") < 0.4, torch.zeros_like(w), w)
    w[3] = 0.0                                   # an all-zero row
    w[4] = 0.0; w[4, V // 2] = 2.0               # a single token
    u = torch.rand(R, generator=g, device="cuda")
    u[5] = 0.0
    tok, mg = binding.sample_bonus(w, u, want_margin=True)
    torch.cuda.synchronize()
    rt, rm = oracle.sample_bonus(w.cpu().numpy(), u.cpu().numpy())
    tok = tok.cpu().numpy()
    for r in range(R):
        if tok[r] != rt[r]:
            assert rm[r] < 1e-6, (r, tok[r], rt[r], rm[r])
    assert tok[3] == -1 and tok[4] == V // 2
    assert (tok == rt).mean() > 0.95


def test_host_buffer_api_matches_device_api():
    w = small("host", 5000, "bf16", 2, 1, 2, 3)
    batch = make_batch(w, seed=9, device="cpu")
    hv = binding.HostVerifier(w.B, w.N, w.V, torch.bfloat16, algorithm="traversal")
    pin = lambda t: t.pin_memory()
    out = hv.run(pin(batch.target_logits), pin(batch.draft_logits), pin(batch.parent), pin(batch.token),
                 pin(batch.u_accept), pin(batch.u_bonus))
    _, ref = run_oracle(batch, "traversal")
    np.testing.assert_array_equal(out["accepted_node"].numpy(), ref.accepted_node)
    np.testing.assert_array_equal(out["out_tokens"].numpy(), ref.out_tokens)
    assert hv.h2d_bytes() > 2 * w.B * w.N * w.V * 2 and hv.d2h_bytes() > 0


# ---------------------------------------------------------------------------------------------
# truncated sampling distributions (top-k / top-p)
# ---------------------------------------------------------------------------------------------
TRUNC = [dict(top_k=50), dict(top_p=0.95), dict(top_k=200, top_p=0.9), dict(top_k=1), dict(top_p=0.5)]


def _check_tree_probs_truncated(V, dtype, trunc, scale=3.0, temperatures=(1.0, 0.6)):
    g = torch.Generator(device="cuda").manual_seed(11)
    z = (torch.randn((2, 3, V), generator=g, device="cuda") * scale).to(dtype)
    z[0, 0, : V // 2] = z[0, 0, V // 2: 2 * (V // 2)]          # exact ties everywhere in one row
    z[1, 1, 5] = -0.0
    z[1, 1, 6] = 0.0
    for T in temperatures:
        probs, stats = binding.tree_probs(z, 0, temperature=T, **trunc)
        torch.cuda.synchronize()
        zb = z.cpu()
        bits = zb.view(torch.int16).numpy().view(np.uint16) if dtype == torch.bfloat16 else zb.numpy()
        inp = oracle.TreeInputs(bits, bits, np.array([-1, 0, 0], np.int32), np.zeros((2, 3), np.int32),
                                np.zeros((2, 3), np.float32), np.zeros((2, 3), np.float32), temperature=T,
                                top_k=trunc.get("top_k", 0), top_p=trunc.get("top_p", 1.0))
        rp, rs, _ = oracle.tree_probs(inp, 0)
        sure = rs[..., 5] >= 1e-6                      # rows whose nucleus boundary is not within 1e-6 of top_p
        assert sure.mean() > 0.8
        got = probs.cpu().numpy()
        st = stats.cpu().numpy().astype(np.float64)
        assert np.abs(got - rp)[sure].max() < PROB_TOL
        np.testing.assert_array_equal(st[..., 2][sure], rs[..., 2][sure])          # kept count
        np.testing.assert_array_equal(st[..., 5][sure], rs[..., 6][sure].astype(np.float32))   # threshold logit


@pytest.mark.parametrize("V,dtype", [(1000, torch.float32), (4099, torch.bfloat16), (128256, torch.bfloat16)])
@pytest.mark.parametrize("trunc", TRUNC, ids=lambda d: "_".join(f"{k}{v}" for k, v in d.items()))
def test_tree_probs_truncated(V, dtype, trunc):
    _check_tree_probs_truncated(V, dtype, trunc)


@pytest.mark.parametrize("V,dtype,scale,trunc", [
    (4099, torch.bfloat16, 0.05, dict(top_p=0.9)),      # flat row: the nucleus window reaches across zero
    (4099, torch.bfloat16, 3.0, dict(top_k=600)),       # k above what the per-thread maxima can bound
    (20000, torch.float32, 0.5, dict(top_p=0.9)),       # more candidates than the list holds
    (20000, torch.float32, 0.5, dict(top_k=3000, top_p=0.99)),
], ids=["flat_bf16_p", "bf16_k600", "f32_overflow_p", "f32_k3000_p"])
def test_tree_probs_truncated_rows_left_to_the_general_kernel(V, dtype, scale, trunc):
    """Rows the candidate-based fast path cannot settle are listed for the general selection kernel."""
    _check_tree_probs_truncated(V, dtype, trunc, scale=scale, temperatures=(1.0,))


TRUNC_SHAPES = [
    Workload("t_v1000_f32_k", 6, 1000, "f32", 2, 0, 3, 1.0, temperature=0.8, top_k=20),
    Workload("t_v4100_bf16_p", 5, 4100, "bf16", 3, 1, 2, 0.7, temperature=0.6, top_p=0.95),
    Workload("t_v32000_bf16_kp", 4, 32000, "bf16", 4, 1, 3, 1.0, temperature=0.7, top_k=100, top_p=0.9),
    Workload("t_v151936_bf16_p", 2, 151936, "bf16", 8, 0, 2, 0.7, temperature=0.6, top_p=0.95),
    Workload("t_v128256_bf16_k", 2, 128256, "bf16", 8, 2, 2, 1.2, temperature=0.3, top_k=50),
]


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("w", TRUNC_SHAPES, ids=lambda w: w.name)
def test_truncated_verification(algo, w):
    batch = make_batch(w, seed=2, device="cuda")
    t = check_batch(batch, algo)
    assert t.sequences_set_aside == 0, vars(t)


def test_traversal_weight_one_with_a_vanishing_residual():
    """A node of weight 1 whose residual mass after its child is about 1e-17 (a one-token nucleus that the
    draft nearly matches): the weight update S / (S + 1 - w) must give 1, not S / ((S + 1) - 1) = S / 0."""
    w = Workload("t_v1000_f32_p9", 12, 1000, "f32", 2, 1, 3, 1.0, top_p=0.9)
    batch = make_batch(w, seed=106, device="cuda")
    check_batch(batch, "traversal", full=True)
    check_batch(batch, "specinfer", full=True)


def test_traversal_skipping_does_not_change_the_outcome():
    """Without per-node diagnostics the Traversal call skips subtrees that come wholly after a node already
    known to be accepted, and nodes below a weight of 0.  Outcome and residual must be those of the call
    that evaluates every node (diagnostics on), on trees wide and deep enough for both kinds of skipping."""
    skipped_something = 0
    for seed in range(10):
        w = small("skip", 6000, "bf16", 4, 2, 4, 6, sigma=0.6)
        batch = make_batch(w, seed=seed, device="cuda")
        plain = gpu_verify(batch, "traversal", residual=True)
        full = gpu_verify(batch, "traversal", residual=True, node_thr=True, node_w_in=True, margin=True)
        for name in ("accepted_node", "accept_len", "bonus_token", "out_tokens", "status"):
            assert torch.equal(getattr(plain, name), getattr(full, name)), (seed, name)
        assert torch.equal(plain.residual, full.residual), seed
        # the accepted node is rarely the last one in traversal order: then there was something to skip
        N = w.N
        skipped_something += int((full.accepted_node != 0).sum().item())
        assert (full.node_thr[:, 0] == 1.0).all() and full.node_thr.shape == (w.B, N)
    assert skipped_something > 0


TREE_SHAPES = [
    Workload("s_k8_root", 6, 3000, "bf16", 8, 0, 3, 0.6),        # N = 25: a wide root
    Workload("s_k2_deep", 6, 2000, "f32", 2, 3, 6, 0.4),          # N = 16: deep branches
    Workload("s_k5_d1", 6, 5000, "bf16", 5, 1, 6, 0.5),           # N = 32: the largest tree with a post-order table
    Workload("s_k6_d1", 4, 4000, "bf16", 6, 1, 6, 0.5),           # N = 38: no table, nothing skipped by rank
]


@pytest.mark.parametrize("w", TREE_SHAPES, ids=lambda w: w.name)
def test_traversal_on_wide_and_deep_trees(w):
    """Traversal's hand-out hints (weight 0 at an ancestor, subtree after a known acceptance) on trees of other
    shapes than the configs', at and beyond the size limit of the post-order table."""
    total = Tally()
    for seed in range(100, 108):
        total.add(check_batch(make_batch(w, seed=seed, device="cuda"), "traversal", full=(seed % 4 == 0)))
    assert total.near_margin_mismatches <= 1, vars(total)
