"""Randomised parity campaign: many seeds x shapes x both verifiers, every output against the CPU
oracle under the single 1e-5 / exact-decision rule of tests/parity.py.  The shapes cover the regimes
in which residual masses are small differences of large probabilities (near-greedy temperatures
without truncation, top-k / top-p), duplicate sibling tokens, masked target logits, many sequences
per cluster, wide and deep trees, misaligned rows."""
import numpy as np
import pytest
import torch

from paper_2602_16994_b200.synth import Workload, make_batch
from tests.parity import Tally, check_batch

pytestmark = pytest.mark.gpu

# name, B, V, dtype, K, L1, L2, sigma, sampling
MAIN = [
    ("c_v128256_d2", 8, 128256, "bf16", 4, 2, 4, 1.0, {}),
    ("c_v32000_root", 16, 32000, "bf16", 8, 0, 3, 0.7, {}),
    ("c_v50257_f32", 6, 50257, "f32", 3, 1, 3, 1.0, {"temperature": 0.8}),
    ("c_v128256_topk", 6, 128256, "bf16", 4, 2, 3, 1.2, {"temperature": 0.3, "top_k": 50}),
    ("c_v151936_topp", 4, 151936, "bf16", 8, 0, 2, 0.7, {"temperature": 0.6, "top_p": 0.95}),
    ("c_v4099_kp", 12, 4099, "bf16", 3, 1, 3, 1.0, {"temperature": 0.7, "top_k": 100, "top_p": 0.9}),
    ("c_v1000_f32_p", 12, 1000, "f32", 2, 1, 3, 1.0, {"top_p": 0.9}),
    ("c_v262144", 4, 262144, "bf16", 4, 2, 4, 0.75, {}),
]
COLD = [
    ("k_T02", 8, 50000, "bf16", 4, 1, 3, 1.0, {"temperature": 0.2}),
    ("k_T015", 8, 50000, "bf16", 4, 1, 3, 0.3, {"temperature": 0.15}),
    ("k_T02_wide", 6, 128256, "bf16", 8, 0, 2, 0.5, {"temperature": 0.2}),
    ("k_T015_f32", 8, 32000, "f32", 4, 2, 2, 0.5, {"temperature": 0.15}),
]
ODD = [
    ("d_wide16", 5, 20001, "bf16", 16, 0, 1, 1.0, {}),
    ("d_deep", 6, 8191, "bf16", 1, 0, 12, 0.5, {}),
    ("d_manyseq", 96, 4096, "bf16", 3, 1, 2, 1.0, {}),
    ("d_tinyV", 40, 5, "f32", 3, 1, 2, 1.0, {}),
    ("d_v300k", 2, 300000, "bf16", 2, 1, 2, 1.0, {}),
    ("d_hot", 8, 50000, "bf16", 4, 1, 3, 0.3, {"temperature": 2.5}),
    ("d_cold_k", 8, 32000, "f32", 4, 1, 3, 1.5, {"temperature": 0.2, "top_k": 5}),
    ("d_p_small", 8, 32000, "bf16", 6, 0, 2, 1.0, {"top_p": 0.3}),
    ("d_misaligned", 6, 12345, "bf16", 3, 1, 2, 1.0, {}),
]
TOTAL = Tally()


def _run(shape, seed, full, disturb=False):
    name, B, V, dt, K, L1, L2, sig, kw = shape
    w = Workload(name, B, V, dt, K, L1, L2, sig, **kw)
    batch = make_batch(w, seed=seed, device="cuda")
    if disturb and V > 100:
        # a tenth of the vocabulary gets target probability 0, and two siblings share a token
        g = torch.Generator(device="cuda").manual_seed(seed)
        mask = torch.rand((V,), generator=g, device="cuda") < 0.1
        batch.target_logits[:, :, mask] = float("-inf")
        par = batch.parent.cpu().numpy()
        kids = [c for c in range(1, w.N) if par[c] == L1]
        if len(kids) >= 2:
            batch.token[:, kids[1]] = batch.token[:, kids[0]]
    for algo in ("specinfer", "traversal"):
        TOTAL.add(check_batch(batch, algo, full=full))


@pytest.mark.parametrize("shape", MAIN, ids=lambda s: s[0])
def test_campaign_main(shape):
    for seed in range(100):
        _run(shape, 100 + seed, full=(seed % 3 == 0))


@pytest.mark.parametrize("shape", COLD, ids=lambda s: s[0])
def test_campaign_near_greedy(shape):
    for seed in range(40):
        _run(shape, 300 + seed, full=True)


@pytest.mark.parametrize("shape", ODD, ids=lambda s: s[0])
def test_campaign_odd_shapes(shape):
    for seed in range(12):
        _run(shape, 500 + seed, full=(seed % 2 == 0), disturb=(seed % 2 == 1))


def test_campaign_tolerated_differences():
    """Runs after the campaigns above (same module, file order)."""
    assert TOTAL.decisions > 100000, "the campaigns did not run before this one"
    assert TOTAL.near_margin_mismatches < 1e-4 * TOTAL.decisions, vars(TOTAL)
    print(vars(TOTAL))
