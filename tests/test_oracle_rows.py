"""Pins for the oracle's row-level pieces: logits -> distribution and the inverse-CDF draw.

The distribution is checked against library routines (scipy softmax / entropy), against a sort-based
statement of top-k / top-p written here with numpy on tie-free rows, and through properties that
fix the tie rules (permutation equivariance, whole value groups).  The draw is checked against
``numpy.searchsorted`` on the running sum and at the exact interval boundaries.
"""
import numpy as np
import pytest
import scipy.special
import scipy.stats
import torch

import oracle
from oracle import TreeInputs


def test_plain_softmax_matches_scipy():
    rng = np.random.default_rng(0)
    for T in (1.0, 0.3, 2.5):
        z = rng.standard_normal(1000) * 4
        p, st = oracle.row_probs(z, T)
        np.testing.assert_allclose(p, scipy.special.softmax(z / T), rtol=1e-13, atol=0)
        assert st[3] == pytest.approx(scipy.stats.entropy(p), rel=1e-12)
        assert st[4] == p.max() and st[2] == z.size
        assert st[0] == (z / T).max()
        assert st[1] == pytest.approx(np.exp(z / T - (z / T).max()).sum(), rel=1e-13)


def sorted_truncation(z, T, top_k, top_p):
    """top-k then top-p by sorting probabilities, for rows without equal logits."""
    p = scipy.special.softmax(z / T)
    order = np.argsort(-p, kind="stable")
    keep = np.zeros(z.size, bool)
    n = z.size if not (0 < top_k < z.size) else top_k
    keep[order[:n]] = True
    if top_p < 1.0:
        pk = np.where(keep, p, 0.0); pk /= pk.sum()
        cum = np.cumsum(pk[order])
        m = int(np.searchsorted(cum, top_p, side="left")) + 1      # fewest leading tokens with cum >= top_p
        keep2 = np.zeros(z.size, bool); keep2[order[:min(m, n)]] = True
        keep &= keep2
    out = np.where(keep, p, 0.0)
    return out / out.sum()


@pytest.mark.parametrize("T,top_k,top_p", [(1.0, 50, 1.0), (0.6, 0, 0.95), (0.3, 50, 1.0), (1.0, 20, 0.9),
                                           (1.0, 0, 0.5), (1.7, 1, 1.0), (1.0, 0, 0.999)])
def test_truncation_matches_sorted_definition_without_ties(T, top_k, top_p):
    rng = np.random.default_rng(1)
    for _ in range(5):
        z = rng.standard_normal(2000) * 3            # float64 draws: no equal values
        p, st = oracle.row_probs(z, T, top_k, top_p)
        want = sorted_truncation(z, T, top_k, top_p)
        np.testing.assert_allclose(p, want, rtol=1e-12, atol=0)
        assert st[2] == (want > 0).sum()
        assert abs(p.sum() - 1) < 1e-12


def test_ties_kept_as_whole_groups_and_order_free():
    rng = np.random.default_rng(2)
    z = np.round(rng.standard_normal(600) * 2, 1)            # heavy ties, like bf16 logits
    for top_k, top_p in [(10, 1.0), (0, 0.7), (25, 0.8), (0, 0.3)]:
        p, st = oracle.row_probs(z, 1.0, top_k, top_p)
        kept = p > 0
        thr = z[kept].min()
        assert (kept == (z >= thr)).all()                   # a value threshold: whole groups
        if top_k:
            assert kept.sum() >= min(top_k, (z >= np.sort(z)[-top_k]).sum()) or top_p < 1
        perm = rng.permutation(z.size)
        p2, _ = oracle.row_probs(z[perm], 1.0, top_k, top_p)
        np.testing.assert_allclose(p2, p[perm], rtol=1e-12, atol=1e-18)
        np.testing.assert_allclose(p[kept], scipy.special.softmax(z[kept]), rtol=1e-12)


def test_topk_value_threshold_counts_multiplicity():
    z = np.array([5.0, 3.0, 3.0, 3.0, 1.0, 0.0])
    p, st = oracle.row_probs(z, 1.0, 2, 1.0)                 # 2nd largest is a 3.0: all three stay
    assert (p > 0).tolist() == [True, True, True, True, False, False] and st[2] == 4 and st[6] == 3.0
    p, st = oracle.row_probs(z, 1.0, 1, 1.0)
    assert (p > 0).tolist() == [True, False, False, False, False, False]


def test_topp_minimal_prefix_of_groups():
    # masses .5, .2, .2, .1 with the two .2 tokens tied
    z = np.log(np.array([0.5, 0.2, 0.2, 0.1]))
    for top_p, n in [(0.4, 1), (0.5, 1), (0.51, 3), (0.89, 3), (0.95, 4)]:
        p, st = oracle.row_probs(z, 1.0, 0, top_p)
        assert (p > 0).sum() == n, (top_p, p)
    p, st = oracle.row_probs(z, 1.0, 0, 0.6)
    assert st[5] == pytest.approx(0.1, abs=1e-12)            # nearer cumulative mass: .5


def test_temperature_is_a_division_of_logits():
    rng = np.random.default_rng(4)
    z = rng.standard_normal(300)
    a, _ = oracle.row_probs(z, 0.5, 7, 0.9)
    b, _ = oracle.row_probs(z * 2.0, 1.0, 7, 0.9)
    np.testing.assert_allclose(a, b, rtol=1e-14)


def test_bad_rows():
    with pytest.raises(ValueError):
        oracle.row_probs(np.array([0.0, np.nan]), 1.0)
    with pytest.raises(ValueError):
        oracle.row_probs(np.array([0.0, 1.0]), 0.0)
    with pytest.raises(ValueError):
        oracle.row_probs(np.array([-np.inf, -np.inf]), 1.0)


def test_bf16_rows_are_widened_exactly():
    g = torch.Generator().manual_seed(0)
    z = (torch.randn(2, 3, 400, generator=g) * 3).to(torch.bfloat16)
    bits = z.view(torch.int16).numpy().view(np.uint16)
    inp = TreeInputs(bits, bits, np.array([-1, 0, 0], np.int32), np.zeros((2, 3), np.int32),
                     np.zeros((2, 3), np.float32), np.zeros((2, 3), np.float32), temperature=0.8)
    probs, stats, status = oracle.tree_probs(inp, 0)
    want = scipy.special.softmax(z.to(torch.float64).numpy() / np.float64(np.float32(0.8)), axis=-1)
    np.testing.assert_allclose(probs, want, rtol=1e-12)
    assert (status == 0).all()


# ---------------------------------------------------------------------------------------------
# inverse CDF
# ---------------------------------------------------------------------------------------------
def test_inverse_cdf_matches_searchsorted_and_boundaries():
    rng = np.random.default_rng(5)
    w = rng.random(257); w[rng.random(257) < 0.3] = 0.0; w[-1] = 0.0
    c = np.cumsum(w)                                         # numpy cumsum is the same sequential sum
    W = c[-1]
    for u in rng.random(2000):
        t, m = oracle.inverse_cdf(w, u)
        want = int(np.searchsorted(c, u * W, side="right"))
        assert t == want and w[t] > 0
        lo = u * W - (c[t - 1] if t else 0.0)
        assert m == pytest.approx(min(lo, c[t] - u * W) / W, abs=1e-15)
    # u = 0 gives the first positive-weight token; u just below 1 the last positive one
    first, last = int(np.nonzero(w)[0][0]), int(np.nonzero(w)[0][-1])
    assert oracle.inverse_cdf(w, 0.0)[0] == first
    assert oracle.inverse_cdf(w, np.nextafter(1.0, 0.0))[0] == last
    # exactly on a boundary the draw moves to the next token with weight (C_t > target is strict)
    w2 = np.array([0.25, 0.0, 0.25, 0.5])
    assert oracle.inverse_cdf(w2, 0.25)[0] == 2 and oracle.inverse_cdf(w2, 0.5)[0] == 3
    assert oracle.inverse_cdf(w2, 0.2499999)[0] == 0
    assert oracle.inverse_cdf(np.zeros(4), 0.3)[0] == -1


def test_inverse_cdf_law_on_a_grid():
    w = np.array([3.0, 0.0, 1.0, 4.0, 2.0])
    M = 10000
    counts = np.zeros(5)
    for i in range(M):
        counts[oracle.inverse_cdf(w, (i + 0.5) / M)[0]] += 1
    np.testing.assert_allclose(counts / M, w / w.sum(), atol=1.5 / M)


def test_sample_bonus_rows():
    rng = np.random.default_rng(6)
    w = rng.random((7, 100)).astype(np.float32)
    u = rng.random(7).astype(np.float32)
    tok, mg = oracle.sample_bonus(w, u)
    for r in range(7):
        t, m = oracle.inverse_cdf(w[r].astype(np.float64), float(u[r]))
        assert tok[r] == t and mg[r] == m
