"""Pins of the top-k split recovery oracle (deployment appendix of the paper: the cloud truncates
h_cloud = h_LLM - beta*h_SLM- to its k largest entries, the edge adds beta*h_SLM+ there and resamples).

Each test ties the oracle to something other than itself: exact rational arithmetic, numpy's sort on rows where
the float32 arithmetic is exact, the full-vocabulary softmax of Eq. 8 (scipy) when nothing is truncated, and the
sampling law by a dense grid of uniforms.
"""
from fractions import Fraction

import numpy as np
import pytest
from scipy.special import log_softmax


@pytest.fixture(scope="module")
def o(oracle_mod):
    return oracle_mod


def _exact_rows(rng, V, lo=-64, hi=64, q=16):
    """float32 rows whose entries are multiples of 1/q: sums and products with small powers of two stay exact."""
    return [(rng.integers(lo * q, hi * q, size=V) / q).astype(np.float32) for _ in range(3)]


@pytest.mark.parametrize("beta", [0.5, 1.0, 2.0])
def test_cloud_topk_against_exact_rational_brute_force(o, beta):
    rng = np.random.default_rng(1)
    for V, k in ((12, 5), (9, 9), (7, 3), (33, 32)):
        L, _, M = _exact_rows(rng, V, -8, 8, 4)           # few distinct values: ties are frequent
        h = [Fraction(float(L[v])) - Fraction(beta) * Fraction(float(M[v])) for v in range(V)]
        order = sorted(range(V), key=lambda v: (-h[v], v))[:k]
        idx, val = o.cloud_topk_row(L, M, beta, k)
        assert idx.tolist() == order
        assert [Fraction(float(x)) for x in val] == [h[v] for v in order]


def test_cloud_topk_matches_numpy_sort_when_beta_is_one(o):
    """beta = 1: one float32 subtraction, which numpy rounds the same way as a fused multiply-add by -1."""
    rng = np.random.default_rng(2)
    L = rng.normal(0, 2, 5000).astype(np.float32)
    M = rng.normal(0, 2, 5000).astype(np.float32)
    h = L - M
    order = np.lexsort((np.arange(5000), -h.astype(np.float64)))[:32]
    idx, val = o.cloud_topk_row(L, M, 1.0, 32)
    assert np.array_equal(idx, order) and np.array_equal(val, h[order])
    # bf16 storage: the same after exact widening
    Lb = (L.view(np.uint32) >> 16).astype(np.uint16)
    Mb = (M.view(np.uint32) >> 16).astype(np.uint16)
    Lw = (Lb.astype(np.uint32) << 16).view(np.float32)
    Mw = (Mb.astype(np.uint32) << 16).view(np.float32)
    hb = Lw - Mw
    idx, val = o.cloud_topk_row(Lb, Mb, 1.0, 32)
    assert np.array_equal(idx, np.lexsort((np.arange(5000), -hb.astype(np.float64)))[:32])


def test_ties_nan_and_short_rows(o):
    L = np.zeros(10, np.float32)
    M = np.zeros(10, np.float32)
    idx, val = o.cloud_topk_row(L, M, 1.0, 4)
    assert idx.tolist() == [0, 1, 2, 3] and (val == 0).all()          # ties: lower token id first
    L[3] = np.nan                                                       # NaN is never selected
    L[7] = -np.inf
    idx, val = o.cloud_topk_row(L, M, 1.0, 10)
    assert idx.tolist() == [0, 1, 2, 4, 5, 6, 8, 9, 7, -1]
    assert val[8] == -np.inf and val[9] == -np.inf
    # adding a constant to the generalist's row moves the values, not the selection
    rng = np.random.default_rng(3)
    L, _, M = _exact_rows(rng, 300)
    i0, v0 = o.cloud_topk_row(L, M, 2.0, 32)
    i1, v1 = o.cloud_topk_row(L + np.float32(5.0), M, 2.0, 32)
    assert np.array_equal(i0, i1) and np.array_equal(v1, v0 + np.float32(5.0))


@pytest.mark.parametrize("beta,T", [(1.0, 1.0), (2.0, 0.5), (0.5, 1.5)])
def test_no_truncation_reduces_to_the_softmax_of_eq8(o, beta, T):
    """With k = V the edge samples the full Softmax(h_rec / T): compare with scipy and with the Eq. 8 oracle."""
    rng = np.random.default_rng(4)
    V = 200
    L, Pp, M = _exact_rows(rng, V, -6, 6)
    idx, val = o.cloud_topk_row(L, M, beta, V)
    r = o.edge_resample_row(Pp, beta, T, idx, val, 0.37)
    h_rec = (L.astype(np.float64) + beta * (Pp.astype(np.float64) - M.astype(np.float64))) / T
    want = np.exp(log_softmax(h_rec))
    got = np.empty(V)
    got[idx] = r["probs"]
    assert np.allclose(got, want, rtol=1e-12, atol=0)
    full = o.row(L, Pp, M, beta=beta, temperature=T)
    assert np.allclose(np.log(got), full["logp_star"], atol=1e-12)
    assert abs(r["logprob"] - np.log(got[r["token"]])) < 1e-12


def test_truncated_law_and_inverse_cdf_in_list_order(o):
    """k < V: the law is the softmax of h_rec over the kept tokens only; a dense grid of uniforms reproduces it
    and walks the list in the transmitted order (highest h_cloud first)."""
    rng = np.random.default_rng(5)
    V, k, beta, T = 64, 6, 2.0, 0.5
    L, Pp, M = _exact_rows(rng, V, -4, 4)
    idx, val = o.cloud_topk_row(L, M, beta, k)
    h_rec = (val.astype(np.float64) + beta * Pp[idx].astype(np.float64)) / T
    want = np.exp(h_rec - h_rec.max())
    want /= want.sum()
    N = 20000
    counts = np.zeros(k)
    prev_j = 0
    for i in range(N):
        u = (i + 0.5) / N
        r = o.edge_resample_row(Pp, beta, T, idx, val, u)
        j = int(np.where(idx == r["token"])[0][0])
        assert j >= prev_j                                   # the CDF walk follows the list order
        prev_j = j
        counts[j] += 1
        assert abs(r["logprob"] - np.log(want[j])) < 1e-12
    assert np.abs(counts / N - want).max() <= 1.0 / N + 1e-12
    r = o.edge_resample_row(Pp, beta, T, idx, val, 0.0)
    assert r["token"] == idx[np.argmax(want > 0)]
    # slots without a token (short rows) carry no mass
    idx2 = idx.copy(); idx2[-2:] = -1
    r2 = o.edge_resample_row(Pp, beta, T, idx2, val, 0.999999)
    assert r2["token"] in idx[:-2] and r2["probs"][-2:].sum() == 0
