"""Pins for the CPU oracle: what the paper and the mathematics fix, computed by other means.

Each test names the passage it pins.  The comparisons go through library routines
(scipy / torch float64 softmax), hand-derived rationals (tests/golden/) or exhaustive
grids, never through a second copy of the oracle's own code.
"""
import json
import os

import numpy as np
import pytest
import scipy.special as sps
import torch

GOLD = os.path.join(os.path.dirname(__file__), "golden", "rational_v4.json")


def _rand_rows(rng, B, K, V, scale=2.0):
    L = (scale * rng.standard_normal((B, K + 1, V))).astype(np.float32)
    P = (L + rng.standard_normal((B, K + 1, V))).astype(np.float32)
    M = (L + 0.5 * rng.standard_normal((B, K + 1, V))).astype(np.float32)
    return L, P, M


def _round(o, L, P, M, tok, u_acc, u_rec, lam=0.5, beta=1.0, T=1.0, length=None, **kw):
    B, K1, _ = L.shape
    K = K1 - 1
    full = lambda x: np.full(B, x, np.float32) if np.isscalar(x) else np.asarray(x, np.float32)
    length = np.full(B, K, np.int32) if length is None else np.asarray(length, np.int32)
    return o.verify_recover_round(L, P, M, tok, length, full(lam), full(beta), full(T), u_acc, u_rec, **kw)


# ---------------------------------------------------------------- log-sum-exp (library routine)
def test_logsumexp_matches_scipy(oracle_mod):
    rng = np.random.default_rng(1)
    for n in (1, 2, 7, 1000, 40000):
        x = rng.standard_normal(n) * 30.0
        assert oracle_mod.logsumexp(x) == pytest.approx(sps.logsumexp(x), rel=0, abs=1e-12)
    x = np.array([-np.inf, 0.0, -np.inf])
    assert oracle_mod.logsumexp(x) == 0.0
    assert oracle_mod.logsumexp(np.array([-np.inf, -np.inf])) == -np.inf
    assert np.isnan(oracle_mod.logsumexp(np.array([0.0, np.nan])))
    assert oracle_mod.logsumexp(np.array([1e4, 1e4 + 1.0])) == pytest.approx(1e4 + 1.0 + np.log1p(np.exp(-1.0)))


# ---------------------------------------------------------------- Eq. 2-4, 8: fused target / recovery softmax
@pytest.mark.parametrize("beta,T", [(1.0, 1.0), (0.0, 1.0), (2.5, 0.7), (0.5, 1.5)])
def test_row_matches_float64_softmax(oracle_mod, beta, T):
    rng = np.random.default_rng(2)
    V = 517
    L, P, M = (a[0, 0] for a in _rand_rows(rng, 1, 0, V))
    got = oracle_mod.row(L, P, M, beta=beta, temperature=T)
    l, p, m = (torch.from_numpy(a).double() / T for a in (L, P, M))
    h_rec = l + beta * (p - m)                                   # Eq. 8 (tempered)
    np.testing.assert_allclose(got["logp_star"], torch.log_softmax(h_rec, 0).numpy(), atol=1e-12)
    want_lse = [torch.logsumexp(x, 0).item() for x in (l, p, m, h_rec)]
    np.testing.assert_allclose(got["lse"], want_lse, atol=1e-12)
    assert got["W"] == pytest.approx(1.0, abs=1e-12)             # distributions sum to 1
    np.testing.assert_allclose(got["weights"], torch.softmax(h_rec, 0).numpy(), atol=1e-14)
    # adding a constant to any logit row changes nothing
    got2 = oracle_mod.row(L + np.float32(3.0), P - np.float32(2.0), M + np.float32(1.0), beta=beta, temperature=T)
    np.testing.assert_allclose(got2["logp_star"], got["logp_star"], atol=2e-6)


def test_log_z_is_partition_function_of_eq2(oracle_mod):
    """log_z = log sum_v P_LLM(v) (P+(v)/P-(v))^beta, computed here from probabilities (Eq. 2, Eq. 3)."""
    rng = np.random.default_rng(3)
    B, K, V = 3, 2, 64
    L, P, M = _rand_rows(rng, B, K, V)
    tok = rng.integers(0, V, (B, K)).astype(np.int32)
    beta = np.array([1.0, 0.5, 2.0], np.float32)
    T = np.array([1.0, 0.7, 1.3], np.float32)
    length = np.array([2, 1, 2], np.int32)
    u_acc = np.array([[0.0, 1.0], [0.0, 0.0], [0.0, 0.0]], np.float32)     # request 0 is rejected at position 1
    out = _round(oracle_mod, L, P, M, tok, u_acc, rng.random(B, np.float32),
                 lam=np.array([1e6, 0.5, 0.5], np.float32), beta=beta, T=T, length=length, flags=oracle_mod.FLAG_BONUS)
    assert out["accept_len"].tolist() == [1, 1, 2]
    for b in range(B):
        pl, pp, pm = (sps.softmax(a[b].astype(np.float64) / float(T[b]), axis=-1) for a in (L, P, M))
        z = (pl * (pp / pm) ** float(beta[b])).sum(-1)
        # rows 0 .. draft_len: with the bonus row part of the round, its log Z_t is reported whatever accept_len is
        # (request 0 stops at position 1 and still reports row 2); rows beyond draft_len are not read
        ln = int(length[b])
        np.testing.assert_allclose(out["log_z"][b, :ln + 1], np.log(z[:ln + 1]), atol=1e-10)
        assert np.isnan(out["log_z"][b, ln + 1:]).all()
        for t in range(ln):
            y = tok[b, t]
            assert out["logp_llm"][b, t] == pytest.approx(np.log(pl[t, y]), abs=1e-10)
            assert out["logp_plus"][b, t] == pytest.approx(np.log(pp[t, y]), abs=1e-10)
            assert out["logp_minus"][b, t] == pytest.approx(np.log(pm[t, y]), abs=1e-10)
            ps = pl[t] * (pp[t] / pm[t]) ** float(beta[b]) / z[t]
            assert out["logp_star"][b, t] == pytest.approx(np.log(ps[y]), abs=1e-10)


# ---------------------------------------------------------------- hand-derived rationals
def _gold_rows(K):
    g = json.load(open(GOLD))
    L = np.log(np.array(g["p_llm"], np.float64)).astype(np.float32)
    P = np.log(np.array(g["p_plus"], np.float64)).astype(np.float32)
    M = np.log(np.array(g["p_minus"], np.float64)).astype(np.float32)
    rep = lambda a: np.tile(a, (1, K + 1, 1))
    return g, rep(L), rep(P), rep(M)


def test_golden_acceptance_probabilities(oracle_mod):
    g, L, P, M = _gold_rows(4)
    tok = np.array([[0, 1, 2, 3]], np.int32)
    u = np.zeros((1, 4), np.float32)
    for lam, key in ((1.0, "eq7_ratio_lambda_1"), (0.5, "eq7_ratio_lambda_half"), (4.0, "eq7_ratio_lambda_4")):
        out = _round(oracle_mod, L, P, M, tok, u, np.zeros(1, np.float32), lam=lam)
        np.testing.assert_allclose(out["alpha"][0], g[key]["alpha"], atol=1e-7)
    out = _round(oracle_mod, L, P, M, tok, u, np.zeros(1, np.float32), lam=1.0,
                 accept_mode=oracle_mod.ACCEPT_EXACT_Z)
    np.testing.assert_allclose(out["alpha"][0], g["eq6_exact_beta_1"]["alpha"], atol=1e-7)
    np.testing.assert_allclose(out["log_z"][0, :4], np.log(g["eq4_fused_beta_1"]["z"]), atol=1e-7)
    np.testing.assert_allclose(np.exp(out["logp_star"][0]), g["eq4_fused_beta_1"]["p_star"], atol=1e-7)


def test_golden_recovery_distributions(oracle_mod):
    g, L, P, M = _gold_rows(0)
    l, p, m = L[0, 0], P[0, 0], M[0, 0]
    r = oracle_mod.row(l, p, m, beta=1.0)
    np.testing.assert_allclose(r["weights"], g["eq4_fused_beta_1"]["p_star"], atol=1e-7)
    r = oracle_mod.row(l, p, m, beta=0.0)
    np.testing.assert_allclose(r["weights"], g["eq8_beta_0"]["p_rec"], atol=1e-7)
    r = oracle_mod.row(l, p, m, beta=2.0)
    np.testing.assert_allclose(r["weights"], g["eq8_beta_2"]["p_rec"], atol=1e-7)
    assert r["lse"][3] - r["lse"][0] - 2.0 * (r["lse"][1] - r["lse"][2]) == pytest.approx(np.log(g["eq8_beta_2"]["z"]), abs=1e-7)
    r = oracle_mod.row(l, p, m, beta=0.0, temperature=0.5)
    np.testing.assert_allclose(r["weights"], g["temperature_half_beta_0"]["p_rec"], atol=1e-7)
    r = oracle_mod.row(l, p, m, beta=1.0, recover_mode=oracle_mod.RECOVER_RESIDUAL)
    assert r["W"] == pytest.approx(g["residual_beta_1"]["sum"], abs=1e-7)
    np.testing.assert_allclose(r["weights"] / r["W"], g["residual_beta_1"]["dist"], atol=1e-6)


def test_golden_sequence_break_and_inverse_cdf(oracle_mod):
    """Algorithm 1: accept while u <= alpha, stop at the first rejection, sample once there."""
    g, L, P, M = _gold_rows(3)
    s = g["sequence"]
    for u_rec, want in zip(s["u_recover"], s["rec_token"]):
        out = _round(oracle_mod, L, P, M, np.array([s["drafts"]], np.int32),
                     np.array([s["u_accept"]], np.float32), np.array([u_rec], np.float32), lam=1.0)
        assert out["accept_len"][0] == s["accept_len"]
        assert list(out["accept_flags"][0]) == [1, 1, 0]
        assert out["rec_token"][0] == want
        assert list(out["out_tokens"][0]) == s["drafts"][:2] + [want, -1]
        assert out["n_out"][0] == 3
    # u equal to alpha is an acceptance ("Uniform(0,1) <= alpha"): alpha is exactly 1 at position 1
    out = _round(oracle_mod, L, P, M, np.array([s["drafts"]], np.int32),
                 np.array([[0.49, 1.0, 0.49]], np.float32), np.array([0.0], np.float32), lam=1.0)
    assert out["accept_len"][0] == 3 and out["rec_token"][0] == -1 and out["n_out"][0] == 3
    # with the bonus flag the row after the drafts yields one more token
    out = _round(oracle_mod, L, P, M, np.array([s["drafts"]], np.int32),
                 np.array([[0.49, 0.0, 0.49]], np.float32), np.array([0.9], np.float32), lam=1.0,
                 flags=oracle_mod.FLAG_BONUS)
    assert out["accept_len"][0] == 3 and out["rec_token"][0] == 3 and out["n_out"][0] == 4


# ---------------------------------------------------------------- special cases of Eq. 7 / Eq. 8
def test_generalist_equals_baseline_accepts_everything(oracle_mod):
    """h_LLM == h_SLM- and lambda <= 1 make every ratio >= 1 (Eq. 7); and P* = P+ = Q (Eq. 4)."""
    rng = np.random.default_rng(5)
    B, K, V = 4, 5, 300
    L, P, _ = _rand_rows(rng, B, K, V)
    tok = rng.integers(0, V, (B, K)).astype(np.int32)
    u = np.nextafter(np.float32(1), np.float32(0)) * np.ones((B, K), np.float32)
    for lam in (1.0, 0.5):
        out = _round(oracle_mod, L, P, L.copy(), tok, u, rng.random(B, np.float32), lam=lam)
        assert (out["accept_len"] == K).all() and (out["alpha"] == 1.0).all()
    out = _round(oracle_mod, L, P, L.copy(), tok, u, rng.random(B, np.float32), lam=1.0,
                 accept_mode=oracle_mod.ACCEPT_EXACT_Z)
    np.testing.assert_allclose(out["logp_star"], out["logp_plus"], atol=1e-10)
    np.testing.assert_allclose(out["log_z"][:, :K], 0.0, atol=1e-10)
    assert (out["accept_len"] == K).all()


def test_no_private_context_means_zero_reward(oracle_mod):
    """h_SLM+ == h_SLM- gives r == 0 (Eq. 3): P* = P_LLM, Z = 1, recovery = the standard fallback."""
    rng = np.random.default_rng(6)
    L, P, _ = _rand_rows(rng, 2, 3, 100)
    tok = rng.integers(0, 100, (2, 3)).astype(np.int32)
    out = _round(oracle_mod, L, P, P.copy(), tok, rng.random((2, 3), np.float32), rng.random(2, np.float32),
                 beta=1.7)
    np.testing.assert_allclose(out["logp_star"], out["logp_llm"], atol=1e-10)
    np.testing.assert_allclose(out["log_z"][:, :3], 0.0, atol=1e-10)


def test_alpha_monotone_in_lambda(oracle_mod):
    rng = np.random.default_rng(7)
    L, P, M = _rand_rows(rng, 8, 4, 64)
    tok = rng.integers(0, 64, (8, 4)).astype(np.int32)
    u = rng.random((8, 4), np.float32)
    prev = None
    for lam in (1e-6, 0.01, 0.1, 0.5, 1.0, 4.0):
        out = _round(oracle_mod, L, P, M, tok, u, rng.random(8, np.float32), lam=lam)
        if prev is not None:
            assert (out["alpha"] <= prev + 1e-15).all()
        prev = out["alpha"]
        if lam == 1e-6:
            assert (out["accept_len"] == 4).all()
    ratio = np.exp(out["logp_llm"] - out["logp_minus"]) / 4.0
    np.testing.assert_allclose(out["alpha"], np.minimum(1.0, ratio), rtol=1e-12)


def test_standard_speculative_decoding_special_case(oracle_mod):
    """h_SLM- := h_SLM+, lambda = 1, beta = 0, RESIDUAL is textbook speculative sampling with target P_LLM."""
    rng = np.random.default_rng(8)
    V = 50
    L, P, _ = _rand_rows(rng, 1, 1, V)
    pl, pp = sps.softmax(L[0, 0].astype(np.float64)), sps.softmax(P[0, 0].astype(np.float64))
    res = np.maximum(0.0, pl - pp)
    for y in range(V):
        out = _round(oracle_mod, L, P, P.copy(), np.array([[y]], np.int32), np.array([[0.999999]], np.float32),
                     np.array([0.37], np.float32), lam=1.0, beta=0.0, recover_mode=oracle_mod.RECOVER_RESIDUAL)
        assert out["alpha"][0, 0] == pytest.approx(min(1.0, pl[y] / pp[y]), rel=1e-10)
        if out["accept_len"][0] == 0:
            want = int(np.searchsorted(np.cumsum(res), np.float64(np.float32(0.37)) * res.sum(), side="right"))
            assert out["rec_token"][0] == want
            assert out["rec_logprob"][0] == pytest.approx(np.log(res[want] / res.sum()), abs=1e-9)


def test_residual_zero_where_nonpositive(oracle_mod):
    rng = np.random.default_rng(9)
    L, P, M = (a[0, 0] for a in _rand_rows(rng, 1, 0, 400))
    for beta in (0.3, 1.0, 2.0):
        r = oracle_mod.row(L, P, M, beta=beta, recover_mode=oracle_mod.RECOVER_RESIDUAL)
        l, p, m = (torch.from_numpy(a).double() for a in (L, P, M))
        diff = (torch.softmax(l + beta * (p - m), 0) - torch.softmax(p, 0)).numpy()
        assert (r["weights"][diff <= 0] == 0).all()
        np.testing.assert_allclose(r["weights"][diff > 0], diff[diff > 0], atol=1e-15)
        assert r["W"] == pytest.approx(diff[diff > 0].sum(), rel=1e-12)


# ---------------------------------------------------------------- output-token law (Algorithm 1 + Eq. 5)
def _tiny_case(seed, V=8, K=1):
    rng = np.random.default_rng(seed)
    L = rng.standard_normal((K + 1, V)).astype(np.float32) * 1.5
    P = (L + rng.standard_normal((K + 1, V))).astype(np.float32)
    M = (L + 0.7 * rng.standard_normal((K + 1, V))).astype(np.float32)
    return L, P, M


def _closed_form_law(L, P, M, lam, beta, exact, residual):
    """Per row: a(v) = P+(v) alpha(v) (accepted mass per token), reject mass, recovery distribution."""
    l, p, m = (x.astype(np.float64) for x in (L, P, M))
    pl, pp, pm = sps.softmax(l, -1), sps.softmax(p, -1), sps.softmax(m, -1)
    pstar = sps.softmax(l + beta * (p - m), -1)
    alpha = np.minimum(1.0, pstar / pp) if exact else np.minimum(1.0, pl / (lam * pm))
    acc = pp * alpha
    rec = pstar
    if residual:
        res = np.maximum(0.0, pstar - pp)
        rec = np.where(res.sum(-1, keepdims=True) > 0, res / np.maximum(res.sum(-1, keepdims=True), 1e-300), pstar)
    return acc, 1.0 - acc.sum(-1), rec, pstar


@pytest.mark.parametrize("exact,residual", [(False, False), (True, True)])
def test_single_position_law_by_exhaustive_grid(oracle_mod, exact, residual):
    """V=8, K=1: enumerate every draft token and a midpoint grid of both uniforms; the weighted histogram of
    the emitted token must equal P_out(y) = P+(y) alpha(y) + (1 - sum_v P+(v) alpha(v)) P_rec(y).  With the exact
    rule and the residual this is the speculative-sampling theorem: P_out = P* = Softmax(h_rec)."""
    V, lam, beta, n = 8, 0.8, 1.3, 256
    L, P, M = _tiny_case(11, V, 1)
    acc, rej, rec, pstar = _closed_form_law(L[0], P[0], M[0], lam, beta, exact, residual)
    want = acc + rej * rec
    if exact and residual:
        np.testing.assert_allclose(want, pstar, atol=1e-12)       # the theorem itself
    grid = ((np.arange(n) + 0.5) / n).astype(np.float32)
    ua, ur = np.meshgrid(grid, grid, indexing="ij")
    B = n * n
    pp = sps.softmax(P[0].astype(np.float64))
    hist = np.zeros(V)
    for y in range(V):
        out = oracle_mod.verify_recover_round(
            np.broadcast_to(L, (B, 2, V)).copy(), np.broadcast_to(P, (B, 2, V)).copy(),
            np.broadcast_to(M, (B, 2, V)).copy(), np.full((B, 1), y, np.int32), np.ones(B, np.int32),
            np.full(B, lam, np.float32), np.full(B, beta, np.float32), np.ones(B, np.float32),
            ua.reshape(B, 1), ur.reshape(B),
            accept_mode=oracle_mod.ACCEPT_EXACT_Z if exact else oracle_mod.ACCEPT_RATIO,
            recover_mode=oracle_mod.RECOVER_RESIDUAL if residual else oracle_mod.RECOVER_STEER, nthreads=4)
        emitted = out["out_tokens"][:, 0]
        assert (out["n_out"] == 1).all()
        hist += pp[y] * np.bincount(emitted, minlength=V) / B
    np.testing.assert_allclose(hist, want, atol=2.0 / n)


def test_multi_position_law_monte_carlo(oracle_mod):
    """V=8, K=3, 10^6 rounds with fresh drafts and uniforms: accepted-length law P(n>=t) = prod_{i<t} a_i and the
    joint law of (n, recovered token) = prod_{i<n} a_i (1-a_n) P_rec,n(y)."""
    V, K, N, lam, beta = 8, 3, 1_000_000, 0.7, 1.0
    L, P, M = _tiny_case(12, V, K)
    acc, rej, rec, _ = _closed_form_law(L, P, M, lam, beta, False, False)
    a = acc.sum(-1)
    rng = np.random.default_rng(13)
    pp = sps.softmax(P.astype(np.float64), -1)
    tok = np.stack([rng.choice(V, size=N, p=pp[t]) for t in range(K)], 1).astype(np.int32)
    out = oracle_mod.verify_recover_round(
        np.broadcast_to(L, (N, K + 1, V)).copy(), np.broadcast_to(P, (N, K + 1, V)).copy(),
        np.broadcast_to(M, (N, K + 1, V)).copy(), tok, np.full(N, K, np.int32),
        np.full(N, lam, np.float32), np.full(N, beta, np.float32), np.ones(N, np.float32),
        rng.random((N, K), np.float32), rng.random(N, np.float32), flags=oracle_mod.FLAG_BONUS, nthreads=8)
    n = out["accept_len"]
    reach = np.concatenate([[1.0], np.cumprod(a[:K])])
    want_n = np.array([reach[t] * (1 - a[t]) for t in range(K)] + [reach[K]])
    got_n = np.bincount(n, minlength=K + 1) / N
    np.testing.assert_allclose(got_n, want_n, atol=5.0 / np.sqrt(N))
    for t in range(K + 1):
        sel = n == t
        got = np.bincount(out["rec_token"][sel], minlength=V) / N
        np.testing.assert_allclose(got, want_n[t] * rec[t], atol=5.0 / np.sqrt(N))
    # accepted draft tokens at position 0 follow P+(v) alpha(v)
    got0 = np.bincount(tok[n >= 1, 0], minlength=V) / N
    np.testing.assert_allclose(got0, acc[0], atol=5.0 / np.sqrt(N))


# ---------------------------------------------------------------- defined behaviour on degenerate input
def test_status_words_and_degenerate_inputs(oracle_mod):
    o = oracle_mod
    rng = np.random.default_rng(14)
    B, K, V = 6, 2, 16
    L, P, M = _rand_rows(rng, B, K, V)
    tok = rng.integers(0, V, (B, K)).astype(np.int32)
    tok[0, 0] = V                     # bad token -> rejection with alpha 0 at that position
    length = np.array([K, K + 1, K, K, 0, K], np.int32)   # request 1: bad length -> treated as 0
    L[2, 1, 3] = np.nan               # request 2: non-finite row 1
    T = np.array([1, 1, 1, 0.0, 1, 1], np.float32)        # request 3: bad temperature
    L[5, 0, :] = -np.inf              # request 5: an empty distribution
    u = np.zeros((B, K), np.float32)
    out = _round(o, L, P, M, tok, u, np.full(B, 0.5, np.float32), T=T, length=length, flags=o.FLAG_BONUS)
    assert out["req_status"][0] == o.REQ_BAD_TOKEN and out["accept_len"][0] == 0 and out["alpha"][0, 0] == 0
    assert out["rec_token"][0] >= 0 and out["n_out"][0] == 1
    assert out["req_status"][1] == o.REQ_BAD_LEN and out["accept_len"][1] == 0 and out["n_out"][1] == 1
    assert out["req_status"][2] == o.REQ_NONFINITE and out["accept_len"][2] == 1
    assert out["rec_token"][2] == -1 and out["n_out"][2] == 1
    assert out["req_status"][3] == o.REQ_BAD_PARAM and out["n_out"][3] == 0 and out["rec_token"][3] == -1
    assert out["req_status"][4] == 0 and out["accept_len"][4] == 0 and out["n_out"][4] == 1
    assert out["req_status"][5] == o.REQ_NONFINITE and out["accept_len"][5] == 0 and out["n_out"][5] == 0
    # every problem a request shows is reported: a bad length together with a bad parameter gives both bits
    length[3] = -1
    out = _round(o, L, P, M, tok, u, np.full(B, 0.5, np.float32), T=T, length=length, flags=o.FLAG_BONUS)
    assert out["req_status"][3] == (o.REQ_BAD_PARAM | o.REQ_BAD_LEN) and out["n_out"][3] == 0 and out["accept_len"][3] == 0


# ---------------------------------------------------------------- the round reading what Algorithm 1 reads
def test_alg1_reads_equals_the_full_round_on_finite_inputs(oracle_mod):
    """Algorithm 1 Phase 2 uses P_LLM and P_SLM- only (Eq. 7) and Phase 3 the three logit rows of one position
    (Eq. 8).  On finite inputs the round that reads nothing else decides, samples and reports exactly what the full
    round does; what it never forms (logp_plus, logp_star, log_z) stays NaN.  Acceptance against scipy's softmax."""
    o = oracle_mod
    rng = np.random.default_rng(50)
    B, K, V = 12, 3, 97
    L, P, M = _rand_rows(rng, B, K, V)
    tok = rng.integers(0, V, (B, K)).astype(np.int32)
    ua, ur = rng.random((B, K)).astype(np.float32), rng.random(B).astype(np.float32)
    length = rng.integers(0, K + 1, B).astype(np.int32)
    beta = rng.choice([0.5, 1.0, 2.0], B).astype(np.float32)
    T = rng.choice([0.7, 1.0], B).astype(np.float32)
    lam = rng.choice([0.5, 2.0, 8.0], B).astype(np.float32)
    for rmode in (o.RECOVER_STEER, o.RECOVER_ARGMAX):
        for fl in (0, o.FLAG_BONUS):
            full = _round(o, L, P, M, tok, ua, ur, lam=lam, beta=beta, T=T, length=length, recover_mode=rmode, flags=fl)
            alg1 = _round(o, L, P, M, tok, ua, ur, lam=lam, beta=beta, T=T, length=length, recover_mode=rmode,
                          flags=fl | o.FLAG_ALG1_READS)
            for k in ("accept_len", "accept_flags", "alpha", "logp_llm", "logp_minus", "rec_token", "rec_logprob",
                      "out_tokens", "n_out", "req_status", "accept_margin", "cdf_margin"):
                assert np.array_equal(full[k], alg1[k], equal_nan=True), k
            for k in ("logp_plus", "logp_star", "log_z"):
                assert np.isnan(alg1[k]).all(), k
    assert (full["accept_len"] < length).any() and (full["accept_len"] == length).any()
    for b in range(B):
        pl = sps.softmax(L[b].astype(np.float64) / float(T[b]), -1)
        pm = sps.softmax(M[b].astype(np.float64) / float(T[b]), -1)
        for t in range(int(length[b])):
            y = tok[b, t]
            assert alg1["alpha"][b, t] == pytest.approx(min(1.0, pl[t, y] / (float(lam[b]) * pm[t, y])), abs=1e-12)   # Eq. 7


def test_alg1_reads_never_touches_h_slm_plus_on_drafted_rows(oracle_mod):
    """NaN in h_SLM+ everywhere except the row the new token comes from changes nothing; NaN or +inf on that row
    is a non-finite recovery row; Eq. 6 cannot be asked of this round."""
    o = oracle_mod
    rng = np.random.default_rng(51)
    B, K, V = 10, 3, 61
    L, P, M = _rand_rows(rng, B, K, V)
    tok = rng.integers(0, V, (B, K)).astype(np.int32)
    ua, ur = rng.random((B, K)).astype(np.float32), rng.random(B).astype(np.float32)
    for fl in (0, o.FLAG_BONUS):
        clean = _round(o, L, P, M, tok, ua, ur, lam=2.0, flags=fl | o.FLAG_ALG1_READS)
        Pn = np.full_like(P, np.nan)
        for b in range(B):
            Pn[b, clean["accept_len"][b]] = P[b, clean["accept_len"][b]]
        got = _round(o, L, Pn, M, tok, ua, ur, lam=2.0, flags=fl | o.FLAG_ALG1_READS)
        for k in clean:
            assert np.array_equal(clean[k], got[k], equal_nan=True), k
        assert (got["req_status"] == 0).all()
        # the full round sees the poison on the first drafted row
        assert (_round(o, L, Pn, M, tok, ua, ur, lam=2.0, flags=fl)["req_status"][clean["accept_len"] > 0] == o.REQ_NONFINITE).all()
        assert (clean["accept_len"] > 0).any() and (clean["accept_len"] < K).any()
    b = int(np.argmax(clean["rec_token"] >= 0))
    Pbad = P.copy()
    Pbad[b, clean["accept_len"][b], 7] = np.inf
    got = _round(o, L, Pbad, M, tok, ua, ur, lam=2.0, flags=o.FLAG_BONUS | o.FLAG_ALG1_READS)
    assert got["req_status"][b] == o.REQ_NONFINITE and got["rec_token"][b] == -1
    assert got["accept_len"][b] == clean["accept_len"][b] and got["n_out"][b] == clean["accept_len"][b]
    with pytest.raises(RuntimeError):
        _round(o, L, P, M, tok, ua, ur, accept_mode=o.ACCEPT_EXACT_Z, flags=o.FLAG_ALG1_READS)


def test_forced_decisions_and_margins(oracle_mod):
    g, L, P, M = _gold_rows(2)
    tok = np.array([[2, 3]], np.int32)
    u = np.array([[0.5 + 4e-6, 0.2]], np.float32)     # alpha = 0.5 at lambda=1: a rejection by a hair
    out = _round(oracle_mod, L, P, M, tok, u, np.array([0.5 - 2e-6], np.float32), lam=1.0)
    assert out["accept_len"][0] == 0 and out["accept_margin"][0, 0] < 1e-5
    assert out["cdf_margin"][0] < 1e-5 and out["rec_token"][0] == 1
    assert out["rec_token_lo"][0] == 1 and out["rec_token_hi"][0] == 2
    forced = _round(oracle_mod, L, P, M, tok, u, np.array([0.9], np.float32), lam=1.0,
                    force_accept=np.array([[1, -1]], np.int8))
    assert forced["accept_len"][0] == 2


# ---------------------------------------------------------------- greedy recovery (the paper decodes greedily)
def _grid_rows(rng, B, K, V, q=4, lo=-8, hi=8):
    """Rows on a grid of 1/q: every h_rec with beta in {0, 0.5, 1, 2} is exact in float32, ties are frequent."""
    f = lambda: (rng.integers(lo * q, hi * q, size=(B, K + 1, V)) / q).astype(np.float32)
    return f(), f(), f()


@pytest.mark.parametrize("beta", [0.0, 0.5, 1.0, 2.0])
def test_argmax_recovery_is_the_first_maximiser_of_h_rec(oracle_mod, beta):
    """Eq. 8 under greedy decoding, by exhaustive search with exact rationals (lowest id among equals); the accept
    decisions are those of the sampling round."""
    from fractions import Fraction
    o = oracle_mod
    rng = np.random.default_rng(40)
    B, K, V = 6, 3, 23
    L, P, M = _grid_rows(rng, B, K, V)
    tok = rng.integers(0, V, (B, K)).astype(np.int32)
    ua, ur = rng.random((B, K)).astype(np.float32), rng.random(B).astype(np.float32)
    g = _round(o, L, P, M, tok, ua, ur, beta=beta, recover_mode=o.RECOVER_ARGMAX, flags=o.FLAG_BONUS)
    s = _round(o, L, P, M, tok, ua, ur, beta=beta, recover_mode=o.RECOVER_STEER, flags=o.FLAG_BONUS)
    for k in ("accept_len", "accept_flags", "alpha", "logp_llm", "logp_minus", "log_z", "req_status"):
        assert np.array_equal(g[k], s[k], equal_nan=True), k
    for b in range(B):
        n = int(g["accept_len"][b])
        h = [Fraction(float(L[b, n, v])) + Fraction(beta) * (Fraction(float(P[b, n, v])) - Fraction(float(M[b, n, v])))
             for v in range(V)]
        want = min(range(V), key=lambda v: (-h[v], v))
        assert g["rec_token"][b] == want and g["n_out"][b] == n + 1
        assert g["out_tokens"][b][n] == want and (g["out_tokens"][b][:n] == tok[b][:n]).all()
        hr = np.array([float(x) for x in h])
        assert g["rec_logprob"][b] == pytest.approx(sps.log_softmax(hr)[want], abs=1e-12)
        runner_up = max(h[v] for v in range(V) if v != want)
        assert g["cdf_margin"][b] == float(h[want] - runner_up)       # the gap to the runner-up, exact on this grid
        assert g["rec_token_lo"][b] == want                           # float32 forms these values exactly too


def test_argmax_recovery_with_beta_zero_is_numpy_argmax_of_the_generalist(oracle_mod):
    o = oracle_mod
    rng = np.random.default_rng(41)
    L, P, M = _rand_rows(rng, 5, 2, 4001)
    tok = rng.integers(0, 4001, (5, 2)).astype(np.int32)
    g = _round(o, L, P, M, tok, np.ones((5, 2), np.float32), rng.random(5).astype(np.float32), beta=0.0,
               recover_mode=o.RECOVER_ARGMAX)          # u = 1: the first draft is rejected unless alpha = 1
    for b in range(5):
        n = int(g["accept_len"][b])
        if g["rec_token"][b] >= 0:
            assert g["rec_token"][b] == int(np.argmax(L[b, n]))


def test_argmax_recovery_ignores_the_temperature_but_reports_the_tempered_probability(oracle_mod):
    o = oracle_mod
    rng = np.random.default_rng(42)
    L, P, M = _rand_rows(rng, 4, 1, 999)
    tok = np.zeros((4, 1), np.int32)
    ua, ur = np.ones((4, 1), np.float32), np.zeros(4, np.float32)
    toks = []
    for T in (0.25, 1.0, 3.0):
        g = _round(o, L, P, M, tok, ua, ur, beta=1.5, T=T, length=[0, 0, 0, 0], recover_mode=o.RECOVER_ARGMAX,
                   flags=o.FLAG_BONUS)
        toks.append(g["rec_token"].copy())
        for b in range(4):
            hr = (L[b, 0].astype(np.float64) + 1.5 * (P[b, 0].astype(np.float64) - M[b, 0].astype(np.float64))) / T
            assert g["rec_logprob"][b] == pytest.approx(sps.log_softmax(hr)[g["rec_token"][b]], abs=1e-9)
    assert np.array_equal(toks[0], toks[1]) and np.array_equal(toks[1], toks[2])


def test_argmax_recovery_orders_h_rec_over_the_reals_and_reports_what_single_precision_would_do(oracle_mod):
    """Two entries whose exact h_rec differ by 2^-30 (Eq. 8 is a statement about real numbers): the larger one is
    the token, the gap is 2^-30, and the token single precision would order first - there the two are equal, so the
    lower id - is reported beside it without deciding anything.  A difference float32 resolves moves both."""
    o = oracle_mod
    L = np.array([[[1.0, 1.0, 0.0]]], np.float32)
    P = np.array([[[0.0, 2.0 ** -30, 0.0]]], np.float32)
    M = np.zeros((1, 1, 3), np.float32)
    kw = dict(tok=np.zeros((1, 0), np.int32), u_acc=np.zeros((1, 0), np.float32), u_rec=np.zeros(1, np.float32),
              recover_mode=o.RECOVER_ARGMAX, flags=o.FLAG_BONUS)
    g = _round(o, L, P, M, **kw)
    assert g["rec_token"][0] == 1 and g["cdf_margin"][0] == 2.0 ** -30 and g["rec_token_lo"][0] == 0
    assert g["out_tokens"][0][0] == 1 and g["rec_token_hi"][0] == 1
    assert g["rec_logprob"][0] == pytest.approx(sps.log_softmax(np.array([1.0, 1.0 + 2.0 ** -30, 0.0]))[1], abs=1e-15)
    P[0, 0, 1] = 2.0 ** -20
    g = _round(o, L, P, M, **kw)
    assert g["rec_token"][0] == 1 and g["rec_token_lo"][0] == 1 and g["cdf_margin"][0] == 2.0 ** -20
    # bf16 logits go the same way (their values are exact in both precisions)
    bits = lambda a: (a.view(np.uint32) >> 16).astype(np.uint16)
    P[0, 0, 1] = 2.0 ** -30
    g = _round(o, bits(L), bits(P), bits(M), **kw)
    assert g["rec_token"][0] == 1 and g["rec_token_lo"][0] == 0 and g["cdf_margin"][0] == 2.0 ** -30


def test_argmax_recovery_on_float32_logits_is_numpy_argmax_in_double(oracle_mod):
    """Random float32 rows, several beta: the token is numpy's argmax of h_rec formed in double, the gap the
    difference of its two largest values."""
    o = oracle_mod
    rng = np.random.default_rng(44)
    B, V = 5, 2003
    L, P, M = _rand_rows(rng, B, 0, V)
    beta = np.array([1.0, 0.5, 2.0, 0.3, 2.7], np.float32)
    g = _round(o, L, P, M, np.zeros((B, 0), np.int32), np.zeros((B, 0), np.float32), np.zeros(B, np.float32), beta=beta,
               recover_mode=o.RECOVER_ARGMAX, flags=o.FLAG_BONUS)
    for b in range(B):
        r = L[b, 0].astype(np.float64) + float(beta[b]) * (P[b, 0].astype(np.float64) - M[b, 0].astype(np.float64))
        assert g["rec_token"][b] == int(np.argmax(r))
        top2 = np.sort(r)[-2:]
        assert g["cdf_margin"][b] == pytest.approx(top2[1] - top2[0], abs=1e-15)


def test_argmax_recovery_on_float64_logits_orders_in_double_and_reports_the_gap(oracle_mod):
    """Logits that were themselves computed (float64): numpy's argmax of h_rec in double, lowest id among equals, and
    the distance to the runner-up in cdf_margin."""
    o = oracle_mod
    rng = np.random.default_rng(43)
    B, V = 4, 3001
    L, P, M = (rng.standard_normal((B, 1, V)) * 2 for _ in range(3))
    L[1, 0, 77] = L[1, 0, 2000] = 50.0                  # an exact tie between two ids: the lower one, gap 0
    P[1, 0, 77] = P[1, 0, 2000] = M[1, 0, 77] = M[1, 0, 2000] = 0.0
    beta = np.array([1.0, 0.5, 2.0, 0.0], np.float32)
    g = o.verify_recover_round(L, P, M, np.zeros((B, 0), np.int32), np.zeros(B, np.int32), np.ones(B, np.float32), beta,
                               np.ones(B, np.float32), np.zeros((B, 0), np.float32), np.zeros(B, np.float32),
                               recover_mode=o.RECOVER_ARGMAX, flags=o.FLAG_BONUS)
    for b in range(B):
        r = L[b, 0] + float(beta[b]) * (P[b, 0] - M[b, 0])
        assert g["rec_token"][b] == int(np.argmax(r))
        top2 = np.sort(r)[-2:]
        assert g["cdf_margin"][b] == pytest.approx(top2[1] - top2[0], abs=1e-15)
        assert g["rec_logprob"][b] == pytest.approx(sps.log_softmax(r)[g["rec_token"][b]], abs=1e-12)
    assert g["rec_token"][1] == 77 and g["cdf_margin"][1] == 0.0
    f = o.verify_recover_round(L.astype(np.float32), P.astype(np.float32), M.astype(np.float32), np.zeros((B, 0), np.int32),
                               np.zeros(B, np.int32), np.ones(B, np.float32), beta, np.ones(B, np.float32),
                               np.zeros((B, 0), np.float32), np.zeros(B, np.float32), recover_mode=o.RECOVER_ARGMAX,
                               flags=o.FLAG_BONUS)
    assert np.isfinite(f["cdf_margin"]).all() and f["cdf_margin"][1] == 0.0 and f["rec_token"][1] == 77
