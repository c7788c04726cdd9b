"""Pins of the LM-head step of the oracle: h = x W^T from bf16 hidden states and head weights (the logits that
Algorithm 1's verification and recovery steps read), in float64, followed by the round as it stands.

Each test ties the new code to something other than itself: IEEE bit patterns, exact rational arithmetic,
one-hot heads whose logits are the hidden states themselves, a first-order closed form that only float64 logits
can satisfy, and the float32 round (pinned elsewhere) on logits that both representations hold exactly.
"""
from fractions import Fraction

import numpy as np
import pytest


@pytest.fixture(scope="module")
def o(oracle_mod):
    return oracle_mod


def _bf16_bits(a):
    """bf16 bit patterns of float32 values that are exactly representable in bf16."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32)
    assert ((bits & 0xffff) == 0).all(), "value is not a bf16 number"
    return (bits >> 16).astype(np.uint16)


def _grid(rng, shape, q=8, lo=-4, hi=4):
    """Multiples of 1/q in [lo, hi): at most 7 significant bits, so exactly bf16."""
    return (rng.integers(lo * q, hi * q, size=shape) / q).astype(np.float32)


def test_bf16_decode_against_ieee_bit_patterns(o):
    bits = np.array([0x3F80, 0xC000, 0x3FC0, 0x0000, 0x8000, 0x0001, 0x0080, 0x7F7F, 0x7F80, 0xFF80], np.uint16)
    want = [1.0, -2.0, 1.5, 0.0, -0.0, 2.0 ** -133, 2.0 ** -126, (2 - 2.0 ** -7) * 2.0 ** 127, np.inf, -np.inf]
    got = o.bf16_to_f64(bits)
    assert got.tolist() == want
    assert np.signbit(got[4]) and not np.signbit(got[3])
    assert np.isnan(o.bf16_to_f64(np.array([0x7FC0], np.uint16))[0])


def test_lmhead_logits_against_exact_rational_arithmetic(o):
    rng = np.random.default_rng(0)
    x = _grid(rng, (3, 5))            # 3 rows, d = 5
    w = _grid(rng, (7, 5))            # V = 7: no two extents agree, a transposed operand cannot pass
    h = o.lmhead_logits(_bf16_bits(x), _bf16_bits(w))
    assert h.shape == (3, 7) and h.dtype == np.float64
    for r in range(3):
        for v in range(7):
            exact = sum(Fraction(float(x[r, i])) * Fraction(float(w[v, i])) for i in range(5))
            assert Fraction(float(h[r, v])) == exact


def test_lmhead_logits_keep_the_leading_axes(o):
    rng = np.random.default_rng(1)
    x = _grid(rng, (2, 3, 4))
    w = _grid(rng, (6, 4))
    h = o.lmhead_logits(_bf16_bits(x), _bf16_bits(w))
    assert h.shape == (2, 3, 6)
    for b in range(2):
        for t in range(3):
            assert (h[b, t] == o.lmhead_logits(_bf16_bits(x[b, t][None]), _bf16_bits(w))[0]).all()


def test_one_hot_head_returns_the_hidden_state(o):
    rng = np.random.default_rng(2)
    x = _grid(rng, (4, 6))
    perm = rng.permutation(6)
    w = np.zeros((6, 6), np.float32)
    w[np.arange(6), perm] = 2.0       # row v of the head picks hidden dimension perm[v], doubled
    h = o.lmhead_logits(_bf16_bits(x), _bf16_bits(w))
    assert (h == 2.0 * x[:, perm].astype(np.float64)).all()


def test_float64_logits_are_not_rounded_to_float32(o):
    """Logits c + d_v with |d_v| far below float32 resolution: log sum exp = c + log V + mean(d) to first order,
    which a decode through float32 (where every d_v vanishes) misses by mean(d)."""
    V, c = 1000, 3.0
    d = 1e-9 * (np.arange(V) - 200.0)
    h = c + d
    r = o.row(h, h, h, beta=1.0, temperature=1.0)
    want = c + np.log(V) + d.mean() + 0.5 * d.var()
    assert abs(r["lse"][0] - want) < 1e-13
    assert abs(d.mean()) > 1e-7       # the float32 reading would be off by this much
    # and log Softmax(h_rec) with h_rec = h: entry v differs from the uniform law by d_v - mean(d)
    assert np.abs(r["logp_star"] - (-np.log(V) + d - d.mean())).max() < 1e-13


def test_float64_round_equals_float32_round_on_float32_values(o, tmp_path):
    rng = np.random.default_rng(3)
    B, K, V = 5, 3, 257
    hl = rng.normal(0, 2, (B, K + 1, V)).astype(np.float32)
    hp = (hl + rng.normal(0, 1, hl.shape)).astype(np.float32)
    hm = (hl + rng.normal(0, 0.5, hl.shape)).astype(np.float32)
    tok = rng.integers(0, V, (B, K)).astype(np.int32)
    dl = np.array([3, 2, 0, 3, 1], np.int32)
    args = (tok, dl, np.full(B, 0.5, np.float32), np.array([1, 0.5, 2, 0, 1.5], np.float32),
            np.array([1, 0.7, 1.3, 1, 0.4], np.float32), rng.random((B, K)).astype(np.float32),
            rng.random(B).astype(np.float32))
    for am, rm in ((o.ACCEPT_RATIO, o.RECOVER_STEER), (o.ACCEPT_EXACT_Z, o.RECOVER_RESIDUAL)):
        a = o.verify_recover_round(hl, hp, hm, *args, accept_mode=am, recover_mode=rm, flags=o.FLAG_BONUS)
        b = o.verify_recover_round(hl.astype(np.float64), hp.astype(np.float64), hm.astype(np.float64), *args,
                                   accept_mode=am, recover_mode=rm, flags=o.FLAG_BONUS)
        for k in a:
            assert np.array_equal(a[k], b[k], equal_nan=True), k


def test_lmhead_round_reduces_to_the_round_on_its_logits(o):
    """Heads and hidden states on a coarse grid: every logit is exact in float32 as well, so the LM-head round
    must reproduce the float32 round on those logits, output by output."""
    rng = np.random.default_rng(4)
    B, K, V, dL, dS = 4, 2, 61, 8, 4
    xl, wl = _grid(rng, (B, K + 1, dL), 4, -2, 2), _grid(rng, (V, dL), 4, -2, 2)
    xp, xm, ws = _grid(rng, (B, K + 1, dS), 4, -2, 2), _grid(rng, (B, K + 1, dS), 4, -2, 2), _grid(rng, (V, dS), 4, -2, 2)
    hl = np.einsum("bti,vi->btv", xl.astype(np.float64), wl.astype(np.float64))
    hp = np.einsum("bti,vi->btv", xp.astype(np.float64), ws.astype(np.float64))
    hm = np.einsum("bti,vi->btv", xm.astype(np.float64), ws.astype(np.float64))
    for h in (hl, hp, hm):
        assert (h.astype(np.float32).astype(np.float64) == h).all()
    tok = rng.integers(0, V, (B, K)).astype(np.int32)
    args = (tok, np.array([2, 1, 2, 0], np.int32), np.full(B, 0.5, np.float32), np.array([1, 2, 0.5, 1], np.float32),
            np.array([1, 0.5, 2, 1], np.float32), rng.random((B, K)).astype(np.float32), rng.random(B).astype(np.float32))
    a = o.lmhead_verify_recover_round(_bf16_bits(xl), _bf16_bits(wl), _bf16_bits(xp), _bf16_bits(ws), _bf16_bits(xm),
                                      _bf16_bits(ws), *args, flags=o.FLAG_BONUS)
    b = o.verify_recover_round(hl.astype(np.float32), hp.astype(np.float32), hm.astype(np.float32), *args,
                               flags=o.FLAG_BONUS)
    for k in a:
        assert np.array_equal(a[k], b[k], equal_nan=True), k
    # a planted mistake must show: the two small models' hidden states exchanged
    c = o.lmhead_verify_recover_round(_bf16_bits(xl), _bf16_bits(wl), _bf16_bits(xm), _bf16_bits(ws), _bf16_bits(xp),
                                      _bf16_bits(ws), *args, flags=o.FLAG_BONUS)
    assert not np.allclose(a["logp_plus"], c["logp_plus"], equal_nan=True)
