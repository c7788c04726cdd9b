"""GPU-vs-oracle parity, through the C ABI, on seeded synthetic rounds.

All five configurations are compared request by request in full, in the launch configuration the benchmark
times, in every mode (ratio rule + steering recovery + bonus row; exact rule + residual recovery; the two-phase
round against the oracle round that reads only what Algorithm 1 reads).  Edge cases cover ragged and empty
inputs, tails, unaligned rows and degenerate logits.
"""
import numpy as np
import pytest
import torch

import _parity as P

pytestmark = pytest.mark.gpu

MODES = [("ratio_steer_bonus", 0, 0, 1), ("exact_residual", 1, 1, 0)]


@pytest.fixture(scope="module")
def env(oracle_mod):
    from paper_2603_16219_b200 import binding, build, synth
    assert torch.cuda.is_available(), "these tests need the CUDA device"
    build.build()
    ctx = binding.Context(max_B=8192, max_K=8, max_V=262144, device=0)
    yield {"ctx": ctx, "binding": binding, "synth": synth, "oracle": oracle_mod}
    ctx.close()


def _small(synth, B, K, V, dtype="f32", seed=0, **kw):
    spec = synth.RoundSpec("small", B, K, V, dtype, **kw)
    return spec, synth.make_round(spec, device="cuda", seed=seed)


# ------------------------------------------------------------------ the five configurations
@pytest.mark.parametrize("cfg", [0, 1, 2])
@pytest.mark.parametrize("mode", MODES, ids=[m[0] for m in MODES])
def test_config_full_parity(env, cfg, mode):
    synth = env["synth"]
    spec = synth.CONFIGS[cfg]
    inputs = synth.make_round(spec, device="cuda", seed=0)
    _, am, rm, fl = mode
    gpu = P.run_gpu(env["ctx"], inputs, am, rm, fl)
    stats = P.compare(env["oracle"], gpu, P.to_np_inputs(inputs), am, rm, fl, P.TOL[inputs["h_llm"].dtype])
    print(spec.name, mode[0], stats, "acceptance", gpu["accept_len"].sum() / inputs["draft_len"].sum().item())
    assert stats["excused_accept"] + stats["excused_token"] <= max(1, spec.B // 16)


ALG1_KEYS = ("accept_len", "accept_flags", "alpha", "logp_llm", "logp_minus", "rec_token", "rec_logprob", "out_tokens",
             "n_out", "req_status")


def _two_phase_round(env, inputs, flags, recover_mode=0, force=True):
    """The round asked for Algorithm 1's outputs only; returns (outputs as numpy, launches)."""
    b = env["binding"]
    B, K = inputs["draft_tokens"].shape
    outs = {k: v for k, v in b.alloc_outputs(B, K, "cuda").items() if k in ALG1_KEYS}
    d = b.make_desc(inputs, outs, recover_mode=recover_mode, flags=flags | (b.FLAG_TWO_PHASE if force else 0))
    before = env["ctx"].launch_count
    env["ctx"].verify_round(d)
    env["ctx"].recover_sample(d)
    torch.cuda.synchronize()
    assert env["ctx"].device_error() == 0
    return {k: v.cpu().numpy() for k, v in outs.items()}, env["ctx"].launch_count - before


@pytest.mark.parametrize("cfg", [3, 4])
def test_config_full_size_parity_every_request(env, cfg):
    """The two largest configurations at full size, every request against the oracle, in every mode."""
    synth = env["synth"]
    spec = synth.CONFIGS[cfg]
    inputs = synth.make_round(spec, device="cuda", seed=0)
    npin = P.to_np_inputs(inputs)
    tol = P.TOL[inputs["h_llm"].dtype]
    for name, am, rm, fl in MODES:
        gpu = P.run_gpu(env["ctx"], inputs, am, rm, fl)
        P.invariants(gpu, inputs, fl, tol)
        stats = P.compare(env["oracle"], gpu, npin, am, rm, fl, tol)
        print(spec.name, name, stats, "acceptance", gpu["accept_len"].sum() / inputs["draft_len"].sum().item())
        assert stats["requests"] == spec.B and stats["excused_accept"] + stats["excused_token"] <= spec.B // 64
    # run-to-run determinism on the full-size launch (fixed reduction order everywhere)
    again = P.run_gpu(env["ctx"], inputs, *MODES[1][1:])
    for k in gpu:
        assert np.array_equal(gpu[k], again[k], equal_nan=True), k
    # the launch without the h_SLM+ normaliser (logp_plus and log_z not requested): decisions and tokens equal those
    # of the full launch; the float outputs agree to rounding (a chunk whose h_SLM+ sum overflows the first attempt
    # is redone with per-batch tests in the full launch only, which changes the last bits of that chunk's other sums)
    b = env["binding"]
    full = P.run_gpu(env["ctx"], inputs, 0, 0, 1)
    lean = {k: v for k, v in b.alloc_outputs(spec.B, spec.K, "cuda").items() if k not in ("logp_plus", "log_z")}
    d = b.make_desc(inputs, lean, flags=1)
    env["ctx"].verify_round(d)
    env["ctx"].recover_sample(d)
    torch.cuda.synchronize()
    for k, v in lean.items():
        got = v.cpu().numpy()
        if got.dtype.kind in "iu":
            assert np.array_equal(got, full[k]), k
        else:
            assert np.array_equal(np.isnan(got), np.isnan(full[k])), k
            assert np.nanmax(np.abs(got - full[k]), initial=0.0) <= 1e-5, k
    # the two-phase round (these batches are large enough for it to be automatic): h_LLM and h_SLM- over the drafted
    # rows, then one recovery row per request; every request against the oracle round that reads the same
    alg1, launches = _two_phase_round(env, inputs, 1, force=False)
    assert launches == 5      # row references + stream + epilogue; recovery rows' stream + sampling
    stats = P.compare(env["oracle"], alg1, npin, 0, 0, 1, tol, alg1=True, keys=ALG1_KEYS)
    print(spec.name, "two_phase", stats)
    assert stats["excused_accept"] + stats["excused_token"] <= spec.B // 64


# ------------------------------------------------------------------ shapes, tails, strides
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V", [1, 3, 8, 100, 2047, 2048, 2049, 4100, 6151])
def test_vocabulary_tails(env, V, dtype):
    spec, inputs = _small(env["synth"], 5, 3, V, dtype, seed=V, ragged=True, beta_choices=(0.5, 1.0, 2.0),
                          temp_choices=(0.7, 1.0))
    for _, am, rm, fl in MODES:
        gpu = P.run_gpu(env["ctx"], inputs, am, rm, fl)
        P.compare(env["oracle"], gpu, P.to_np_inputs(inputs), am, rm, fl, P.TOL[inputs["h_llm"].dtype])


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V,ld", [(1000, 1000 + 8), (1001, 1001), (2500, 2503), (4099, 4104)])
def test_row_strides_and_unaligned_rows(env, V, ld, dtype):
    """Row stride > V, and strides that break 16-byte alignment (served by the generic kernel)."""
    spec, inputs = _small(env["synth"], 4, 2, V, dtype, seed=ld)
    for k in ("h_llm", "h_slm_plus", "h_slm_minus"):
        padded = torch.full((4, 3, ld), float("nan"), dtype=inputs[k].dtype, device="cuda")
        padded[:, :, :V] = inputs[k]
        inputs[k] = padded
    gpu = P.run_gpu(env["ctx"], inputs, 0, 0, 1, V=V)
    npin = P.to_np_inputs(inputs)
    P.compare(env["oracle"], gpu, npin, 0, 0, 1, P.TOL[inputs["h_llm"].dtype], V=V)
    # a base pointer that is not 16-byte aligned
    if ld > V:
        shifted = dict(inputs)
        for k in ("h_llm", "h_slm_plus", "h_slm_minus"):
            flat = inputs[k].reshape(-1)
            n = 4 * 3 * ld
            buf = torch.empty(n + 1, dtype=flat.dtype, device="cuda")
            buf[1:] = flat
            shifted[k] = buf[1:].view(4, 3, ld)
        gpu2 = P.run_gpu(env["ctx"], shifted, 0, 0, 1, V=V)
        for key in ("accept_len", "rec_token", "accept_flags"):
            assert np.array_equal(gpu[key], gpu2[key])
        np.testing.assert_allclose(gpu["logp_star"], gpu2["logp_star"], atol=1e-5, equal_nan=True)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_outputs_not_requested_skip_the_plus_normaliser(env, dtype):
    """Algorithm 1 needs the normalisers of h_LLM, h_SLM- (Eq. 7) and h_rec (Eq. 8) only.  Without logp_plus and
    log_z the library does not form the one of h_SLM+; every other output must be unchanged (bit for bit here: no
    chunk of these rows overflows its first attempt)."""
    b = env["binding"]
    spec, inputs = _small(env["synth"], 7, 4, 9001, dtype, seed=21, ragged=True, beta_choices=(0.5, 1.0, 2.0))
    full = b.alloc_outputs(spec.B, spec.K, "cuda")
    lean = {k: v for k, v in b.alloc_outputs(spec.B, spec.K, "cuda").items() if k not in ("logp_plus", "log_z")}
    for outs in (full, lean):
        d = b.make_desc(inputs, outs, flags=b.FLAG_BONUS)
        env["ctx"].verify_round(d)
        env["ctx"].recover_sample(d)
    torch.cuda.synchronize()
    assert env["ctx"].device_error() == 0
    for k, v in lean.items():
        assert np.array_equal(v.cpu().numpy(), full[k].cpu().numpy(), equal_nan=True), k
    gpu = {k: v.cpu().numpy() for k, v in full.items()}
    P.compare(env["oracle"], gpu, P.to_np_inputs(inputs), 0, 0, 1, P.TOL[inputs["h_llm"].dtype])


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("flags", [0, 1])
def test_algorithm1_outputs_only_leave_h_slm_plus_unread_in_verification(env, dtype, flags):
    """RATIO + STEER with none of logp_plus, logp_star, log_z requested: verification reads h_LLM and h_SLM- alone
    (Eq. 7 needs nothing else; to prove it h_SLM+ is poisoned on every row that is not a recovery row) and
    the recovery call forms the normalisers of its one row.  Decisions and tokens must match the oracle."""
    b = env["binding"]
    spec, inputs = _small(env["synth"], 9, 4, 9004 if dtype == "f32" else 12288, dtype, seed=31, ragged=True,
                          beta_choices=(0.5, 1.0, 2.0), temp_choices=(0.7, 1.0))
    inputs["draft_len"][0] = 0
    inputs["u_accept"][1] = 0.0                      # everything accepted: the bonus row (or nothing) is recovered
    inputs["h_llm"][2, 1, 17] = float("nan")         # a non-finite drafted row
    inputs["lam"][3] = 1e30                          # rejected at once, and row 0 is non-finite only through h_SLM+:
    inputs["h_slm_plus"][3, 0, 5] = float("inf")     # verification cannot see it, the recovery of that row does
    ora = P.run_oracle(env["oracle"], P.to_np_inputs(inputs), 0, 0, flags, alg1=True)
    # poison h_SLM+ wherever Algorithm 1 does not need it: all rows but row accept_len of a sampling request
    poisoned = dict(inputs)
    hp = inputs["h_slm_plus"].clone()
    keep = torch.zeros(hp.shape[:2], dtype=torch.bool, device="cuda")
    for r in range(spec.B):
        n, ln = int(ora["accept_len"][r]), int(inputs["draft_len"][r])
        if n < ln or flags:
            keep[r, n] = True
    hp[~keep] = float("nan")
    poisoned["h_slm_plus"] = hp
    gpu, launches = _two_phase_round(env, poisoned, flags)
    assert launches == 4      # stream + epilogue; recovery rows' stream + sampling (which forms their normalisers)
    # every request, poisoned inputs on both sides: the oracle round that reads what Algorithm 1 reads
    stats = P.compare(env["oracle"], gpu, P.to_np_inputs(poisoned), 0, 0, flags, P.TOL[inputs["h_llm"].dtype], alg1=True,
                      keys=ALG1_KEYS)
    assert stats["requests"] == spec.B and stats["excused_accept"] + stats["excused_token"] <= 1
    assert gpu["req_status"][3] == b.REQ_NONFINITE and gpu["rec_token"][3] == -1 and gpu["accept_len"][3] == 0
    assert gpu["req_status"][2] == b.REQ_NONFINITE


def test_draft_length_extremes_and_no_bonus(env):
    """len 0 (with and without the bonus row: a request that reads nothing), len K, ragged in between."""
    spec, inputs = _small(env["synth"], 9, 4, 3000, "f32", seed=3)
    inputs["draft_len"] = torch.tensor([0, 4, 1, 0, 2, 3, 0, 4, 4], dtype=torch.int32, device="cuda")
    for am, rm, fl in ((0, 0, 0), (0, 0, 1), (1, 1, 0)):
        gpu = P.run_gpu(env["ctx"], inputs, am, rm, fl)
        P.compare(env["oracle"], gpu, P.to_np_inputs(inputs), am, rm, fl, 1e-4)
        if fl == 0:
            assert (gpu["n_out"][[0, 3, 6]] == 0).all() and (gpu["rec_token"][[0, 3, 6]] == -1).all()


def test_all_accepted_and_rejected_at_row_zero(env):
    spec, inputs = _small(env["synth"], 6, 5, 5000, "bf16", seed=4)
    inputs["h_slm_minus"] = inputs["h_llm"].clone()                 # ratio >= 1 everywhere (lambda 0.5)
    gpu = P.run_gpu(env["ctx"], inputs, 0, 0, 1)
    assert (gpu["accept_len"] == 5).all() and (gpu["alpha"] == 1).all() and (gpu["n_out"] == 6).all()
    P.compare(env["oracle"], gpu, P.to_np_inputs(inputs), 0, 0, 1, 2e-3)
    inputs["lam"] = torch.full((6,), 1e30, device="cuda")           # ratio ~ 0: rejected at row 0
    inputs["u_accept"] = torch.full((6, 5), 0.5, device="cuda")
    gpu = P.run_gpu(env["ctx"], inputs, 0, 0, 0)
    assert (gpu["accept_len"] == 0).all() and (gpu["n_out"] == 1).all()
    P.compare(env["oracle"], gpu, P.to_np_inputs(inputs), 0, 0, 0, 2e-3)


def test_degenerate_logits_and_status_words(env):
    b = env["binding"]
    spec, inputs = _small(env["synth"], 8, 2, 2600, "f32", seed=5)
    L, Pp, M = inputs["h_llm"], inputs["h_slm_plus"], inputs["h_slm_minus"]
    L[0, :, 100:2300] = float("-inf"); Pp[0, :, 100:2300] = float("-inf"); M[0, :, 100:2300] = float("-inf")  # masked vocabulary -> NaN in r
    L[1, :, ::2] = float("-inf")                                    # half of the generalist's vocabulary masked
    L[2, 1, 7] = float("nan")                                       # NaN in a reached row
    L[3, 0, :] *= 40.0; Pp[3, 0, :] *= 40.0; M[3, 0, :] *= 40.0     # huge dynamic range
    inputs["draft_tokens"][4, 0] = 2600                             # token out of range
    inputs["draft_len"][5] = 7                                      # length out of range
    inputs["temperature"][6] = 0.0                                  # bad temperature ...
    inputs["draft_len"][6] = -3                                     # ... and a bad length: both bits are reported
    L[7, 2, 5] = float("inf")                                       # +inf in the bonus row
    inputs["u_accept"][:] = 0.0
    inputs["u_accept"][2, 0] = 0.0
    for am, rm, fl in ((0, 0, 1), (1, 1, 1)):
        gpu = P.run_gpu(env["ctx"], inputs, am, rm, fl)
        stats = P.compare(env["oracle"], gpu, P.to_np_inputs(inputs), am, rm, fl, 1e-4)
        assert gpu["req_status"][0] == b.REQ_NONFINITE
        assert gpu["req_status"][4] & b.REQ_BAD_TOKEN and gpu["accept_len"][4] == 0
        assert gpu["req_status"][5] == b.REQ_BAD_LEN
        assert gpu["req_status"][6] == (b.REQ_BAD_PARAM | b.REQ_BAD_LEN) and gpu["n_out"][6] == 0
        assert gpu["req_status"][2] & b.REQ_NONFINITE or gpu["accept_len"][2] == 0


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_outliers_after_the_first_batch_of_a_chunk(env, dtype):
    """Full chunks are reduced relative to the maxima of their first 256 entries; an entry hundreds of binades
    above those must overflow that attempt and send the chunk through the variant that tests every batch.
    Spikes sit past the first batch of a chunk, in each stream, at low temperature too.  Their size keeps the
    spread of a row below ~1000 binades: log2(e)/T is a float32 in the kernels, so a log-probability carries an
    error of about 2^-25 times the distance (in binades) of the token from the row maximum."""
    spec, inputs = _small(env["synth"], 6, 3, 5000, dtype, seed=17, temp_choices=(0.25, 1.0), beta_choices=(1.0, 2.5))
    L, Pp, M = inputs["h_llm"], inputs["h_slm_plus"], inputs["h_slm_minus"]
    L[0, 0, 300] = 160.0                    # one stream only
    Pp[1, 1, 1900] = 150.0
    M[2, 0, 2900] = 170.0
    L[3, :, 777] += 140.0; Pp[3, :, 777] += 140.0; M[3, :, 777] += 140.0   # a shared spike: r stays moderate
    L[4, 2, 4999] = 165.0                   # in the ragged last chunk
    Pp[5, 0, 600] = 150.0; M[5, 0, 601] = 155.0; L[5, 0, 1100] = 145.0
    for am, rm in ((0, 0), (1, 1)):
        gpu = P.run_gpu(env["ctx"], inputs, am, rm, 1)
        P.compare(env["oracle"], gpu, P.to_np_inputs(inputs), am, rm, 1, P.TOL[L.dtype])


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_extreme_temperatures(env, dtype):
    """Very low temperatures stretch a row over thousands of binades (nearly every chunk overflows its first
    attempt and is redone with per-batch tests); very high ones flatten it.  Logits of ordinary size."""
    spec, inputs = _small(env["synth"], 6, 3, 7000, dtype, seed=23, beta_choices=(0.5, 1.0, 2.0))
    inputs["temperature"] = torch.tensor([0.02, 0.05, 0.1, 5.0, 50.0, 1.0], dtype=torch.float32, device="cuda")
    tol = P.TOL[inputs["h_llm"].dtype]
    for am, rm in ((0, 0), (1, 1)):
        gpu = P.run_gpu(env["ctx"], inputs, am, rm, 1)
        P.compare(env["oracle"], gpu, P.to_np_inputs(inputs), am, rm, 1, tol)


@pytest.mark.parametrize("K", [20, 70])
def test_long_drafts(env, K):
    """More draft positions than the usual handful; beyond 64 rows a request's epilogue runs in several passes."""
    b = env["binding"]
    spec = env["synth"].RoundSpec("long_drafts", 3, K, 900, "f32", ragged=True)
    inputs = env["synth"].make_round(spec, device="cuda", seed=K)
    inputs["draft_len"] = torch.tensor([K, K // 2, 1], dtype=torch.int32, device="cuda")
    inputs["lam"][:] = 0.05                                  # accept almost everything so that late rows matter
    ctx = b.Context(max_B=3, max_K=K, max_V=900)
    for am, rm, fl in ((0, 0, 1), (1, 1, 0)):
        gpu = P.run_gpu(ctx, inputs, am, rm, fl)
        P.compare(env["oracle"], gpu, P.to_np_inputs(inputs), am, rm, fl, 1e-4)
    ctx.close()


def test_many_requests_cross_the_slab_limit(env):
    spec, inputs = _small(env["synth"], 5000, 2, 64, "bf16", seed=6, ragged=True)
    gpu = P.run_gpu(env["ctx"], inputs, 0, 0, 1)
    rng = np.random.default_rng(0)
    sel = np.sort(np.concatenate([[0, 1023, 1024, 2047, 2048, 4095, 4096, 4999], rng.choice(5000, 60, replace=False)]))
    sel = np.unique(sel)
    npin = P.to_np_inputs(inputs, torch.as_tensor(sel, device="cuda"))
    P.compare(env["oracle"], gpu, npin, 0, 0, 1, 2e-3, sel=sel)
    # the two-phase round over the same slabs: same decisions and tokens
    b = env["binding"]
    lean = {k: v for k, v in b.alloc_outputs(5000, 2, "cuda").items() if k not in ("logp_plus", "logp_star", "log_z")}
    d = b.make_desc(inputs, lean, flags=b.FLAG_BONUS | b.FLAG_TWO_PHASE)
    env["ctx"].verify_round(d)
    env["ctx"].recover_sample(d)
    torch.cuda.synchronize()
    assert env["ctx"].device_error() == 0
    for k in ("accept_len", "accept_flags", "rec_token", "out_tokens", "n_out", "req_status"):
        assert np.array_equal(lean[k].cpu().numpy(), gpu[k]), k


def test_zero_requests_and_zero_drafts(env):
    b = env["binding"]
    spec, inputs = _small(env["synth"], 3, 0, 500, "f32", seed=7)
    gpu = P.run_gpu(env["ctx"], inputs, 0, 0, 1)                     # K = 0: only the bonus row
    P.compare(env["oracle"], gpu, P.to_np_inputs(inputs), 0, 0, 1, 1e-4)
    empty = {k: v[:0] for k, v in inputs.items()}
    out = b.verify_recover_round(env["ctx"], empty, flags=1)
    assert out["accept_len"].numel() == 0


# ------------------------------------------------------------------ the law, on the GPU
def test_output_law_monte_carlo_on_gpu(env):
    """4096 identical V=8 requests x 64 rounds with fresh drafts and uniforms against the closed-form law."""
    import scipy.special as sps
    V, K, Bn, rounds, lam, beta = 8, 2, 4096, 64, 0.7, 1.2
    g = torch.Generator(device="cpu"); g.manual_seed(21)
    rows = [(1.5 * torch.randn(K + 1, V, generator=g)) for _ in range(3)]
    L, Pp, M = rows[0], rows[0] + rows[1], rows[0] + 0.7 * rows[2]
    l, p, m = (x.double().numpy() for x in (L, Pp, M))
    pl, pp, pm = sps.softmax(l, -1), sps.softmax(p, -1), sps.softmax(m, -1)
    pstar = sps.softmax(l + beta * (p - m), -1)
    alpha = np.minimum(1.0, pl / (lam * pm))
    a = (pp * alpha).sum(-1)
    reach = np.concatenate([[1.0], np.cumprod(a[:K])])
    want_n = np.array([reach[t] * (1 - a[t]) for t in range(K)] + [reach[K]])
    inputs = {
        "h_llm": L.expand(Bn, K + 1, V).contiguous().cuda(), "h_slm_plus": Pp.expand(Bn, K + 1, V).contiguous().cuda(),
        "h_slm_minus": M.expand(Bn, K + 1, V).contiguous().cuda(),
        "draft_len": torch.full((Bn,), K, dtype=torch.int32, device="cuda"),
        "lam": torch.full((Bn,), lam, device="cuda"), "beta": torch.full((Bn,), beta, device="cuda"),
        "temperature": torch.ones(Bn, device="cuda"),
    }
    cnt_n = np.zeros(K + 1); cnt_tok = np.zeros((K + 1, V))
    gg = torch.Generator(device="cuda"); gg.manual_seed(22)
    ppt = torch.from_numpy(pp).cuda()
    for _ in range(rounds):
        inputs["draft_tokens"] = torch.stack(
            [torch.multinomial(ppt[t], Bn, replacement=True, generator=gg) for t in range(K)], 1).to(torch.int32)
        inputs["u_accept"] = torch.rand(Bn, K, device="cuda", generator=gg)
        inputs["u_recover"] = torch.rand(Bn, device="cuda", generator=gg)
        gpu = P.run_gpu(env["ctx"], inputs, 0, 0, 1)
        cnt_n += np.bincount(gpu["accept_len"], minlength=K + 1)
        for t in range(K + 1):
            cnt_tok[t] += np.bincount(gpu["rec_token"][gpu["accept_len"] == t], minlength=V)
    N = Bn * rounds
    np.testing.assert_allclose(cnt_n / N, want_n, atol=5.0 / np.sqrt(N))
    for t in range(K + 1):
        np.testing.assert_allclose(cnt_tok[t] / N, want_n[t] * pstar[t], atol=5.0 / np.sqrt(N))


# ------------------------------------------------------------------ boundary behaviour
def test_guard_regions_and_determinism(env):
    """Outputs live inside sentinel-filled buffers: nothing outside the declared extents may change,
    and a second run must reproduce every byte."""
    b = env["binding"]
    spec, inputs = _small(env["synth"], 7, 3, 4100, "bf16", seed=8, ragged=True)
    B, K = 7, 3
    PAD = 64
    bufs, outs = {}, {}
    for name, (dt, shp) in b._OUT_SPECS.items():
        n = B * int(np.prod(shp(K))) if shp(K) else B
        raw = torch.full((n + 2 * PAD,), 0x5A, dtype=torch.uint8, device="cuda").repeat_interleave(
            torch.empty((), dtype=dt).element_size())
        bufs[name] = raw
        es = torch.empty((), dtype=dt).element_size()
        outs[name] = raw[PAD * es:(PAD + n) * es].view(dt).view((B,) + shp(K))
    runs = []
    for _ in range(2):
        b.verify_recover_round(env["ctx"], inputs, accept_mode=1, recover_mode=1, flags=1, outputs=outs)
        torch.cuda.synchronize()
        runs.append({k: v.clone() for k, v in bufs.items()})
    for name, raw in bufs.items():
        es = torch.empty((), dtype=b._OUT_SPECS[name][0]).element_size()
        assert (raw[:PAD * es] == 0x5A).all() and (raw[-PAD * es:] == 0x5A).all(), name
        assert torch.equal(runs[0][name], runs[1][name]), name


def test_error_codes_on_device(env):
    b = env["binding"]
    spec, inputs = _small(env["synth"], 2, 2, 300, "f32", seed=9)
    outs = b.alloc_outputs(2, 2, "cuda")
    desc = b.make_desc(inputs, outs, flags=1)
    small_ctx = b.Context(max_B=1, max_K=2, max_V=300)
    with pytest.raises(b.SpecSteerError) as e:
        small_ctx.verify_round(desc)
    assert e.value.code == b.ERR_UNSUPPORTED
    fresh = b.Context(max_B=4, max_K=2, max_V=300)
    with pytest.raises(b.SpecSteerError) as e:
        fresh.recover_sample(desc)
    assert e.value.code == b.ERR_ORDER
    desc.ld_row = 299
    with pytest.raises(b.SpecSteerError) as e:
        fresh.verify_round(desc)
    assert e.value.code == b.ERR_INVALID_ARG
    desc.ld_row = 300
    desc.accept_len = None
    with pytest.raises(b.SpecSteerError) as e:
        fresh.verify_round(desc)
    assert e.value.code == b.ERR_INVALID_ARG
    assert fresh.launch_count == 0 and fresh.workspace_bytes > 0
    # the timing hook wants both events or none
    ev = torch.cuda.Event(enable_timing=True)
    ev.record()
    with pytest.raises(b.SpecSteerError) as e:
        fresh.time_streaming(ev, None)
    assert e.value.code == b.ERR_INVALID_ARG
    small_ctx.close(); fresh.close()


def test_streaming_kernel_timing_hook(env):
    """The event pair the library records around the streaming kernel gives a positive time below the whole call's,
    and switching the hook off leaves the events untouched."""
    spec, inputs = _small(env["synth"], 8, 3, 50000, "f32", seed=12)
    b = env["binding"]
    outs = b.alloc_outputs(8, 3, "cuda")
    desc = b.make_desc(inputs, outs, flags=1)
    e0, e1, a, z = (torch.cuda.Event(enable_timing=True) for _ in range(4))
    for ev in (e0, e1):
        ev.record()
    torch.cuda.synchronize()
    env["ctx"].time_streaming(e0, e1)
    a.record()
    env["ctx"].verify_round(desc)
    env["ctx"].recover_sample(desc)
    z.record()
    env["ctx"].time_streaming(None, None)
    torch.cuda.synchronize()
    inner, outer = e0.elapsed_time(e1), a.elapsed_time(z)
    assert 0 < inner < outer
    env["ctx"].verify_round(desc)          # hook off: e0/e1 keep their times
    torch.cuda.synchronize()
    assert e0.elapsed_time(e1) == inner


def test_host_round_matches_device_round(env):
    """The host-buffer entry point (copies inside the call) gives the same bytes as the device path."""
    b = env["binding"]
    spec, inputs = _small(env["synth"], 37, 3, 9000, "bf16", seed=10, ragged=True)
    dev = P.run_gpu(env["ctx"], inputs, 0, 0, 1)
    host_in = {k: v.cpu().pin_memory() for k, v in inputs.items()}
    host_out = b.alloc_outputs(37, 3, "cpu", pin=True)
    desc = b.make_desc(host_in, host_out, flags=1)
    env["ctx"].round_host(desc)
    for k, v in host_out.items():
        assert np.array_equal(dev[k], v.numpy(), equal_nan=True), k


@pytest.mark.parametrize("recover_mode", [0, 2], ids=["sampled", "greedy"])
@pytest.mark.parametrize("dtype,flags", [("f32", 1), ("bf16", 0), ("bf16", 1)])
def test_host_round_with_algorithm1_outputs_copies_only_what_it_reads(env, dtype, flags, recover_mode):
    """Only Algorithm 1's outputs requested from host buffers: rows [0, K) of h_LLM and h_SLM- go over first,
    then row accept_len of h_SLM+ (and of the other two when it is the bonus row).  Everything else on the host is
    poisoned with NaN to prove it is never used; results equal the device-resident two-phase round."""
    b = env["binding"]
    V = 9004 if dtype == "f32" else 12288
    spec, inputs = _small(env["synth"], 21, 4, V, dtype, seed=70 + flags, ragged=True,
                          beta_choices=(0.5, 1.0, 2.0), temp_choices=(0.7, 1.0))
    inputs["draft_len"][0] = 0
    inputs["u_accept"][1] = 0.0                  # everything accepted: the bonus row (or nothing) is recovered
    inputs["temperature"][2] = 0.0               # BAD_PARAM
    inputs["h_llm"][3, 0, 11] = float("nan")     # non-finite already in verification
    inputs["lam"][4] = 1e30
    inputs["h_slm_plus"][4, 0, 5] = float("inf")  # non-finite only on the recovery row
    skip = ("logp_plus", "logp_star", "log_z")
    outs = {k: v for k, v in b.alloc_outputs(spec.B, spec.K, "cuda").items() if k not in skip}
    d = b.make_desc(inputs, outs, recover_mode=recover_mode, flags=flags | b.FLAG_TWO_PHASE)
    env["ctx"].verify_round(d)
    env["ctx"].recover_sample(d)
    torch.cuda.synchronize()
    dev = {k: v.cpu().numpy() for k, v in outs.items()}
    # host copies with everything the round does not need turned into NaN
    n, dl = dev["accept_len"], inputs["draft_len"].cpu().numpy()
    host_in = {k: v.cpu().clone() for k, v in inputs.items()}
    rows = torch.arange(spec.K + 1)[None, :]
    drafted = (rows < spec.K).expand(spec.B, -1)      # rows [0, K) of the two tensors travel whatever draft_len is
    rec_row = (rows == torch.as_tensor(n)[:, None]) & torch.as_tensor(
        ((n < dl) | bool(flags)) & ((dev["req_status"] & 16) == 0))[:, None]
    nan = float("nan")
    host_in["h_llm"][~(drafted | rec_row)] = nan
    host_in["h_slm_minus"][~(drafted | rec_row)] = nan
    host_in["h_slm_plus"][~rec_row] = nan
    host_in["h_llm"][3, 0, 11] = nan             # (kept: part of the case)
    host_in = {k: v.pin_memory() for k, v in host_in.items()}
    host_out = {k: v for k, v in b.alloc_outputs(spec.B, spec.K, "cpu", pin=True).items() if k not in skip}
    env["ctx"].round_host(b.make_desc(host_in, host_out, recover_mode=recover_mode, flags=flags))
    assert env["ctx"].device_error() == 0
    for k, v in host_out.items():
        assert np.array_equal(dev[k], v.numpy(), equal_nan=True), k
    assert dev["req_status"][2] == 16 and dev["req_status"][3] & 4 and dev["req_status"][4] & 4


@pytest.mark.parametrize("B,K,V", [(3, 0, 4100), (1100, 1, 520)])
def test_host_round_with_algorithm1_outputs_edge_shapes(env, B, K, V):
    """No drafts at all (only bonus rows travel), and more requests than one slab holds."""
    b = env["binding"]
    spec, inputs = _small(env["synth"], B, K, V, "f32", seed=90 + K)
    skip = ("logp_plus", "logp_star", "log_z")
    for recover_mode in (0, 2):
        outs = {k: v for k, v in b.alloc_outputs(B, K, "cuda").items() if k not in skip}
        d = b.make_desc(inputs, outs, recover_mode=recover_mode, flags=1 | b.FLAG_TWO_PHASE)
        env["ctx"].verify_round(d)
        env["ctx"].recover_sample(d)
        torch.cuda.synchronize()
        host_in = {k: v.cpu().pin_memory() for k, v in inputs.items()}
        host_out = {k: v for k, v in b.alloc_outputs(B, K, "cpu", pin=True).items() if k not in skip}
        env["ctx"].round_host(b.make_desc(host_in, host_out, recover_mode=recover_mode, flags=1))
        assert env["ctx"].device_error() == 0
        for k, v in host_out.items():
            assert np.array_equal(outs[k].cpu().numpy(), v.numpy(), equal_nan=True), (k, recover_mode)
        assert (host_out["rec_token"].numpy() >= 0).all()


# ------------------------------------------------------------------ the one-launch round of small batches
@pytest.mark.parametrize("cfg", [0, 1])
@pytest.mark.parametrize("mode", MODES, ids=[m[0] for m in MODES])
def test_one_launch_round_equals_separate_launches_on_configs(env, cfg, mode):
    """The one-launch round (streaming, epilogue and STEER sample in the streaming kernel: the default for a single
    request, FLAG_ONE_LAUNCH for more) against the same round in three launches.  Same device code per request: every
    output byte equal."""
    b, synth = env["binding"], env["synth"]
    inputs = synth.make_round(synth.CONFIGS[cfg], device="cuda", seed=0)
    _, am, rm, fl = mode
    got = []
    # the library's own choice: one launch for a single request, otherwise the streaming kernel and one launch for
    # epilogue + STEER sample
    default = 1 if synth.CONFIGS[cfg].B == 1 else 2
    for extra, want in ((b.FLAG_ONE_LAUNCH, 1 if rm == 0 else 3), (b.FLAG_SEPARATE_LAUNCHES, 3 if rm == 0 else 4),
                        (0, default if rm == 0 else 3)):
        before = env["ctx"].launch_count
        out = P.run_gpu(env["ctx"], inputs, am, rm, fl | extra)
        if rm == 0:
            assert env["ctx"].launch_count - before == want
        got.append(out)
    for k in got[0]:
        assert np.array_equal(got[0][k], got[1][k], equal_nan=True), k
        assert np.array_equal(got[2][k], got[1][k], equal_nan=True), k


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_one_launch_round_edge_cases(env, dtype):
    """Requests that stream nothing (no drafts and no bonus row; bad parameters), bad tokens, non-finite rows, ragged
    drafts, a ragged last chunk, more requests than CTAs: one launch against three, and against the oracle."""
    b, synth = env["binding"], env["synth"]
    spec, inputs = _small(synth, 200, 3, 2600, dtype, seed=77, ragged=True, beta_choices=(0.5, 1.0, 2.0),
                          temp_choices=(0.7, 1.0))
    inputs["draft_len"][0] = 0
    inputs["draft_len"][7] = 0
    inputs["temperature"][3] = 0.0
    inputs["draft_tokens"][4, 0] = 2600
    inputs["h_llm"][5, 1, 9] = float("nan")
    inputs["draft_len"][6] = 9
    for fl in (0, 1):
        for am in (0, 1):
            one = P.run_gpu(env["ctx"], inputs, am, 0, fl | b.FLAG_ONE_LAUNCH)
            three = P.run_gpu(env["ctx"], inputs, am, 0, fl | b.FLAG_SEPARATE_LAUNCHES)
            two = P.run_gpu(env["ctx"], inputs, am, 0, fl)   # streaming kernel, then epilogue + sample in one launch
            for k in one:
                assert np.array_equal(one[k], three[k], equal_nan=True), (k, fl, am)
                assert np.array_equal(two[k], three[k], equal_nan=True), (k, fl, am)
            P.compare(env["oracle"], one, P.to_np_inputs(inputs), am, 0, fl, P.TOL[inputs["h_llm"].dtype])
    # repeated launches leave the per-request counters at zero: the next round is right again
    again = P.run_gpu(env["ctx"], inputs, 0, 0, 1 | b.FLAG_ONE_LAUNCH)
    ref = P.run_gpu(env["ctx"], inputs, 0, 0, 1 | b.FLAG_SEPARATE_LAUNCHES)
    for k in again:
        assert np.array_equal(again[k], ref[k], equal_nan=True), k


# ------------------------------------------------------------------ the paper's comparison decoders, as inputs to this path
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_standard_speculative_decoding_as_an_input_special_case(env, dtype):
    """Standard speculative decoding (the "Standard SD" row of the paper's efficiency table) is this path with the
    drafter in both Specialist slots, beta = 0, the exact acceptance of Eq. 6 (target P_LLM, proposal P_SLM+) and the
    residual fallback: alpha = min(1, P_LLM/Q) and the resample from max(0, P_LLM - Q).  The two Specialist pointers
    name the same tensor."""
    synth = env["synth"]
    spec, inputs = _small(synth, 24, 4, 9000, dtype, seed=5, ragged=True, temp_choices=(0.7, 1.0))
    inputs["h_slm_minus"] = inputs["h_slm_plus"]       # the same device memory behind both pointers
    inputs["beta"].fill_(0.0)
    inputs["lam"].fill_(1.0)
    gpu = P.run_gpu(env["ctx"], inputs, 1, 1, 0)
    npin = P.to_np_inputs(inputs)
    P.compare(env["oracle"], gpu, npin, 1, 1, 0, P.TOL[inputs["h_llm"].dtype])
    # with beta = 0 the fused target is P_LLM itself: log P* = log P_LLM and log Z = 0 on every verified row
    n = gpu["accept_len"]
    for b in range(spec.B):
        rows = min(int(n[b]) + 1, int(npin["draft_len"][b]))
        if gpu["req_status"][b] == 0 and rows > 0:
            np.testing.assert_allclose(gpu["logp_star"][b, :rows], gpu["logp_llm"][b, :rows], atol=P.TOL[inputs["h_llm"].dtype])
            np.testing.assert_allclose(gpu["log_z"][b, :rows], 0.0, atol=P.TOL[inputs["h_llm"].dtype])


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_always_on_steering_as_an_input_special_case(env, dtype):
    """Steering at every step without drafts (the always-on logit steering the paper compares with): no drafted
    tokens, FLAG_BONUS, so every request samples one token from Softmax(h_LLM + beta (h_SLM+ - h_SLM-)) (Eq. 8) on
    row 0."""
    synth = env["synth"]
    spec, inputs = _small(synth, 40, 3, 12001, dtype, seed=6, beta_choices=(0.5, 1.0, 2.0), temp_choices=(0.7, 1.0))
    inputs["draft_len"].zero_()
    gpu = P.run_gpu(env["ctx"], inputs, 0, 0, 1)
    P.compare(env["oracle"], gpu, P.to_np_inputs(inputs), 0, 0, 1, P.TOL[inputs["h_llm"].dtype])
    assert (gpu["accept_len"] == 0).all() and (gpu["n_out"] == 1).all() and (gpu["rec_token"] >= 0).all()
