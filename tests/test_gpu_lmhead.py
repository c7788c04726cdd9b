"""GPU parity of the round with the LM heads fused in front (specsteer_lmhead_round) with its oracle.

The oracle forms the logits h = x W^T in float64 from the same bf16 hidden states and head weights and runs the
round on them.  The tensor cores accumulate the d products of a logit in float32, so a logit is off by up to a few
1e-5 at d of a few thousand; log-probabilities are therefore compared within 5e-4, and a decision (accept / reject,
sampled token) may differ where the oracle's margin is below 2e-4 - it is then forced in the oracle and the rest
of the request is compared on that branch.
"""
import dataclasses

import numpy as np
import pytest
import torch

import _parity as P

pytestmark = pytest.mark.gpu

TOL = 5e-4
MARGIN = 2e-4


TWO_PHASE_KEYS = ("accept_len", "accept_flags", "alpha", "logp_llm", "logp_minus", "rec_token", "rec_logprob", "out_tokens",
                  "n_out", "req_status")


@pytest.fixture(scope="module")
def env(oracle_mod):
    from paper_2603_16219_b200 import binding, build, synth
    assert torch.cuda.is_available()
    build.build()
    ctx = binding.Context(max_B=128, max_K=8, max_V=48000, device=0)
    yield {"binding": binding, "synth": synth, "oracle": oracle_mod, "ctx": ctx}
    ctx.close()


def _bits(t):
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def _np_inputs(o, inputs, sel=None):
    """Oracle-side inputs: float64 logits from the oracle's own LM-head step, plus the per-request arrays."""
    pick = (lambda t: t) if sel is None else (lambda t: t[sel])
    out = {
        "h_llm": o.lmhead_logits(_bits(pick(inputs["x_llm"])), _bits(inputs["w_llm"])),
        "h_slm_plus": o.lmhead_logits(_bits(pick(inputs["x_slm_plus"])), _bits(inputs["w_slm_plus"])),
        "h_slm_minus": o.lmhead_logits(_bits(pick(inputs["x_slm_minus"])), _bits(inputs["w_slm_minus"])),
    }
    for k in ("draft_tokens", "draft_len", "lam", "beta", "temperature", "u_accept", "u_recover"):
        out[k] = pick(inputs[k]).detach().cpu().numpy()
    return out


def _run_gpu(env, inputs, accept_mode=0, flags=1, drop=()):
    b = env["binding"]
    B, K1 = inputs["x_llm"].shape[:2]
    outs = b.alloc_outputs(B, K1 - 1, "cuda")
    for name in drop:
        outs.pop(name)
    desc = b.make_lmhead_desc(inputs, outs, accept_mode=accept_mode, flags=flags)
    env["ctx"].lmhead_round(desc)
    torch.cuda.synchronize()
    assert env["ctx"].device_error() == 0
    return {k: v.cpu().numpy() for k, v in outs.items()}


def _case(env, spec, d_llm, d_slm, seed=0, accept_mode=0, flags=1, mutate=None):
    inputs = env["synth"].make_lmhead_round(spec, d_llm, d_slm, device="cuda", seed=seed)
    if mutate:
        mutate(inputs)
    gpu = _run_gpu(env, inputs, accept_mode, flags)
    npin = _np_inputs(env["oracle"], inputs)
    stats = P.compare(env["oracle"], gpu, npin, accept_mode, 0, flags, TOL, margin=MARGIN)
    return inputs, gpu, stats


def _spec(env, cfg, **kw):
    return dataclasses.replace(env["synth"].CONFIGS[cfg], **kw)


def test_small_round_one_row_block_ragged_vocabulary(env):
    """20 rows (one block of 128, mostly padding), V = 23 tiles + 57 entries, 5 and 2 stages of hidden entries."""
    _, gpu, stats = _case(env, _spec(env, 0, B=5, K=3, V=3001), 320, 128)
    assert stats["max_logp_err"] < TOL
    assert (gpu["rec_token"] >= 0).all()


def test_several_row_blocks_and_hidden_widths_that_are_not_stage_multiples(env):
    """280 rows = 2 blocks + 24; d_llm = 200 and d_slm = 72 end inside a stage of 64 (zero fill)."""
    _case(env, _spec(env, 0, B=70, K=3, V=1000), 200, 72, seed=1)


def test_more_tiles_than_sms_alternating_accumulators(env):
    """375 vocabulary tiles of one row block on 148 CTAs: every CTA runs 2-3 tiles, so the h_LLM accumulator
    alternates and the epilogue of one tile overlaps the products of the next."""
    _, gpu, _ = _case(env, _spec(env, 1, B=20, K=5, V=48000), 256, 64, seed=2)
    assert len(set(gpu["rec_token"].tolist())) > 5


def test_exact_acceptance_rule(env):
    _case(env, _spec(env, 1, B=12, K=5, V=5000), 192, 64, seed=3, accept_mode=1)


def test_ragged_drafts_mixed_beta_and_temperature_no_bonus(env):
    spec = _spec(env, 4, B=40, K=6, V=7000, ragged=True)
    _, gpu, _ = _case(env, spec, 256, 128, seed=4, flags=0)
    inputs_len = env["synth"].make_lmhead_round(spec, 256, 128, device="cpu", seed=4)["draft_len"].numpy()
    assert ((gpu["rec_token"] >= 0) == (gpu["accept_len"] < inputs_len)).all()


def test_two_different_specialist_heads(env):
    def mutate(inputs):
        g = torch.Generator(device="cuda")
        g.manual_seed(99)
        w = inputs["w_slm_plus"].float()
        inputs["w_slm_minus"] = (w + 0.05 * torch.randn(w.shape, generator=g, device="cuda")).to(torch.bfloat16)
    _case(env, _spec(env, 0, B=9, K=4, V=2500), 128, 64, seed=5, mutate=mutate)


def test_zero_drafts_and_bad_tokens(env):
    def mutate(inputs):
        inputs["draft_len"][0] = 0
        inputs["draft_tokens"][1, 1] = -3
        inputs["draft_tokens"][2, 0] = 2500         # == V: outside the vocabulary
    _, gpu, _ = _case(env, _spec(env, 0, B=6, K=3, V=2500), 128, 64, seed=6, mutate=mutate)
    assert gpu["accept_len"][0] == 0 and gpu["rec_token"][0] >= 0
    assert gpu["req_status"][1] & 1 and gpu["req_status"][2] & 1


def test_outputs_can_be_left_out(env):
    inputs = env["synth"].make_lmhead_round(_spec(env, 0, B=7, K=3, V=1800), 128, 64, device="cuda", seed=7)
    full = _run_gpu(env, inputs)
    lean = _run_gpu(env, inputs, drop=("logp_plus", "log_z", "alpha", "accept_flags", "req_status"))     # still one pass
    for k in lean:
        assert np.array_equal(full[k], lean[k], equal_nan=True), k
    # without logp_star as well the round is two-phase (other tiles, other summation order): same decisions and tokens,
    # floating-point outputs to rounding
    lean = _run_gpu(env, inputs, drop=("logp_plus", "logp_star", "log_z", "alpha", "accept_flags", "req_status"))
    for k in lean:
        if lean[k].dtype.kind in "iu":
            assert np.array_equal(full[k], lean[k]), k
        else:
            assert np.array_equal(np.isnan(full[k]), np.isnan(lean[k])), k
            assert np.nanmax(np.abs(full[k] - lean[k]), initial=0.0) < 1e-4, k


def test_repeated_calls_are_bit_identical(env):
    inputs = env["synth"].make_lmhead_round(_spec(env, 0, B=33, K=4, V=9000), 320, 128, device="cuda", seed=8)
    a = _run_gpu(env, inputs)
    b = _run_gpu(env, inputs)
    for k in a:
        assert np.array_equal(a[k], b[k], equal_nan=True), k


def test_argument_checks(env):
    b = env["binding"]
    inputs = env["synth"].make_lmhead_round(_spec(env, 0, B=2, K=2, V=600), 128, 64, device="cuda", seed=9)
    outs = b.alloc_outputs(2, 2, "cuda")
    d = b.make_lmhead_desc(inputs, outs)
    d.round.recover_mode = b.RECOVER_RESIDUAL
    with pytest.raises(b.SpecSteerError) as e:
        env["ctx"].lmhead_round(d)
    assert e.value.code == b.ERR_UNSUPPORTED
    d = b.make_lmhead_desc(inputs, outs)
    d.d_slm = 60
    with pytest.raises(b.SpecSteerError) as e:
        env["ctx"].lmhead_round(d)
    assert e.value.code == b.ERR_UNSUPPORTED
    d = b.make_lmhead_desc(inputs, outs)
    d.w_llm = None
    with pytest.raises(b.SpecSteerError) as e:
        env["ctx"].lmhead_round(d)
    assert e.value.code == b.ERR_INVALID_ARG
    d = b.make_lmhead_desc(inputs, outs)
    d.round.V = 48001
    with pytest.raises(b.SpecSteerError) as e:
        env["ctx"].lmhead_round(d)
    assert e.value.code == b.ERR_UNSUPPORTED
    torch.cuda.synchronize()
    assert env["ctx"].device_error() == 0


def test_agrees_with_the_streaming_round_on_materialised_logits(env):
    """The same round through the two GPU paths: logits materialised by a float32 product and streamed, against
    the fused path.  Decisions agree except where the fused path's own oracle margin is small (checked above), so
    here only gross agreement is asserted: most requests identical, log-probabilities within the tolerance."""
    b = env["binding"]
    inputs = env["synth"].make_lmhead_round(_spec(env, 0, B=48, K=4, V=6000), 256, 128, device="cuda", seed=10)
    fused = _run_gpu(env, inputs)
    mk = lambda x, w: torch.matmul(x.float(), w.float().t()).contiguous()
    li = {k: inputs[k] for k in ("draft_tokens", "draft_len", "lam", "beta", "temperature", "u_accept", "u_recover")}
    li["h_llm"] = mk(inputs["x_llm"], inputs["w_llm"])
    li["h_slm_plus"] = mk(inputs["x_slm_plus"], inputs["w_slm_plus"])
    li["h_slm_minus"] = mk(inputs["x_slm_minus"], inputs["w_slm_minus"])
    ctx2 = b.Context(48, 4, 6000, device=0)
    try:
        streamed = P.run_gpu(ctx2, li, 0, 0, 1)
    finally:
        ctx2.close()
    same = (fused["accept_len"] == streamed["accept_len"]) & (fused["rec_token"] == streamed["rec_token"])
    assert same.mean() > 0.9
    ok = same[:, None] & np.isfinite(streamed["logp_llm"])
    assert np.abs(fused["logp_llm"][ok] - streamed["logp_llm"][ok]).max() < TOL


def test_full_size_sampled_requests():
    """The benchmark shape (256 requests, K = 4, V = 151936, hidden widths 5120 and 2048) in the launch the bench
    times; 32 requests spread over the batch are checked against the oracle, whose logits are formed 16384
    vocabulary entries at a time (each logit is still one float64 dot product)."""
    import oracle as o
    from paper_2603_16219_b200 import binding as b, build, synth
    o.build()
    build.build()
    spec = synth.CONFIGS[3]
    inputs = synth.make_lmhead_round(spec, 5120, 2048, device="cuda", seed=0)
    ctx = b.Context(spec.B, spec.K, spec.V, device=0)
    try:
        outs = b.alloc_outputs(spec.B, spec.K, "cuda")
        desc = b.make_lmhead_desc(inputs, outs, flags=1)
        ctx.lmhead_round(desc)
        torch.cuda.synchronize()
        assert ctx.device_error() == 0
        gpu = {k: v.cpu().numpy() for k, v in outs.items()}
        # the same batch with only Algorithm 1's outputs requested: the two-phase round, as `bench.py --lmhead --lean` times it
        outs2 = {k: v for k, v in b.alloc_outputs(spec.B, spec.K, "cuda").items() if k in TWO_PHASE_KEYS}
        before = ctx.launch_count
        ctx.lmhead_round(b.make_lmhead_desc(inputs, outs2, flags=1))
        torch.cuda.synchronize()
        assert ctx.device_error() == 0 and ctx.launch_count - before == 7
        gpu2 = {k: v.cpu().numpy() for k, v in outs2.items()}
    finally:
        ctx.close()
    P.invariants(gpu, {"draft_tokens": inputs["draft_tokens"], "draft_len": inputs["draft_len"]}, 1, TOL)
    sel = np.unique(np.linspace(0, spec.B - 1, 32).astype(int))
    selt = torch.as_tensor(sel, device="cuda")

    def logits(xn, wn):
        x = _bits(inputs[xn][selt])
        w = _bits(inputs[wn])
        return np.concatenate([o.lmhead_logits(x, w[v0:v0 + 16384]) for v0 in range(0, spec.V, 16384)], axis=2)

    npin = {"h_llm": logits("x_llm", "w_llm"), "h_slm_plus": logits("x_slm_plus", "w_slm_plus"),
            "h_slm_minus": logits("x_slm_minus", "w_slm_minus")}
    for k in ("draft_tokens", "draft_len", "lam", "beta", "temperature", "u_accept", "u_recover"):
        npin[k] = inputs[k][selt].cpu().numpy()
    stats = P.compare(o, gpu, npin, 0, 0, 1, TOL, sel=sel, margin=MARGIN)
    print("lmhead full size", stats)
    assert stats["requests"] == 32
    stats2 = P.compare(o, gpu2, npin, 0, 0, 1, TOL, sel=sel, margin=MARGIN, alg1=True, keys=TWO_PHASE_KEYS)
    print("lmhead full size, two-phase", stats2)
    assert stats2["requests"] == 32
    # over the whole batch the two rounds agree wherever neither decision is near a margin (a handful may differ)
    same = (gpu["accept_len"] == gpu2["accept_len"]) & (gpu["rec_token"] == gpu2["rec_token"])
    assert same.mean() > 0.97, same.mean()


def test_no_drafts_at_all_and_empty_batch(env):
    """K = 0: every request has its bonus row only (Eq. 8 with nothing to verify); B = 0: nothing is launched."""
    b = env["binding"]
    _, gpu, _ = _case(env, _spec(env, 0, B=9, K=0, V=1500), 128, 64, seed=11)
    assert (gpu["accept_len"] == 0).all() and (gpu["n_out"] == 1).all()
    inputs = env["synth"].make_lmhead_round(_spec(env, 0, B=3, K=2, V=700), 128, 64, device="cuda", seed=12)
    empty = {k: (v[:0].contiguous() if k.startswith("x_") or not k.startswith("w_") else v) for k, v in inputs.items()}
    outs = b.alloc_outputs(0, 2, "cuda")
    before = env["ctx"].launch_count
    env["ctx"].lmhead_round(b.make_lmhead_desc(empty, outs))
    assert env["ctx"].launch_count == before


def test_bad_parameters_are_reported_per_request(env):
    def mutate(inputs):
        inputs["temperature"][1] = 0.0
        inputs["lam"][3] = -1.0
        inputs["beta"][4] = float("nan")
    inputs = env["synth"].make_lmhead_round(_spec(env, 0, B=6, K=3, V=2000), 128, 64, device="cuda", seed=13)
    mutate(inputs)
    gpu = _run_gpu(env, inputs)
    for r in (1, 3, 4):
        assert gpu["req_status"][r] & 16 and gpu["accept_len"][r] == 0 and gpu["rec_token"][r] == -1
    ok = [0, 2, 5]
    npin = _np_inputs(env["oracle"], inputs, sel=torch.as_tensor(ok, device="cuda"))
    P.compare(env["oracle"], gpu, npin, 0, 0, 1, TOL, sel=ok, margin=MARGIN)


def test_one_context_serves_both_paths_and_changing_shapes(env):
    """The fused path has its own workspace: a streaming round in between must not disturb it, and shapes may change
    from call to call."""
    b = env["binding"]
    lm = env["synth"].make_lmhead_round(_spec(env, 0, B=10, K=3, V=3000), 192, 64, device="cuda", seed=14)
    first = _run_gpu(env, lm)
    st = env["synth"].make_round(_spec(env, 0, B=4, K=2, V=5000), device="cuda", seed=1)
    P.run_gpu(env["ctx"], st, 0, 0, 1)
    _case(env, _spec(env, 1, B=3, K=5, V=9000), 128, 128, seed=15)
    again = _run_gpu(env, lm)
    for k in first:
        assert np.array_equal(first[k], again[k], equal_nan=True), k


@pytest.mark.parametrize("V,d_llm,d_slm", [(100, 8, 8), (128, 64, 16), (129, 72, 8), (5, 16, 8)])
def test_tiny_vocabularies_and_hidden_widths(env, V, d_llm, d_slm):
    """A vocabulary below one tile, exactly one tile, one entry more; hidden widths below one stage of 64."""
    _case(env, _spec(env, 0, B=4, K=2, V=V), d_llm, d_slm, seed=20 + V)


def test_many_rows_few_vocabulary_tiles(env):
    """1024 rows = 8 row blocks over 3 vocabulary tiles: fewer tiles than SMs, every CTA at most one tile."""
    _case(env, _spec(env, 2, B=128, K=7, V=300, ragged=True), 128, 64, seed=30)


# ------------------------------------------------------------------ greedy recovery on the fused path
def _greedy_case(env, spec, d_llm, d_slm, seed, flags=1, accept_mode=0, mutate=None):
    inputs = env["synth"].make_lmhead_round(spec, d_llm, d_slm, device="cuda", seed=seed)
    if mutate:
        mutate(inputs)
    b = env["binding"]
    B, K1 = inputs["x_llm"].shape[:2]
    outs = b.alloc_outputs(B, K1 - 1, "cuda")
    before = env["ctx"].launch_count
    env["ctx"].lmhead_round(b.make_lmhead_desc(inputs, outs, accept_mode=accept_mode, recover_mode=b.RECOVER_ARGMAX, flags=flags))
    torch.cuda.synchronize()
    assert env["ctx"].device_error() == 0 and env["ctx"].launch_count - before == 3
    gpu = {k: v.cpu().numpy() for k, v in outs.items()}
    stats = P.compare(env["oracle"], gpu, _np_inputs(env["oracle"], inputs), accept_mode, 2, flags, TOL, margin=MARGIN)
    return inputs, gpu, stats


@pytest.mark.parametrize("V,d_llm,d_slm", [(3001, 320, 128), (48000, 256, 64), (100, 64, 32)])
def test_greedy_recovery_on_the_fused_path(env, V, d_llm, d_slm):
    """The token of largest h_rec, taken from the per-tile maxima the tensor-core pass leaves.  The order is that of
    float32 accumulators, so a token other than the oracle's is admissible only where the two largest values are
    within the margin (compare() checks that the token is then itself within the margin of the largest)."""
    _, gpu, stats = _greedy_case(env, _spec(env, 1, B=12, K=4, V=V), d_llm, d_slm, seed=50 + V % 7)
    assert (gpu["rec_token"] >= 0).all() and stats["excused_token"] <= 1


def test_greedy_recovery_fused_ragged_no_bonus_exact_rule(env):
    spec = _spec(env, 4, B=30, K=6, V=7000, ragged=True)

    def mutate(inputs):
        inputs["temperature"][2] = -1.0
        inputs["draft_len"][3] = 0
    inputs, gpu, _ = _greedy_case(env, spec, 256, 128, seed=57, flags=0, accept_mode=1, mutate=mutate)
    assert gpu["rec_token"][2] == -1 and gpu["rec_token"][3] == -1
    dl = inputs["draft_len"].cpu().numpy()
    ok = np.ones(30, bool); ok[2] = False
    assert ((gpu["rec_token"] >= 0) == (gpu["accept_len"] < dl))[ok].all()


def test_greedy_and_sampled_fused_rounds_share_the_verification(env):
    b = env["binding"]
    inputs = env["synth"].make_lmhead_round(_spec(env, 0, B=16, K=3, V=9000), 192, 64, device="cuda", seed=58)
    sampled = _run_gpu(env, inputs)
    outs = b.alloc_outputs(16, 3, "cuda")
    env["ctx"].lmhead_round(b.make_lmhead_desc(inputs, outs, recover_mode=b.RECOVER_ARGMAX, flags=1))
    torch.cuda.synchronize()
    for k in ("accept_len", "accept_flags", "alpha", "logp_llm", "logp_minus", "logp_plus", "logp_star", "log_z", "req_status"):
        assert np.array_equal(outs[k].cpu().numpy(), sampled[k], equal_nan=True), k


# ------------------------------------------------------------------ the two-phase round on this path
def _two_phase_case(env, spec, d_llm, d_slm, seed, flags=1, recover_mode=0, mutate=None, launches=7):
    """Only Algorithm 1's outputs requested: verification forms h_LLM and h_SLM- alone (tiles of 128 x 256), the
    recovery rows are compacted and get all three products.  Every request against the oracle round that reads only
    what Algorithm 1 reads, on float64 logits."""
    b = env["binding"]
    inputs = env["synth"].make_lmhead_round(spec, d_llm, d_slm, device="cuda", seed=seed)
    if mutate:
        mutate(inputs)
    outs = {k: v for k, v in b.alloc_outputs(spec.B, spec.K, "cuda").items() if k in TWO_PHASE_KEYS}
    desc = b.make_lmhead_desc(inputs, outs, recover_mode=recover_mode, flags=flags)
    before = env["ctx"].launch_count
    env["ctx"].lmhead_round(desc)
    torch.cuda.synchronize()
    assert env["ctx"].device_error() == 0 and env["ctx"].launch_count - before == launches
    gpu = {k: v.cpu().numpy() for k, v in outs.items()}
    stats = P.compare(env["oracle"], gpu, _np_inputs(env["oracle"], inputs), 0, recover_mode, flags, TOL, margin=MARGIN,
                      alg1=True, keys=TWO_PHASE_KEYS)
    return inputs, gpu, stats


@pytest.mark.parametrize("recover_mode", [0, 2], ids=["sampled", "greedy"])
def test_two_phase_round_small_ragged_vocabulary(env, recover_mode):
    _, gpu, stats = _two_phase_case(env, _spec(env, 0, B=5, K=3, V=3001), 320, 128, seed=0, recover_mode=recover_mode)
    assert (gpu["rec_token"] >= 0).all() and stats["max_logp_err"] < TOL


def test_two_phase_round_several_row_blocks_odd_hidden_widths_no_bonus(env):
    """280 rows = 2 blocks + 24 in verification, 70 compact rows in recovery; widths that end inside a stage of 64."""
    spec = _spec(env, 4, B=70, K=3, V=1000, ragged=True)
    inputs, gpu, _ = _two_phase_case(env, spec, 200, 72, seed=1, flags=0)
    dl = inputs["draft_len"].cpu().numpy()
    assert ((gpu["rec_token"] >= 0) == (gpu["accept_len"] < dl)).all()


def test_two_phase_round_more_tiles_than_sms(env):
    """188 vocabulary tiles of 256 on 148 CTAs: the accumulators are reused, each epilogue runs under the other product."""
    _, gpu, _ = _two_phase_case(env, _spec(env, 1, B=20, K=5, V=48000), 256, 64, seed=2)
    assert len(set(gpu["rec_token"].tolist())) > 5


def test_two_phase_round_degenerate_requests(env):
    def mutate(inputs):
        inputs["draft_len"][0] = 0                   # nothing drafted: only the bonus row
        inputs["draft_tokens"][1, 1] = -3            # bad tokens
        inputs["draft_tokens"][2, 0] = 2500
        inputs["temperature"][3] = 0.0               # bad parameter: nothing accepted, no token
        inputs["u_accept"][4] = 0.0                  # everything accepted: the bonus row is the recovery row
        inputs["lam"][5] = 1e30                      # rejected at once
    _, gpu, _ = _two_phase_case(env, _spec(env, 0, B=8, K=3, V=2500), 128, 64, seed=6, mutate=mutate)
    assert gpu["accept_len"][0] == 0 and gpu["rec_token"][0] >= 0
    assert gpu["req_status"][1] & 1 and gpu["req_status"][2] & 1
    assert gpu["req_status"][3] == 16 and gpu["rec_token"][3] == -1 and gpu["n_out"][3] == 0
    assert gpu["accept_len"][4] == 3 and gpu["n_out"][4] == 4
    assert gpu["accept_len"][5] == 0 and gpu["n_out"][5] == 1


def test_two_phase_round_twice_gives_the_same_bits(env):
    spec = _spec(env, 0, B=33, K=4, V=9000)
    _, a, _ = _two_phase_case(env, spec, 320, 128, seed=8)
    _, c, _ = _two_phase_case(env, spec, 320, 128, seed=8)
    for k in a:
        assert np.array_equal(a[k], c[k], equal_nan=True), k
