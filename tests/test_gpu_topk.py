"""GPU parity of the top-k split recovery (specsteer_cloud_topk + specsteer_edge_resample) with its oracle.

The truncation is integer work on float32 values both sides form with one fused multiply-add, so the kept token
ids and values must match bit for bit; the sampled token must match unless the oracle's CDF margin is below 1e-5.
"""
import numpy as np
import pytest
import torch

import _parity as P

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env(oracle_mod):
    from paper_2603_16219_b200 import binding, build, synth
    assert torch.cuda.is_available()
    build.build()
    ctx = binding.Context(max_B=512, max_K=8, max_V=262144, device=0)
    yield {"binding": binding, "synth": synth, "oracle": oracle_mod, "ctx": ctx}
    ctx.close()


def _run(env, inputs, k, flags, V=None, cloud_only_verification=False):
    b, o = env["binding"], env["oracle"]
    hl = inputs["h_llm"]
    B, K = hl.shape[0], hl.shape[1] - 1
    outs = b.alloc_outputs(B, K, "cuda")
    if cloud_only_verification:      # verification that never reads h_SLM+, as on the paper's cloud
        for name in ("logp_plus", "logp_star", "log_z"):
            outs.pop(name)
    desc = b.make_desc(inputs, outs, flags=flags | (b.FLAG_TWO_PHASE if cloud_only_verification else 0), V=V)
    idx = torch.full((B, k), -7, dtype=torch.int32, device="cuda")
    val = torch.full((B, k), 123.0, dtype=torch.float32, device="cuda")
    env["ctx"].verify_round(desc)
    env["ctx"].cloud_topk(desc, idx, val)
    env["ctx"].edge_resample(desc, idx, val)
    torch.cuda.synchronize()
    assert env["ctx"].device_error() == 0
    gpu = {k_: v.cpu().numpy() for k_, v in outs.items()}
    gpu["topk_idx"], gpu["topk_val"] = idx.cpu().numpy(), val.cpu().numpy()
    npin = P.to_np_inputs(inputs)
    if V is not None:
        npin = {k_: (v[..., :V] if k_.startswith("h_") else v) for k_, v in npin.items()}
        npin = {k_: (np.ascontiguousarray(v) if k_.startswith("h_") else v) for k_, v in npin.items()}
    ora = P.run_oracle(o, npin, 0, 0, flags & 1)
    safe = (ora["accept_margin"] > P.MARGIN).all(axis=1)
    assert np.array_equal(gpu["accept_len"][safe], ora["accept_len"][safe])
    top = o.topk_recover_round(npin["h_llm"], npin["h_slm_plus"], npin["h_slm_minus"], npin["draft_len"], npin["beta"],
                               npin["temperature"], npin["u_recover"], ora["accept_len"], ora["req_status"], k, flags)
    n_checked = 0
    for r in range(B):
        if gpu["accept_len"][r] != ora["accept_len"][r]:
            continue                                   # a sub-margin acceptance decision: another row was recovered
        n_checked += 1
        assert np.array_equal(gpu["topk_idx"][r], top["topk_idx"][r]), r
        assert np.array_equal(gpu["topk_val"][r], top["topk_val"][r]), r
        n = int(ora["accept_len"][r])
        if top["cdf_margin"][r] > P.MARGIN:
            assert gpu["rec_token"][r] == top["rec_token"][r], r
        else:
            assert gpu["rec_token"][r] in top["topk_idx"][r]
        if gpu["rec_token"][r] == top["rec_token"][r] and top["rec_token"][r] >= 0:
            assert abs(gpu["rec_logprob"][r] - top["rec_logprob"][r]) <= 1e-5 * max(1.0, abs(top["rec_logprob"][r]))
        want_n = n + (1 if gpu["rec_token"][r] >= 0 else 0)
        assert gpu["n_out"][r] == want_n
        assert np.array_equal(gpu["out_tokens"][r][:n], npin["draft_tokens"][r][:n])
        if gpu["rec_token"][r] >= 0:
            assert gpu["out_tokens"][r][n] == gpu["rec_token"][r]
        assert (gpu["out_tokens"][r][want_n:] == -1).all()
    assert n_checked >= B - max(1, B // 64)
    return gpu, top


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V,k", [(5, 32), (31, 32), (100, 5), (2047, 32), (4099, 1), (20011, 32)])
def test_topk_small_vocabularies_and_tails(env, V, k, dtype):
    spec = env["synth"].RoundSpec("topk_small", 6, 3, V, dtype, ragged=True, beta_choices=(0.5, 1.0, 2.0),
                                  temp_choices=(0.7, 1.0))
    inputs = env["synth"].make_round(spec, device="cuda", seed=V + k)
    for flags in (0, 1):
        _run(env, inputs, k, flags)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_topk_ties_nan_and_infinities(env, dtype):
    spec = env["synth"].RoundSpec("topk_ties", 5, 2, 3000, dtype)
    inputs = env["synth"].make_round(spec, device="cuda", seed=9)
    for name in ("h_llm", "h_slm_minus"):                    # coarse values: many equal h_cloud entries
        inputs[name] = (inputs[name].float() * 2).round().div(2).to(inputs[name].dtype)
    inputs["h_llm"][1, :, 100:2900] = float("-inf")          # fewer finite entries than k on some rows
    inputs["h_llm"][2, :, ::3] = float("nan")                # NaN entries are never kept (and make the row non-finite)
    inputs["h_slm_minus"][3, :, 5] = float("-inf")           # +inf in h_cloud
    inputs["beta"][4] = 0.0                                   # the private term drops out
    inputs["u_accept"][:] = 0.999                             # reject early so that rows get recovered
    _run(env, inputs, 32, 1)
    _run(env, inputs, 7, 0)


def test_topk_unaligned_rows(env):
    b = env["binding"]
    spec = env["synth"].RoundSpec("topk_unaligned", 4, 2, 1001, "bf16")
    base = env["synth"].make_round(spec, device="cuda", seed=3)
    ld = 1003                                                  # rows start on odd element offsets
    inputs = dict(base)
    for name in ("h_llm", "h_slm_plus", "h_slm_minus"):
        buf = torch.zeros((4, 3, ld), dtype=base[name].dtype, device="cuda")
        buf[..., :1001] = base[name]
        inputs[name] = buf
    _run(env, inputs, 32, 1, V=1001)


@pytest.mark.parametrize("cfg", [0, 2, 3, 4])
def test_topk_on_benchmark_shapes(env, cfg):
    """The benchmark configurations at their full batch size, every request."""
    spec = env["synth"].CONFIGS[cfg]
    inputs = env["synth"].make_round(spec, device="cuda", seed=cfg)
    gpu, top = _run(env, inputs, 32, 1)
    assert (gpu["rec_token"] >= 0).all() and gpu["rec_token"].shape[0] == spec.B


def test_topk_after_verification_without_h_slm_plus(env):
    """The deployment the appendix describes: the cloud verifies with h_LLM and h_SLM- alone and truncates, the edge
    adds its private term.  h_SLM+ is read by the edge kernel only."""
    spec = env["synth"].RoundSpec("topk_cloud", 7, 4, 16384, "bf16", ragged=True, beta_choices=(0.5, 1.0, 2.0))
    inputs = env["synth"].make_round(spec, device="cuda", seed=41)
    before = env["ctx"].launch_count
    _run(env, inputs, 32, 1, cloud_only_verification=True)
    assert env["ctx"].launch_count - before == 4      # streaming (two tensors) + epilogue, cloud_topk, edge_resample


def test_topk_argument_checks(env):
    b = env["binding"]
    spec = env["synth"].RoundSpec("topk_args", 2, 2, 64, "f32")
    inputs = env["synth"].make_round(spec, device="cuda", seed=0)
    outs = b.alloc_outputs(2, 2, "cuda")
    desc = b.make_desc(inputs, outs)
    idx = torch.zeros((2, 33), dtype=torch.int32, device="cuda")
    val = torch.zeros((2, 33), dtype=torch.float32, device="cuda")
    env["ctx"].verify_round(desc)
    with pytest.raises(b.SpecSteerError) as e:
        env["ctx"].cloud_topk(desc, idx, val)                # k beyond SPECSTEER_TOPK_MAX
    assert e.value.code == b.ERR_INVALID_ARG
    ctx2 = b.Context(4, 2, 64, device=0)
    with pytest.raises(b.SpecSteerError) as e:
        ctx2.cloud_topk(desc, idx[:, :8].contiguous(), val[:, :8].contiguous())   # no verify_round before it
    assert e.value.code == b.ERR_ORDER
    ctx2.close()
    torch.cuda.synchronize()
