"""GPU parity of greedy recovery (SPECSTEER_RECOVER_ARGMAX: the token of largest h_rec, Eq. 8; the paper decodes
greedily) with the oracle.  The oracle orders h_rec in double; the GPU forms it in float32 with one fused
multiply-add.  compare() demands the oracle's token wherever the gap to the runner-up exceeds the float32 rounding
of the three terms, a token inside that near-tie set otherwise, and in every case the token the documented float32
tie-break picks.  An accept decision may differ where the oracle's margin is below 1e-5 (it is then forced in the
oracle).
"""
import numpy as np
import pytest
import torch

import _parity as P

pytestmark = pytest.mark.gpu
ARGMAX = 2


@pytest.fixture(scope="module")
def env(oracle_mod):
    from paper_2603_16219_b200 import binding, build, synth
    assert torch.cuda.is_available()
    build.build()
    ctx = binding.Context(max_B=2048, max_K=8, max_V=262144, device=0)
    yield {"ctx": ctx, "binding": binding, "synth": synth, "oracle": oracle_mod}
    ctx.close()


def _check(env, inputs, flags=1, accept_mode=0, V=None, sel=None, near_ties=0):
    gpu = P.run_gpu(env["ctx"], inputs, accept_mode, ARGMAX, flags, V=V)
    npin = P.to_np_inputs(inputs, None if sel is None else torch.as_tensor(sel, device="cuda"))
    if V is not None:
        npin = {k: (np.ascontiguousarray(v[..., :V]) if k.startswith("h_") else v) for k, v in npin.items()}
    stats = P.compare(env["oracle"], gpu, npin, accept_mode, ARGMAX, flags, P.TOL[inputs["h_llm"].dtype], V=V, sel=sel)
    print("greedy", stats)
    assert stats["excused_token"] <= near_ties     # tokens that differ from the double-precision order (near-ties)
    return gpu


@pytest.mark.parametrize("cfg", [0, 1, 2])
def test_benchmark_configurations(env, cfg):
    synth = env["synth"]
    inputs = synth.make_round(synth.CONFIGS[cfg], device="cuda", seed=0)
    gpu = _check(env, inputs)
    assert (gpu["rec_token"] >= 0).all()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V", [1, 7, 8, 9, 4095, 4097, 40000])
def test_vocabulary_sizes_and_splits(env, V, dtype):
    """One request: up to 16 CTAs share the row (V = 40000 gives 9 parts); three requests: fewer parts each."""
    synth = env["synth"]
    for B in (1, 3):
        spec = synth.RoundSpec("g", B, 2, V, dtype, beta_choices=(0.5, 1.0, 2.0), temp_choices=(0.7, 1.3))
        _check(env, synth.make_round(spec, device="cuda", seed=V + B))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_rows_that_are_not_16_byte_aligned(env, dtype):
    synth = env["synth"]
    V, ld = 9001, 9003
    spec = synth.RoundSpec("g", 5, 3, ld, dtype)
    inputs = synth.make_round(spec, device="cuda", seed=3)
    _check(env, inputs, V=V)


def test_ties_go_to_the_lowest_id_across_parts(env):
    """Constant rows: every entry is a maximiser, the answer is token 0 although 16 CTAs each report their own first."""
    synth = env["synth"]
    spec = synth.RoundSpec("g", 2, 1, 70000, "f32")
    inputs = synth.make_round(spec, device="cuda", seed=0)
    for k in ("h_llm", "h_slm_plus", "h_slm_minus"):
        inputs[k].fill_(0.25)
    inputs["h_llm"][1, :, 65000:] = 0.5          # second request: the maximisers start at 65000
    gpu = _check(env, inputs)
    n = gpu["accept_len"]
    assert gpu["rec_token"][0] == 0 and gpu["rec_token"][1] == 65000
    assert gpu["n_out"][0] == n[0] + 1


def test_ragged_no_bonus_exact_rule_and_bad_requests(env):
    synth = env["synth"]
    spec = synth.RoundSpec("g", 24, 6, 5000, "bf16", ragged=True, beta_uniform=(0.0, 3.0), temp_choices=(0.3, 1.0, 1.5))
    inputs = synth.make_round(spec, device="cuda", seed=5)
    inputs["temperature"][2] = -1.0               # BAD_PARAM: nothing accepted, nothing emitted
    inputs["draft_len"][3] = 0                     # no drafts and no bonus row: nothing to emit
    gpu = _check(env, inputs, flags=0, accept_mode=1)
    assert gpu["rec_token"][2] == -1 and gpu["rec_token"][3] == -1
    dl = inputs["draft_len"].cpu().numpy()
    ok = np.ones(24, bool); ok[2] = False
    assert ((gpu["rec_token"] >= 0) == (gpu["accept_len"] < dl))[ok].all()


@pytest.mark.parametrize("cfg", [3, 4])
def test_full_size_every_request(env, cfg):
    """The two largest configurations, every request: one-pass greedy round with every output, then the two-phase
    greedy round against the oracle round that reads only what Algorithm 1 reads."""
    synth, b = env["synth"], env["binding"]
    spec = synth.CONFIGS[cfg]
    inputs = synth.make_round(spec, device="cuda", seed=0)
    gpu = _check(env, inputs, near_ties=spec.B // 64)
    P.invariants(gpu, inputs, 1, P.TOL[inputs["h_llm"].dtype])
    keys = ("accept_len", "accept_flags", "alpha", "logp_llm", "logp_minus", "rec_token", "rec_logprob", "out_tokens",
            "n_out", "req_status")
    outs = {k: v for k, v in b.alloc_outputs(spec.B, spec.K, "cuda").items() if k in keys}
    d = b.make_desc(inputs, outs, recover_mode=ARGMAX, flags=1)
    before = env["ctx"].launch_count
    env["ctx"].verify_round(d)
    env["ctx"].recover_sample(d)
    torch.cuda.synchronize()
    assert env["ctx"].device_error() == 0 and env["ctx"].launch_count - before == 4   # row references, stream, epilogue, argmax
    two = {k: v.cpu().numpy() for k, v in outs.items()}
    stats = P.compare(env["oracle"], two, P.to_np_inputs(inputs), 0, ARGMAX, 1, P.TOL[inputs["h_llm"].dtype], alg1=True,
                      keys=keys)
    print(spec.name, "two-phase greedy", stats)
    assert stats["requests"] == spec.B and stats["excused_token"] <= spec.B // 64
    for k in ("accept_len", "rec_token", "n_out", "out_tokens", "req_status", "accept_flags"):
        assert np.array_equal(two[k], gpu[k]), k


def test_host_round_in_greedy_mode(env):
    b, synth = env["binding"], env["synth"]
    spec = synth.RoundSpec("g", 6, 3, 3000, "f32")
    inputs = synth.make_round(spec, device="cuda", seed=9)
    dev = P.run_gpu(env["ctx"], inputs, 0, ARGMAX, 1)
    host_in = {k: v.cpu().pin_memory() for k, v in inputs.items()}
    host_out = b.alloc_outputs(spec.B, spec.K, "cpu", pin=True)
    env["ctx"].round_host(b.make_desc(host_in, host_out, recover_mode=ARGMAX, flags=1))
    for k, v in host_out.items():
        assert np.array_equal(v.numpy(), dev[k], equal_nan=True), k


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("flags", [0, 1])
def test_two_phase_greedy_round(env, dtype, flags):
    """Only Algorithm 1's outputs, greedy: verification reads h_LLM and h_SLM- over the drafted rows (h_SLM+ is
    poisoned everywhere else to prove it), and the argmax pass over row accept_len forms that row's normaliser and
    finiteness check itself.  Three launches."""
    b = env["binding"]
    synth = env["synth"]
    spec = synth.RoundSpec("g", 10, 4, 9004 if dtype == "f32" else 12288, dtype, ragged=True,
                           beta_choices=(0.5, 1.0, 2.0), temp_choices=(0.7, 1.0))
    inputs = synth.make_round(spec, device="cuda", seed=41)
    inputs["draft_len"][0] = 0
    inputs["u_accept"][1] = 0.0                      # everything accepted
    inputs["lam"][3] = 1e30                          # rejected at once; row 0 is non-finite only through h_SLM+
    inputs["h_slm_plus"][3, 0, 5] = float("inf")
    inputs["lam"][4] = 1e30
    inputs["h_slm_plus"][4, 0, :] = float("-inf")    # h_SLM+ is -inf throughout the recovery row: only that pass can tell
    ora = P.run_oracle(env["oracle"], P.to_np_inputs(inputs), 0, ARGMAX, flags, alg1=True)
    hp = inputs["h_slm_plus"].clone()
    keep = torch.zeros(hp.shape[:2], dtype=torch.bool, device="cuda")
    for r in range(spec.B):
        n, ln = int(ora["accept_len"][r]), int(inputs["draft_len"][r])
        if n < ln or flags:
            keep[r, n] = True
    hp[~keep] = float("nan")
    poisoned = dict(inputs)
    poisoned["h_slm_plus"] = hp
    keys = ("accept_len", "accept_flags", "alpha", "logp_llm", "logp_minus", "rec_token", "rec_logprob", "out_tokens",
            "n_out", "req_status")
    outs = {k: v for k, v in b.alloc_outputs(spec.B, spec.K, "cuda").items() if k in keys}
    d = b.make_desc(poisoned, outs, recover_mode=ARGMAX, flags=flags | b.FLAG_TWO_PHASE)
    before = env["ctx"].launch_count
    env["ctx"].verify_round(d)
    env["ctx"].recover_sample(d)
    torch.cuda.synchronize()
    assert env["ctx"].device_error() == 0
    assert env["ctx"].launch_count - before == 3
    gpu = {k: v.cpu().numpy() for k, v in outs.items()}
    # every request, the poisoned tensors on both sides: the oracle round that reads what Algorithm 1 reads
    stats = P.compare(env["oracle"], gpu, P.to_np_inputs(poisoned), 0, ARGMAX, flags, P.TOL[inputs["h_llm"].dtype],
                      alg1=True, keys=keys)
    assert stats["requests"] == spec.B and stats["excused_token"] == 0
    assert gpu["req_status"][3] == b.REQ_NONFINITE and gpu["rec_token"][3] == -1 and gpu["accept_len"][3] == 0
    assert gpu["req_status"][4] == b.REQ_NONFINITE and gpu["rec_token"][4] == -1 and gpu["accept_len"][4] == 0


def test_two_phase_greedy_full_size_equals_one_pass(env):
    """Config 3 at full size: the two-phase greedy round (taken automatically for a batch this large) gives the same
    accepted lengths and tokens as the one-pass greedy round that was asked for every output."""
    b, synth = env["binding"], env["synth"]
    spec = synth.CONFIGS[3]
    inputs = synth.make_round(spec, device="cuda", seed=0)
    full = P.run_gpu(env["ctx"], inputs, 0, ARGMAX, 1)
    outs = {k: v for k, v in b.alloc_outputs(spec.B, spec.K, "cuda").items() if k not in ("logp_plus", "logp_star", "log_z")}
    d = b.make_desc(inputs, outs, recover_mode=ARGMAX, flags=1)
    before = env["ctx"].launch_count
    env["ctx"].verify_round(d)
    env["ctx"].recover_sample(d)
    torch.cuda.synchronize()
    assert env["ctx"].device_error() == 0 and env["ctx"].launch_count - before == 4
    for k in ("accept_len", "rec_token", "n_out", "out_tokens", "req_status", "accept_flags"):
        assert np.array_equal(outs[k].cpu().numpy(), full[k]), k
    assert np.abs(outs["rec_logprob"].cpu().numpy() - full["rec_logprob"]).max() <= 1e-5


def test_two_phase_greedy_is_deterministic(env):
    """The row's parts are merged in index order by whichever CTA finishes last: repeated rounds give the same bits."""
    b, synth = env["binding"], env["synth"]
    spec = synth.RoundSpec("g", 5, 3, 70000, "bf16", beta_choices=(0.5, 1.0, 2.0), temp_choices=(0.7, 1.3))
    inputs = synth.make_round(spec, device="cuda", seed=77)
    outs = {k: v for k, v in b.alloc_outputs(spec.B, spec.K, "cuda").items() if k not in ("logp_plus", "logp_star", "log_z")}
    d = b.make_desc(inputs, outs, recover_mode=ARGMAX, flags=1 | b.FLAG_TWO_PHASE)
    seen = None
    for _ in range(12):
        env["ctx"].verify_round(d)
        env["ctx"].recover_sample(d)
        torch.cuda.synchronize()
        got = (outs["rec_token"].cpu().numpy().copy(), outs["rec_logprob"].cpu().numpy().copy())
        if seen is None:
            seen = got
        assert np.array_equal(seen[0], got[0]) and np.array_equal(seen[1], got[1])
