"""GPU parity of greedy recovery (SPECSTEER_RECOVER_ARGMAX: the token of largest h_rec, Eq. 8; the paper decodes
greedily) with the oracle.  Both sides form h_rec in float32 with one fused multiply-add, so the token must be
identical on every request whose accepted length agrees (an accept decision may still differ where the oracle's
margin is below 1e-5; compare() then forces it in the oracle); no margin applies to the token itself.
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


def _check(env, inputs, flags=1, accept_mode=0, V=None, sel=None):
    gpu = P.run_gpu(env["ctx"], inputs, accept_mode, ARGMAX, flags, V=V)
    npin = P.to_np_inputs(inputs, None if sel is None else torch.as_tensor(sel, device="cuda"))
    if V is not None:
        npin = {k: (np.ascontiguousarray(v[..., :V]) if k.startswith("h_") else v) for k, v in npin.items()}
    stats = P.compare(env["oracle"], gpu, npin, accept_mode, ARGMAX, flags, P.TOL[inputs["h_llm"].dtype], V=V, sel=sel)
    assert stats["excused_token"] == 0
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


def test_full_size_float32_sampled(env):
    synth = env["synth"]
    spec = synth.CONFIGS[3]
    inputs = synth.make_round(spec, device="cuda", seed=0)
    sel = np.unique(np.linspace(0, spec.B - 1, 10).astype(int))
    gpu = _check(env, inputs, sel=sel)
    P.invariants(gpu, inputs, 1, P.TOL[torch.float32])
    # every request, against a float32 restatement on the device, as a property that holds at any size
    n = torch.as_tensor(gpu["accept_len"], device="cuda").long()
    rows = torch.arange(spec.B, device="cuda")
    l, p, m = (inputs[k][rows, n] for k in ("h_llm", "h_slm_plus", "h_slm_minus"))
    r = torch.addcmul(l, inputs["beta"][:, None], p - m)
    got = r[rows, torch.as_tensor(gpu["rec_token"], device="cuda").long()]
    assert ((r.max(dim=1).values - got) <= 1e-5).all()      # torch may round the product and the sum separately


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
