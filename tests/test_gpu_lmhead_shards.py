"""The fused LM-head round with the heads split along the vocabulary, against the oracle of the whole round.

One GPU stands in for G ranks: the shards' kernels are independent launches (none waits for another), so they run
one after the other, each with its own context; the all-gather is a stack of the shards' partials and the MAX
all-reduce an element-wise maximum.  The result must be what the oracle computes on the whole heads.
"""
import dataclasses

import numpy as np
import pytest
import torch

import _parity as P
from test_gpu_lmhead import MARGIN, TOL, _np_inputs

pytestmark = pytest.mark.gpu


def _sharded(binding, sharding, inputs, G, accept_mode, flags, align=8, recover_mode=0):
    B, K1 = inputs["x_llm"].shape[:2]
    K = K1 - 1
    V = inputs["w_llm"].shape[0]
    ctxs, descs, outs, parts, ranges, keep = [], [], [], [], [], []
    for g in range(G):
        lo, hi = sharding.vocab_range(V, g, G, align)
        ranges.append((lo, hi))
        if hi <= lo:
            ctxs.append(None); descs.append(None); outs.append(None); parts.append(None)
            continue
        loc = dict(inputs)
        for name in ("w_llm", "w_slm_plus", "w_slm_minus"):
            loc[name] = inputs[name][lo:hi].contiguous()
        if inputs["w_slm_plus"] is inputs["w_slm_minus"]:
            loc["w_slm_minus"] = loc["w_slm_plus"]           # keep the shared head shared
        ctx = binding.Context(B, K, hi - lo, device=0)
        o = binding.alloc_outputs(B, K, "cuda")
        d = binding.make_lmhead_desc(loc, o, accept_mode=accept_mode, recover_mode=recover_mode, flags=flags)
        keep.append(loc)
        ctxs.append(ctx); descs.append(d); outs.append(o)
        parts.append(torch.empty((B, K1, 64), dtype=torch.uint8, device="cuda"))
    live = [g for g in range(G) if ranges[g][1] > ranges[g][0]]
    for g in live:
        ctxs[g].lmhead_shard_local(descs[g], ranges[g][0], parts[g])
    gathered = torch.stack([parts[g] for g in live], 0).contiguous()
    keys = []
    for r, g in enumerate(live):
        ctxs[g].lmhead_shard_combine(descs[g], gathered, r, ranges[g][0], V)
        if recover_mode == 2:
            keys.append(torch.empty(B, dtype=torch.int64, device="cuda"))
            ctxs[g].lmhead_shard_greedy_local(descs[g], keys[-1])
        else:
            ctxs[g].lmhead_shard_recover(descs[g], gathered, r, ranges[g][0], V)
    if recover_mode == 2:
        best = torch.stack(keys, 0).max(dim=0).values.contiguous()
        for g in live:
            ctxs[g].shard_greedy_finish(descs[g], best)
    torch.cuda.synchronize()
    for g in live:
        assert ctxs[g].device_error() == 0
    res = {k: v.clone() for k, v in outs[live[0]].items()}
    for g in live[1:]:
        for name in ("accept_len", "accept_flags", "alpha", "logp_llm", "logp_minus", "logp_plus", "logp_star",
                     "log_z", "req_status"):
            a, b_ = outs[g][name].cpu().numpy(), res[name].cpu().numpy()
            assert np.array_equal(a, b_, equal_nan=True), (name, g)
        for name in ("rec_token", "rec_logprob", "out_tokens", "n_out"):
            res[name] = torch.maximum(res[name], outs[g][name])
    for c in ctxs:
        if c is not None:
            c.close()
    return {k: v.cpu().numpy() for k, v in res.items()}


@pytest.mark.parametrize("V,G,d_llm,d_slm", [(5000, 2, 192, 64), (20011, 3, 256, 128), (3001, 4, 128, 64), (40000, 8, 320, 64)])
@pytest.mark.parametrize("accept_mode", [0, 1])
def test_sharded_fused_round_matches_the_unsplit_oracle(oracle_mod, V, G, d_llm, d_slm, accept_mode):
    from paper_2603_16219_b200 import binding, build, sharding, synth
    build.build()
    spec = synth.RoundSpec("lm_shards", 6, 3, V, "bf16", ragged=True, beta_choices=(0.5, 1.0, 2.0), temp_choices=(0.7, 1.0))
    inputs = synth.make_lmhead_round(spec, d_llm, d_slm, device="cuda", seed=V + G)
    npin = _np_inputs(oracle_mod, inputs)
    for flags in (1, 0):
        gpu = _sharded(binding, sharding, inputs, G, accept_mode, flags)
        P.compare(oracle_mod, gpu, npin, accept_mode, 0, flags, TOL, margin=MARGIN)


def test_sharded_fused_round_edge_cases(oracle_mod):
    """Tokens on shard borders, a token outside the vocabulary, more shards than vocabulary blocks."""
    from paper_2603_16219_b200 import binding, build, sharding, synth
    build.build()
    spec = synth.RoundSpec("lm_shards_edges", 5, 2, 4096, "bf16")
    inputs = synth.make_lmhead_round(spec, 128, 64, device="cuda", seed=5)
    inputs["draft_tokens"][0, 0] = 1023          # last id of shard 0 (G = 4, 1024 ids each)
    inputs["draft_tokens"][0, 1] = 1024          # first id of shard 1
    inputs["draft_tokens"][1, 0] = 4096          # outside the global vocabulary
    inputs["u_accept"][3] = 0.9999               # early rejection
    npin = _np_inputs(oracle_mod, inputs)
    gpu = _sharded(binding, sharding, inputs, 4, 0, 1)
    P.compare(oracle_mod, gpu, npin, 0, 0, 1, TOL, margin=MARGIN)
    assert gpu["req_status"][1] & 1
    # one shard per 8 ids would leave most shards of a tiny vocabulary empty
    spec = synth.RoundSpec("lm_shards_tiny", 3, 2, 20, "bf16")
    inputs = synth.make_lmhead_round(spec, 64, 32, device="cuda", seed=6)
    gpu = _sharded(binding, sharding, inputs, 8, 0, 1)
    P.compare(oracle_mod, gpu, _np_inputs(oracle_mod, inputs), 0, 0, 1, TOL, margin=MARGIN)


def test_one_shard_equals_the_unsharded_entry_point(oracle_mod):
    from paper_2603_16219_b200 import binding, build, sharding, synth
    build.build()
    spec = synth.RoundSpec("lm_one", 7, 3, 6000, "bf16", beta_choices=(0.5, 1.0), temp_choices=(0.7, 1.0))
    inputs = synth.make_lmhead_round(spec, 192, 64, device="cuda", seed=7)
    one = _sharded(binding, sharding, inputs, 1, 0, 1)
    ctx = binding.Context(spec.B, spec.K, spec.V, device=0)
    outs = binding.alloc_outputs(spec.B, spec.K, "cuda")
    ctx.lmhead_round(binding.make_lmhead_desc(inputs, outs, flags=1))
    torch.cuda.synchronize()
    for k in ("accept_len", "accept_flags", "rec_token", "out_tokens", "n_out", "req_status"):
        assert np.array_equal(outs[k].cpu().numpy(), one[k]), k
    for k in ("logp_llm", "logp_minus", "logp_plus", "logp_star", "log_z", "rec_logprob"):
        assert np.allclose(outs[k].cpu().numpy(), one[k], atol=1e-5, equal_nan=True), k
    ctx.close()



@pytest.mark.parametrize("V,G,d_llm,d_slm", [(5000, 2, 192, 64), (20011, 3, 256, 128), (40000, 8, 320, 64)])
def test_sharded_fused_greedy_round(oracle_mod, V, G, d_llm, d_slm):
    """Greedy recovery with the heads split along the vocabulary: per-tile keys with global ids, each shard's best, the
    maximum over shards, the common last step.  Token as for the unsharded fused round (margin on the runner-up gap)."""
    from paper_2603_16219_b200 import binding, build, sharding, synth
    build.build()
    spec = synth.RoundSpec("lm_shards_greedy", 6, 3, V, "bf16", ragged=True, beta_choices=(0.5, 1.0, 2.0), temp_choices=(0.7, 1.0))
    inputs = synth.make_lmhead_round(spec, d_llm, d_slm, device="cuda", seed=V + G + 1)
    npin = _np_inputs(oracle_mod, inputs)
    for flags in (1, 0):
        gpu = _sharded(binding, sharding, inputs, G, 0, flags, recover_mode=2)
        P.compare(oracle_mod, gpu, npin, 0, 2, flags, TOL, margin=MARGIN)
    # and the sharded result is the unsharded fused greedy round's, token for token
    ctx = binding.Context(spec.B, spec.K, V, device=0)
    outs = binding.alloc_outputs(spec.B, spec.K, "cuda")
    ctx.lmhead_round(binding.make_lmhead_desc(inputs, outs, recover_mode=2, flags=0))
    torch.cuda.synchronize()
    assert np.array_equal(outs["rec_token"].cpu().numpy(), gpu["rec_token"])
    ctx.close()
