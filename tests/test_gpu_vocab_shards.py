"""The vocabulary-sharded round against the oracle of the whole round.

One GPU stands in for G ranks: the shards' kernels are independent launches (none waits for another), so they run
one after the other, each with its own context; the all-gather is a stack of the shards' partials and the MAX
all-reduce an element-wise maximum.  The result must be what the oracle computes on the unsplit vocabulary.
"""
import numpy as np
import pytest
import torch

import _parity as P

pytestmark = pytest.mark.gpu


def _sharded(binding, sharding, inputs, G, accept_mode, flags, align, recover_mode=0):
    hl = inputs["h_llm"]
    B, K1, V = hl.shape
    K = K1 - 1
    ctxs, descs, outs, parts, ranges = [], [], [], [], []
    for g in range(G):
        lo, hi = sharding.vocab_range(V, g, G, align)
        ranges.append((lo, hi))
        loc = dict(inputs)
        for name in ("h_llm", "h_slm_plus", "h_slm_minus"):
            loc[name] = inputs[name][:, :, lo:hi].contiguous() if hi > lo else inputs[name][:, :, :1].contiguous()
        ctx = binding.Context(B, K, max(hi - lo, 1), device=0)
        o = binding.alloc_outputs(B, K, "cuda")
        d = binding.make_desc(loc, o, accept_mode=accept_mode, recover_mode=recover_mode, flags=flags)
        ctxs.append(ctx); descs.append((d, loc)); outs.append(o)
        parts.append(torch.empty((B, K1, 64), dtype=torch.uint8, device="cuda"))
    live = [g for g in range(G) if ranges[g][1] > ranges[g][0]]      # an empty tail shard takes no part
    for g in live:
        ctxs[g].shard_verify_local(descs[g][0], ranges[g][0], parts[g])
    gathered = torch.stack([parts[g] for g in live], 0).contiguous()   # what the all-gather delivers
    keys = []
    for r, g in enumerate(live):
        ctxs[g].shard_verify_combine(descs[g][0], gathered, r, ranges[g][0], V)
        if recover_mode == 2:        # greedy: every shard's best key ...
            keys.append(torch.empty(B, dtype=torch.int64, device="cuda"))
            ctxs[g].shard_greedy_local(descs[g][0], ranges[g][0], keys[-1])
        else:
            ctxs[g].shard_recover_local(descs[g][0], gathered, r, ranges[g][0], V)
    if recover_mode == 2:            # ... the MAX all-reduce, and the same last step everywhere
        best = torch.stack(keys, 0).max(dim=0).values.contiguous()
        for g in live:
            ctxs[g].shard_greedy_finish(descs[g][0], best)
    torch.cuda.synchronize()
    for g in live:
        assert ctxs[g].device_error() == 0
    res = {k: v.clone() for k, v in outs[live[0]].items()}
    for g in live[1:]:
        for name in ("accept_len", "accept_flags", "alpha", "logp_llm", "logp_minus", "logp_plus", "logp_star",
                     "log_z", "req_status"):                          # the combine step is identical on every rank
            a, b_ = outs[g][name].cpu().numpy(), res[name].cpu().numpy()
            assert np.array_equal(a, b_, equal_nan=True), (name, g)
        for name in ("rec_token", "rec_logprob", "out_tokens", "n_out"):   # the MAX all-reduce
            if recover_mode == 2:                                          # greedy: already identical everywhere
                assert np.array_equal(outs[g][name].cpu().numpy(), res[name].cpu().numpy(), equal_nan=True), (name, g)
            res[name] = torch.maximum(res[name], outs[g][name])
    for c in ctxs:
        c.close()
    return {k: v.cpu().numpy() for k, v in res.items()}


@pytest.mark.parametrize("dtype,V,G,align", [("f32", 5000, 2, 4), ("bf16", 20011, 3, 8), ("f32", 3001, 4, 4),
                                             ("bf16", 151936, 8, 8)])
@pytest.mark.parametrize("accept_mode", [0, 1])
def test_sharded_round_matches_the_unsplit_oracle(oracle_mod, dtype, V, G, align, accept_mode):
    from paper_2603_16219_b200 import binding, build, sharding, synth
    build.build()
    B = 6 if V < 100000 else 4
    spec = synth.RoundSpec("vocab_shards", B, 3, V, dtype, ragged=True, beta_choices=(0.5, 1.0, 2.0),
                           temp_choices=(0.7, 1.0))
    inputs = synth.make_round(spec, device="cuda", seed=V + G)
    for flags in (1, 0):
        gpu = _sharded(binding, sharding, inputs, G, accept_mode, flags, align)
        P.compare(oracle_mod, gpu, P.to_np_inputs(inputs), accept_mode, 0, flags, P.TOL[inputs["h_llm"].dtype])


def test_sharded_round_edge_cases(oracle_mod):
    """Tokens on shard borders, a bad token, -inf over a whole shard, more shards than needed."""
    from paper_2603_16219_b200 import binding, build, sharding, synth
    build.build()
    spec = synth.RoundSpec("vocab_shards_edges", 5, 2, 4096, "f32")
    inputs = synth.make_round(spec, device="cuda", seed=5)
    inputs["draft_tokens"][0, 0] = 1023          # last id of shard 0 (G = 4, 1024 ids each)
    inputs["draft_tokens"][0, 1] = 1024          # first id of shard 1
    inputs["draft_tokens"][1, 0] = 4096          # outside the global vocabulary
    inputs["h_llm"][2, :, 1024:2048] = float("-inf")     # shard 1 carries no generalist mass for this request
    inputs["u_accept"][3] = 0.9999               # early rejection
    inputs["u_recover"][4] = 0.9999999           # the CDF target falls in the last shard
    gpu = _sharded(binding, sharding, inputs, 4, 0, 1, 4)
    P.compare(oracle_mod, gpu, P.to_np_inputs(inputs), 0, 0, 1, 1e-4)
    assert gpu["req_status"][1] & binding.REQ_BAD_TOKEN
    # 7 ranks over 4096 ids aligned to 1024: only four non-empty shards take part
    gpu = _sharded(binding, sharding, inputs, 7, 1, 0, 1024)
    P.compare(oracle_mod, gpu, P.to_np_inputs(inputs), 1, 0, 0, 1e-4)



@pytest.mark.parametrize("dtype,V,G,align", [("f32", 5000, 2, 4), ("bf16", 20011, 3, 8), ("bf16", 151936, 8, 8)])
def test_sharded_greedy_round_matches_the_unsplit_oracle(oracle_mod, dtype, V, G, align):
    """Greedy recovery over shards: every shard's best key (value, then the lower global id), their maximum, and the
    same last step on every shard; the token is the unsplit oracle's bit for bit."""
    from paper_2603_16219_b200 import binding, build, sharding, synth
    build.build()
    B = 6 if V < 100000 else 4
    spec = synth.RoundSpec("vocab_shards_greedy", B, 3, V, dtype, ragged=True, beta_choices=(0.5, 1.0, 2.0),
                           temp_choices=(0.7, 1.0))
    inputs = synth.make_round(spec, device="cuda", seed=V + G + 1)
    for flags in (1, 0):
        gpu = _sharded(binding, sharding, inputs, G, 0, flags, align, recover_mode=2)
        stats = P.compare(oracle_mod, gpu, P.to_np_inputs(inputs), 0, 2, flags, P.TOL[inputs["h_llm"].dtype])
        assert stats["excused_token"] == 0


def test_sharded_greedy_tie_across_shards_takes_the_lower_global_id(oracle_mod):
    from paper_2603_16219_b200 import binding, build, sharding, synth
    build.build()
    spec = synth.RoundSpec("vocab_shards_tie", 2, 1, 4096, "f32")
    inputs = synth.make_round(spec, device="cuda", seed=3)
    for k in ("h_llm", "h_slm_plus", "h_slm_minus"):
        inputs[k].fill_(0.5)
    inputs["h_llm"][1, :, 3000] = 2.0            # request 1: one maximiser in the third shard
    gpu = _sharded(binding, sharding, inputs, 4, 0, 1, 4, recover_mode=2)
    assert gpu["rec_token"][0] == 0 and gpu["rec_token"][1] == 3000
    P.compare(oracle_mod, gpu, P.to_np_inputs(inputs), 0, 2, 1, P.TOL[torch.float32])
