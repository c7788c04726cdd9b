"""The entry point that allocates nothing (specsteer_verify_round_static) against specsteer_verify_round.

Some hosts cannot allocate device memory when they call the library - a plug-in under a memory manager
that owns the whole GPU, a latency-critical loop that must avoid the synchronisation an allocation can
imply - so the library keeps a fixed scratch array for them.  Both entry points run the same kernels, so
their outputs must be identical byte for byte, call after call, whatever an earlier call left in the
shared scratch.  This file sorts last on purpose: a run that stops at the first failure has then already
run every other test.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

VERIFY_OUTPUTS = ("accept_len", "accept_flags", "alpha", "logp_llm", "logp_minus", "logp_plus", "logp_star",
                  "log_z", "req_status")


def _both(binding, synth, ctx, spec, seed, accept_mode, recover_mode=0):
    inputs = synth.make_round(spec, device="cuda", seed=seed)
    ref = binding.alloc_outputs(spec.B, spec.K, "cuda")
    got = binding.alloc_outputs(spec.B, spec.K, "cuda")
    for t in got.values():                      # poison: the call must write every verify output itself
        t.view(torch.uint8).fill_(0xA5)
    ctx.verify_round(binding.make_desc(inputs, ref, accept_mode=accept_mode, recover_mode=recover_mode,
                                       flags=binding.FLAG_BONUS))
    desc = binding.make_desc(inputs, got, accept_mode=accept_mode, recover_mode=recover_mode, flags=binding.FLAG_BONUS)
    binding.verify_round_static(desc)           # warm-up: the first call on a device resolves the scratch array's
    torch.cuda.synchronize()                    # address, and the first launch of a kernel loads its code
    for t in got.values():
        t.view(torch.uint8).fill_(0xA5)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]  # the driver's own count of free device memory
    binding.verify_round_static(desc)
    torch.cuda.synchronize()
    # the property the entry point exists for: the call took no device memory
    assert torch.cuda.mem_get_info()[0] == free_before, spec.name
    for k in VERIFY_OUTPUTS:
        a, b = ref[k].cpu().numpy(), got[k].cpu().numpy()
        assert np.array_equal(a, b, equal_nan=True), (spec.name, k)
    return ref


def test_static_entry_point_matches_context_entry_point_on_consecutive_calls():
    from paper_2603_16219_b200 import binding, build, synth
    assert torch.cuda.is_available()
    build.build()
    ctx = binding.Context(max_B=64, max_K=6, max_V=40000, device=0)
    big = synth.RoundSpec("static_big", 40, 6, 33000, "bf16", ragged=True, beta_choices=(0.5, 1.0, 2.0),
                          temp_choices=(0.7, 1.0))
    small = synth.RoundSpec("static_small", 3, 2, 5003, "f32")
    # two calls in a row (the second, smaller one runs over what the first left in the scratch), then again
    out_big = _both(binding, synth, ctx, big, 1, binding.ACCEPT_RATIO)
    _both(binding, synth, ctx, small, 2, binding.ACCEPT_EXACT_Z)
    _both(binding, synth, ctx, big, 3, binding.ACCEPT_EXACT_Z)
    # a greedy-decoding descriptor (the paper's experimental setting) is served like any other: verification does
    # not depend on the recovery mode
    _both(binding, synth, ctx, small, 4, binding.ACCEPT_RATIO, recover_mode=binding.RECOVER_ARGMAX)
    assert int(out_big["accept_len"].sum()) > 0
    ctx.close()


def test_static_entry_point_rejects_shapes_beyond_its_scratch():
    from paper_2603_16219_b200 import binding, build, synth
    build.build()
    spec = synth.RoundSpec("too_many_requests", 1025, 0, 8, "f32")
    inputs = synth.make_round(spec, device="cuda", seed=0)
    outs = binding.alloc_outputs(spec.B, spec.K, "cuda")
    with pytest.raises(binding.SpecSteerError) as e:
        binding.verify_round_static(binding.make_desc(inputs, outs))
    assert e.value.code == binding.ERR_STATIC_LIMIT and "fixed scratch" in str(e.value)
    # too many partial records: 16 requests x 9 rows x ceil(2_000_000 / 1024) chunks
    desc = binding.make_desc(inputs, outs)
    desc.B, desc.K, desc.V, desc.ld_row, desc.ld_req = 16, 8, 2_000_000, 2_000_000, 9 * 2_000_000
    desc.draft_tokens = desc.u_accept = desc.lam      # K > 0 wants these two set; the call is refused before any launch
    with pytest.raises(binding.SpecSteerError) as e:
        binding.verify_round_static(desc)
    assert e.value.code == binding.ERR_STATIC_LIMIT
