"""The library's failure detector, exercised without hanging or faulting anything.

Every wait inside the streaming kernel is bounded; when one runs out the CTA records the error, waits for the
copies it has in flight and returns.  Here the limit is set to a few hundred SM clocks, which the very first wait
for a tile's bytes (a trip to HBM) exceeds: the kernel gives up at once, the host reads SPECSTEER_ERR_TIMEOUT, the
context refuses further rounds, and a fresh context computes the round correctly.
"""
import numpy as np
import pytest
import torch

import _parity as P

pytestmark = pytest.mark.gpu


def test_a_bounded_wait_that_runs_out_is_reported_and_poisons_only_its_context(oracle_mod):
    from paper_2603_16219_b200 import binding as b, build, synth
    assert torch.cuda.is_available()
    build.build()
    spec = synth.CONFIGS[0]
    inputs = synth.make_round(spec, device="cuda", seed=0)
    outs = b.alloc_outputs(spec.B, spec.K, "cuda")
    desc = b.make_desc(inputs, outs, flags=b.FLAG_BONUS)
    ctx = b.Context(spec.B, spec.K, spec.V, device=0)
    assert ctx.device_error() == 0
    with pytest.raises(b.SpecSteerError) as e:
        ctx.set_wait_limit(-1)
    assert e.value.code == b.ERR_INVALID_ARG
    ctx.set_wait_limit(300)                       # SM clocks: far below the latency of the first tile
    ctx.verify_round(desc)                        # the launches themselves succeed: the kernel returns by itself
    ctx.recover_sample(desc)
    torch.cuda.synchronize()                      # no hang, no fault: the device is still usable
    assert ctx.device_error() == b.ERR_TIMEOUT
    assert ctx.device_error() == b.ERR_TIMEOUT    # sticky
    for call in (ctx.verify_round, ctx.recover_sample, ctx.round_host):
        with pytest.raises(b.SpecSteerError) as e:
            call(desc)
        assert e.value.code == b.ERR_TIMEOUT
    ctx.set_wait_limit(0)                         # the default limit does not revive a poisoned context
    with pytest.raises(b.SpecSteerError) as e:
        ctx.verify_round(desc)
    assert e.value.code == b.ERR_TIMEOUT
    ctx.close()
    # a fresh context on the same device is unaffected and matches the oracle
    fresh = b.Context(spec.B, spec.K, spec.V, device=0)
    gpu = P.run_gpu(fresh, inputs, 0, 0, 1)
    P.compare(oracle_mod, gpu, P.to_np_inputs(inputs), 0, 0, 1, 1e-4)
    # and a generous limit changes nothing
    fresh.set_wait_limit(1 << 31)
    again = P.run_gpu(fresh, inputs, 0, 0, 1)
    for k in gpu:
        assert np.array_equal(gpu[k], again[k], equal_nan=True), k
    fresh.close()
