#!/usr/bin/env python
"""Benchmark of the SpecSteer verify + recover round on B200.

One step = specsteer_verify_round + specsteer_recover_sample over one batch of synthetic logits
(default: B=256, K=4, V=151936, float32 - the batched serving shape).  Prints ONE JSON line:
verified draft positions/s with inputs resident in HBM (`value`), the same through the host-buffer
entry point with the copies inside the timed region (`e2e`), the roofline of the streaming kernel,
the CPU oracle timed on this machine's cores, and the clocks seen while timing.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config 0..4] [--impl reference]

Under torchrun every rank runs its own batch (requests shard with no collective on the data path).
"""
import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "verified_draft_positions_per_sec"
UNIT = "positions/s"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1400.0   # sustained, under the power cap
NOMINAL_HBM_GBS = 8000.0
# DRAM bytes (read + write) per used row of the streaming kernel, from the ncu captures summarised under
# profiles/ (taken on 32 requests of the same recipe; traffic grows in proportion to the rows, so the figure for a
# full launch is an extrapolation), keyed by configuration.  Absent = not captured for the kernel as it stands.
NCU_TRAFFIC_BYTES_PER_ROW = {3: 1846800, 4: 1552483}
# The streaming kernel's sources as they were when those counters were taken (sha256 over the files below, in this
# order): when they have changed since, the traffic figure no longer describes the kernel and is reported as null.
NCU_TRAFFIC_SOURCES = ("verify.cu", "common.cuh", "records.cuh", "internal.h")
NCU_TRAFFIC_SOURCE_SHA256 = "163d49c9adb3240b8a6229a919699eb0a8365fb3742fb2991474c04c667fee7d"


def _traffic_still_valid():
    import hashlib
    h = hashlib.sha256()
    try:
        for name in NCU_TRAFFIC_SOURCES:
            with open(os.path.join(ROOT, "paper_2603_16219_b200", "csrc", name), "rb") as f:
                h.update(f.read())
    except OSError:
        return False
    return h.hexdigest() == NCU_TRAFFIC_SOURCE_SHA256


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler(threading.Thread):
    """Reads SM clock and throttle reasons (read-only NVML queries) every ~10 ms while timing runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.samples, self.windows, self._stop_evt = [], [], threading.Event()
        self.max_mhz = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def run(self):
        if self.nv is None:
            return
        nv = self.nv
        while not self._stop_evt.is_set():
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                try:
                    reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    reasons = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.samples.append((time.perf_counter(), mhz, int(reasons)))
            except Exception:
                pass
            time.sleep(0.01)

    def stop(self):
        self._stop_evt.set()

    def window(self, t0, t1):
        self.windows.append((t0, t1))

    def summary(self):
        names = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap",
                 0x80: "hw_power_brake_slowdown"}
        ins = [s for s in self.samples if any(a <= s[0] <= b for a, b in self.windows)]
        scope = "timed regions"
        if not ins:
            ins, scope = self.samples, "whole run (timed regions shorter than the sampling period)"
        if not ins:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0, "scope": "nvml unavailable"}
        mhz = sorted(s[1] for s in ins)
        bits = 0
        for s in ins:
            bits |= s[2]
        return {"sm_mhz": mhz[len(mhz) // 2], "sm_max_mhz": self.max_mhz,
                "reasons": [n for b, n in names.items() if bits & b], "samples": len(ins), "scope": scope}


def _sample_requests(spec, n):
    """Indices of a bounded sample that keeps the workload's mix: spread evenly over the sigma blocks."""
    import numpy as np
    n = max(1, min(n, spec.B))
    return np.unique(np.linspace(0, spec.B - 1, n).round().astype(int))


def _oracle_time(oracle, synth, inputs, sel, flags, nthreads):
    import torch
    idx = torch.as_tensor(sel, device=inputs["h_llm"].device)
    npin = {k: (synth.to_numpy_bits(v[idx]) if k.startswith("h_") else v[idx].cpu().numpy()) for k, v in inputs.items()}
    t0 = time.perf_counter()
    out = oracle.verify_recover_round(
        npin["h_llm"], npin["h_slm_plus"], npin["h_slm_minus"], npin["draft_tokens"], npin["draft_len"],
        npin["lam"], npin["beta"], npin["temperature"], npin["u_accept"], npin["u_recover"],
        flags=flags, nthreads=nthreads)
    dt = time.perf_counter() - t0
    return dt, int(npin["draft_len"].sum()), out


def run_reference(args, rank, world):
    """The reference arm: the CPU oracle, as it stands, on this machine's host cores (rank 0 only)."""
    if rank != 0:
        return
    import torch
    import oracle
    from paper_2603_16219_b200 import synth
    oracle.build()
    spec = synth.CONFIGS[args.config]
    cores = oracle.max_threads()
    # inputs for the sample only: generate a reduced batch of the same recipe on the CPU
    probe_B = min(spec.B, max(8, cores))        # at least one request per host thread
    small = synth.RoundSpec(spec.name + "_sample", probe_B, spec.K, spec.V, spec.dtype, sigma_plus=spec.sigma_plus,
                            heavy_tail=spec.heavy_tail, ragged=spec.ragged, beta_choices=spec.beta_choices,
                            beta_uniform=spec.beta_uniform, temp_choices=spec.temp_choices, lam=spec.lam)
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    inputs = synth.make_round(small, device=dev, seed=0)
    flags = oracle.FLAG_BONUS
    dt, _, _ = _oracle_time(oracle, synth, inputs, list(range(probe_B)), flags, cores)
    per_req = dt / probe_B                        # wall time per request with every thread busy
    budget = 120.0 / max(1, args.steps + args.warmup)
    n_req = int(max(min(probe_B, cores), min(probe_B, budget / max(per_req, 1e-6))))
    ends = [i // 2 if i % 2 == 0 else probe_B - 1 - i // 2 for i in range(probe_B)]   # alternate both regimes
    sel = sorted(ends[:n_req])
    for _ in range(args.warmup):
        _oracle_time(oracle, synth, inputs, sel, flags, cores)
    tot, pos = 0.0, 0
    for _ in range(args.steps):
        dt, p, _ = _oracle_time(oracle, synth, inputs, sel, flags, cores)
        tot += dt
        pos += p
    value = pos / tot
    sample = "%d of %d requests of %s per step (same recipe, seed 0), all %d rows each" % (n_req, spec.B, spec.name, spec.K + 1)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": spec.name, "B": spec.B, "K": spec.K, "V": spec.V, "logit_dtype": spec.dtype,
                   "accept_mode": "ratio", "recover_mode": "steer", "bonus_row": True, "lambda": spec.lam},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def _time_rounds(torch, ctx, descs, stream, steps, barrier, n_pairs=16):
    """Times `steps` whole rounds (verify + recover) cycling over `descs`; on `n_pairs` of them the library also
    records an event pair around the streaming kernel.  Returns (ms per step, streaming-kernel ms, wall window)."""
    n_pairs = max(1, min(steps, n_pairs))
    stride = max(1, steps // n_pairs)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_pairs)]
    for a, b in evs:
        a.record(stream)
        b.record(stream)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for i in range(3):
        ctx.verify_round(descs[i % len(descs)], stream)
        ctx.recover_sample(descs[i % len(descs)], stream)
    barrier()
    w0 = time.perf_counter()
    e0.record(stream)
    used = 0
    for i in range(steps):
        d = descs[i % len(descs)]
        hook = i % stride == 0 and used < n_pairs
        if hook:
            ctx.time_streaming(*evs[used])
        ctx.verify_round(d, stream)
        ctx.recover_sample(d, stream)
        if hook:
            ctx.time_streaming(None, None)
            used += 1
    e1.record(stream)
    barrier()
    w1 = time.perf_counter()
    ks = [a.elapsed_time(b) for a, b in evs[:used]]
    return e0.elapsed_time(e1) / steps, (sum(ks) / used, min(ks)), (w0, w1)


def _ex2_rate(torch, binding, dev, stream, sampler):
    """Measured ex2.approx throughput of this GPU: a few milliseconds of the library's probe kernel, CUDA events.
    Returns (evaluations per second, wall window) - the window lets the clock sampler say at which SM clock."""
    n_sm = torch.cuda.get_device_properties(dev).multi_processor_count
    n_ctas, iters = 2 * n_sm, 4096
    sink = torch.empty(n_ctas * 1024, dtype=torch.float32, device=dev)
    binding.probe_ex2(n_ctas, 64, sink, stream)          # warm-up (loads the kernel)
    torch.cuda.synchronize(dev)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    w0 = time.perf_counter()
    a.record(stream)
    n = 0
    for _ in range(4):
        n += binding.probe_ex2(n_ctas, iters, sink, stream)
    b.record(stream)
    torch.cuda.synchronize(dev)
    w1 = time.perf_counter()
    return n / (a.elapsed_time(b) * 1e-3), (w0, w1), n_sm


def _largest_config(torch, binding, synth, dev, local_rank, stream, barrier, sampler, peak, steps):
    """Config 4 (B=512, K=6, V=256000, bf16; 5.5 GB of logits): the round with every output, and the round asked for
    Algorithm 1's outputs only (two-phase), each with the streaming launch timed by the library's event pair."""
    spec = synth.CONFIGS[4]
    inputs = synth.make_round(spec, device=dev, seed=0)
    rows = synth.used_rows(spec, inputs["draft_len"], bonus=True)
    positions = int(inputs["draft_len"].sum().item())
    ctx = binding.Context(spec.B, spec.K, spec.V, device=local_rank)
    flags = binding.FLAG_BONUS
    outs = binding.alloc_outputs(spec.B, spec.K, dev)
    lean_outs = {k: v for k, v in outs.items() if k not in ("logp_plus", "logp_star", "log_z")}
    block = {"workload": spec.name, "dtype": "bf16", "B": spec.B, "K": spec.K, "V": spec.V,
             "positions_per_step": positions, "l2": "inputs exceed L2"}
    wins = []
    # every output: three tensors, every used row, four normalisers
    ms, (kms, kmin), win = _time_rounds(torch, ctx, [binding.make_desc(inputs, outs, flags=flags)], stream, steps, barrier)
    wins.append(win)
    nbytes = spec.logit_bytes(rows)
    ach = nbytes / (kms * 1e-3) / 1e9
    block["all_outputs"] = {
        "kernel": "verify_kernel", "kernel_ms": kms, "kernel_ms_fastest_launch": kmin,
        "algorithmic_bytes_per_launch": nbytes, "achieved": ach, "unit": "GB/s",
        "frac": ach / peak, "frac_of_nominal_8TBs": ach / NOMINAL_HBM_GBS, "ms_per_step": ms,
        "whole_step_gbs": nbytes / (ms * 1e-3) / 1e9, "whole_step_frac_of_nominal_8TBs": nbytes / (ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
        "positions_per_s": positions / (ms * 1e-3), "steps": steps}
    acc_all = outs["accept_len"].clone()
    # Algorithm 1's outputs only: verification streams h_LLM and h_SLM- over the drafted rows (Eq. 7), recovery then
    # streams row accept_len of every request that takes a token, all three tensors (Eq. 8)
    ms, (kms, kmin), win = _time_rounds(torch, ctx, [binding.make_desc(inputs, lean_outs, flags=flags)], stream, steps, barrier)
    wins.append(win)
    vbytes = 2 * positions * spec.V * spec.elem_bytes
    sampling = int((lean_outs["rec_token"] >= 0).sum().item())
    rbytes = 3 * sampling * spec.V * spec.elem_bytes
    ach = vbytes / (kms * 1e-3) / 1e9
    block["algorithm1_only"] = {
        "kernel": "verify_kernel (two tensors, drafted rows)", "kernel_ms": kms, "kernel_ms_fastest_launch": kmin,
        "algorithmic_bytes_per_launch": vbytes,
        "achieved": ach, "unit": "GB/s", "frac": ach / peak, "frac_of_nominal_8TBs": ach / NOMINAL_HBM_GBS,
        "ms_per_step": ms, "algorithmic_bytes_per_step": vbytes + rbytes,
        "whole_step_gbs": (vbytes + rbytes) / (ms * 1e-3) / 1e9,
        "whole_step_frac_of_nominal_8TBs": (vbytes + rbytes) / (ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
        "positions_per_s": positions / (ms * 1e-3), "steps": steps,
        "same_accept_len_as_all_outputs": bool(torch.equal(lean_outs["accept_len"], acc_all))}
    assert ctx.device_error() == 0
    ctx.close()
    del inputs
    torch.cuda.empty_cache()
    return block, wins


def _vocab_sharded(torch, dist, binding, synth, sharding, dev, local_rank, rank, world, stream, barrier, steps):
    """Config 3 with the vocabulary split over the ranks (a tensor-parallel LM head's layout): the round with one
    all-gather of 64 bytes per row and rank and one MAX all-reduce of the per-request results (NCCL), and the same
    with the three LM heads fused in front, their rows split over the ranks.  One batch for the whole job."""
    spec = synth.CONFIGS[3]
    out = {"workload": spec.name, "ranks": world, "collectives": "all_gather(64 B x rows x ranks) + all_reduce(MAX) of 4 small arrays (NCCL)"}
    full = synth.make_round(spec, device=dev, seed=0)              # the same batch on every rank
    positions = int(full["draft_len"].sum().item())
    lo, hi = sharding.vocab_range(spec.V, rank, world, align=4)
    local = dict(full)
    for k in ("h_llm", "h_slm_plus", "h_slm_minus"):
        local[k] = full[k][:, :, lo:hi].contiguous()
    del full
    torch.cuda.empty_cache()
    ctx = binding.Context(spec.B, spec.K, max(hi - lo, 1), device=local_rank)
    outs = binding.alloc_outputs(spec.B, spec.K, dev)
    desc = binding.make_desc(local, outs, flags=binding.FLAG_BONUS)

    def timed(fn, n):
        for _ in range(3):
            fn()
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(n):
            fn()
        b.record(stream)
        barrier()
        t = torch.tensor([a.elapsed_time(b) / n], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    ms = timed(lambda: sharding.sharded_vocab_round(ctx, desc, outs, lo, spec.V, dist, stream), steps)
    out["logits_split"] = {"ms_per_step": ms, "positions_per_s": positions / (ms * 1e-3), "steps": steps,
                           "logit_bytes_per_rank": 3 * spec.rows * (hi - lo) * spec.elem_bytes,
                           "bytes_exchanged_per_rank": spec.rows * 64 * world + spec.B * (4 + 4 + 4 * (spec.K + 1) + 4)}
    assert ctx.device_error() == 0
    ctx.close()
    del local
    torch.cuda.empty_cache()
    # the fused form: hidden states replicated, the heads' rows split
    dL, dS = 5120, 2048
    lm = synth.make_lmhead_round(spec, dL, dS, device=dev, seed=0)
    lo, hi = sharding.vocab_range(spec.V, rank, world, align=8)
    lml = dict(lm)
    for k in ("w_llm", "w_slm_plus", "w_slm_minus"):
        lml[k] = lm[k][lo:hi].contiguous()
    del lm
    torch.cuda.empty_cache()
    ctx = binding.Context(spec.B, spec.K, max(hi - lo, 1), device=local_rank)
    ldesc = binding.make_lmhead_desc(lml, outs, flags=binding.FLAG_BONUS)
    steps_lm = max(3, min(steps, 30))
    ms = timed(lambda: sharding.sharded_lmhead_round(ctx, ldesc, outs, lo, spec.V, dist, stream), steps_lm)
    out["heads_split"] = {"ms_per_step": ms, "positions_per_s": positions / (ms * 1e-3), "steps": steps_lm,
                          "d_llm": dL, "d_slm": dS, "flops_per_rank": 2.0 * spec.rows * (hi - lo) * (dL + 2 * dS),
                          "tflops_per_rank": 2.0 * spec.rows * (hi - lo) * (dL + 2 * dS) / (ms * 1e-3) / 1e12}
    assert ctx.device_error() == 0
    ctx.close()
    return out


def run_cuda(args, rank, world, local_rank):
    import torch
    from paper_2603_16219_b200 import binding, build, synth
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    build.build()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1 or (args.vocab_sharded and "RANK" in os.environ):
        import torch.distributed as dist
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)

    spec = synth.CONFIGS[args.config]
    if args.requests:   # a reduced batch of the same recipe, for profiler captures that must stay small
        import dataclasses
        spec = dataclasses.replace(spec, B=args.requests, name="%s_first%d" % (spec.name, args.requests))
    flags = binding.FLAG_BONUS | (binding.FLAG_SEPARATE_LAUNCHES if args.separate else 0) | \
        (binding.FLAG_ONE_LAUNCH if args.one_launch else 0)
    inputs = synth.make_round(spec, device=dev, seed=rank)     # every rank owns its own requests
    rows = synth.used_rows(spec, inputs["draft_len"], bonus=True)
    positions = int(inputs["draft_len"].sum().item())
    logit_bytes = spec.logit_bytes(rows)
    two_phase = args.lean and 3 * spec.rows * spec.V * spec.elem_bytes >= 128 << 20   # the library's own rule
    if two_phase:   # the timed streaming launch reads two tensors over the drafted rows only
        logit_bytes = 2 * positions * spec.V * spec.elem_bytes
    ctx = binding.Context(spec.B, spec.K, spec.V, device=local_rank)
    outs = binding.alloc_outputs(spec.B, spec.K, dev)
    if args.lean:   # only what Algorithm 1 needs: verification then reads h_LLM and h_SLM- alone (Eq. 7) over the drafted
        # rows, and the recovery call streams its one row per request (Eq. 8)
        for name in ("logp_plus", "logp_star", "log_z"):
            outs.pop(name)
    rmode = binding.RECOVER_ARGMAX if args.greedy else binding.RECOVER_STEER
    desc = binding.make_desc(inputs, outs, flags=flags, recover_mode=rmode)
    stream = torch.cuda.current_stream(dev)

    # When the batch fits in L2 (126 MB) rotate over enough copies to exceed it; otherwise the batch itself does.
    l2_bytes = 126 << 20
    n_sets = 1 if 3 * spec.rows * spec.V * spec.elem_bytes > 2 * l2_bytes else \
        int((4 * l2_bytes) // max(1, 3 * spec.rows * spec.V * spec.elem_bytes)) + 1
    sets = [(inputs, desc)]
    for i in range(1, n_sets):
        cp = {k: v.clone() for k, v in inputs.items()}
        sets.append((cp, binding.make_desc(cp, outs, flags=flags, recover_mode=rmode)))

    def step(i):
        d = sets[i % n_sets][1]
        ctx.verify_round(d, stream)
        ctx.recover_sample(d, stream)

    sampler = ClockSampler(local_rank)
    sampler.start()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    for i in range(max(3, args.warmup)):
        step(i)
    barrier()
    # ---- the timed region: K whole steps, events on the launching stream.  On every `stride`-th step the library
    # also records an event pair around the streaming kernel (the launch that reads all the logits), so that kernel
    # is timed inside the same region, under the same clocks and power state as the step.  (An event between two
    # launches makes the epilogue wait for the whole streaming kernel instead of sliding under its tail, so the
    # hooked steps are a little slower than the others; hence only 32 of them.)
    n_pairs = min(args.steps, 32)       # few enough that breaking the dependent launch on those steps does not show
    stride = max(1, args.steps // n_pairs)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_pairs)]
    for a, b in evs:            # a first record creates the CUDA handles the hook needs
        a.record(stream)
        b.record(stream)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = ctx.launch_count
    barrier()
    w0 = time.perf_counter()
    e0.record(stream)
    used = 0
    for i in range(args.steps):
        if i % stride == 0 and used < n_pairs:
            ctx.time_streaming(*evs[used])
            step(i)
            ctx.time_streaming(None, None)
            used += 1
        else:
            step(i)
    e1.record(stream)
    barrier()
    w1 = time.perf_counter()
    sampler.window(w0, w1)
    gpu_launches = ctx.launch_count - launches0
    total_ms = e0.elapsed_time(e1)
    kernel_ms = sum(a.elapsed_time(b) for a, b in evs[:used]) / used
    assert ctx.device_error() == 0

    if dist is not None:
        t = torch.tensor([total_ms], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    ms_per_step = total_ms / args.steps
    value = world * positions / (ms_per_step * 1e-3)

    if args.kernels_only:
        extra = {}
        if args.topk:
            # the top-k split recovery in place of recover_sample: the cloud kernel reads two rows per sampling request
            k = args.topk
            tidx = torch.empty((spec.B, k), dtype=torch.int32, device=dev)
            tval = torch.empty((spec.B, k), dtype=torch.float32, device=dev)
            n = min(args.steps, 100)
            ea = [torch.cuda.Event(enable_timing=True) for _ in range(3 * n)]
            for i in range(n + 3):
                d = sets[i % n_sets][1]
                ctx.verify_round(d, stream)
                j = 3 * (i - 3)
                if i >= 3:
                    ea[j].record(stream)
                ctx.cloud_topk(d, tidx, tval, stream)
                if i >= 3:
                    ea[j + 1].record(stream)
                ctx.edge_resample(d, tidx, tval, stream)
                if i >= 3:
                    ea[j + 2].record(stream)
            barrier()
            cloud_ms = sum(ea[3 * i].elapsed_time(ea[3 * i + 1]) for i in range(n)) / n
            edge_ms = sum(ea[3 * i + 1].elapsed_time(ea[3 * i + 2]) for i in range(n)) / n
            topk_bytes = 2 * spec.B * spec.V * spec.elem_bytes      # with the bonus row every request samples
            extra = {"topk_k": k, "cloud_topk_ms": cloud_ms, "cloud_topk_gbs": topk_bytes / (cloud_ms * 1e-3) / 1e9,
                     "cloud_topk_bytes": topk_bytes, "edge_resample_ms": edge_ms}
        if n_sets > 1:   # the cold figures above rotate input sets; the same round on ONE set, resident in L2, labelled
            for _ in range(5):
                step(0)
            w0e, w1e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            barrier()
            w0e.record(stream)
            for _ in range(args.steps):
                step(0)
            w1e.record(stream)
            barrier()
            extra["warm_l2_ms_per_step"] = w0e.elapsed_time(w1e) / args.steps
        sampler.stop()
        if rank == 0:
            line = {"workload": spec.name, "outputs": ("lean, two-phase" if two_phase else "lean, one pass") if args.lean else "all",
                    "recovery": "greedy (argmax of h_rec)" if args.greedy else "sampled", "ms_per_step": ms_per_step,
                    "launches_per_step": gpu_launches / args.steps,
                    "verify_kernel_ms": kernel_ms, "verify_gbs": logit_bytes / (kernel_ms * 1e-3) / 1e9,
                    "positions_per_s": value, "clocks": sampler.summary()}
            line.update(extra)
            print(json.dumps(line), flush=True)
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return
    # ---- beside the headline: the same batch with only the outputs Algorithm 1 needs (the two-phase round for
    # large batches: h_LLM and h_SLM- over the drafted rows, then one recovery row per request)
    alg1 = None
    if not args.lean:
        lean_outs = {k: v for k, v in binding.alloc_outputs(spec.B, spec.K, dev).items()
                     if k not in ("logp_plus", "logp_star", "log_z")}
        lean_sets = [binding.make_desc(si, lean_outs, flags=flags) for si, _ in sets]
        n_lean = min(args.steps, 200)
        for i in range(3):
            ctx.verify_round(lean_sets[i % n_sets], stream)
            ctx.recover_sample(lean_sets[i % n_sets], stream)
        barrier()
        l0, l1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        w0 = time.perf_counter()
        l0.record(stream)
        for i in range(n_lean):
            ctx.verify_round(lean_sets[i % n_sets], stream)
            ctx.recover_sample(lean_sets[i % n_sets], stream)
        l1.record(stream)
        barrier()
        sampler.window(w0, time.perf_counter())
        lean_ms = l0.elapsed_time(l1) / n_lean
        if dist is not None:
            t = torch.tensor([lean_ms], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            lean_ms = float(t.item())
        same = torch.equal(lean_outs["accept_len"], outs["accept_len"]) and torch.equal(lean_outs["rec_token"], outs["rec_token"])
        alg1 = {"value": world * positions / (lean_ms * 1e-3), "unit": UNIT, "ms_per_step": lean_ms, "steps": n_lean,
                "outputs": "no logp_plus, logp_star, log_z", "same_accept_len_and_tokens_as_headline": bool(same)}
        # the same outputs under greedy decoding (the paper's experimental setting): the token of largest h_rec
        greedy_sets = [binding.make_desc(si, lean_outs, flags=flags, recover_mode=binding.RECOVER_ARGMAX) for si, _ in sets]
        for i in range(3):
            ctx.verify_round(greedy_sets[i % n_sets], stream)
            ctx.recover_sample(greedy_sets[i % n_sets], stream)
        barrier()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        w0 = time.perf_counter()
        g0.record(stream)
        for i in range(n_lean):
            ctx.verify_round(greedy_sets[i % n_sets], stream)
            ctx.recover_sample(greedy_sets[i % n_sets], stream)
        g1.record(stream)
        barrier()
        sampler.window(w0, time.perf_counter())
        greedy_ms = g0.elapsed_time(g1) / n_lean
        if dist is not None:
            t = torch.tensor([greedy_ms], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            greedy_ms = float(t.item())
        alg1["greedy_recovery"] = {"value": world * positions / (greedy_ms * 1e-3), "unit": UNIT, "ms_per_step": greedy_ms,
                                   "steps": n_lean,
                                   "same_accept_len_as_headline": bool(torch.equal(lean_outs["accept_len"], outs["accept_len"]))}
    # ---- end to end: pinned host buffers in, pinned host results out, copies inside the timed region
    host_in = {k: v.cpu().pin_memory() for k, v in inputs.items()}
    host_out = binding.alloc_outputs(spec.B, spec.K, "cpu", pin=True)
    if args.lean:
        for name in ("logp_plus", "logp_star", "log_z"):
            host_out.pop(name)
    hdesc = binding.make_desc(host_in, host_out, flags=flags)
    h2d = sum(v.numel() * v.element_size() for v in host_in.values())
    d2h = sum(v.numel() * v.element_size() for v in host_out.values())
    e2e_steps = max(3, min(args.steps, 10))
    for _ in range(2):
        ctx.round_host(hdesc, stream)
    barrier()
    w0 = time.perf_counter()
    for _ in range(e2e_steps):
        ctx.round_host(hdesc, stream)
    torch.cuda.synchronize(dev)
    w1 = time.perf_counter()
    sampler.window(w0, w1)
    e2e_s = (w1 - w0) / e2e_steps
    if dist is not None:
        t = torch.tensor([e2e_s], device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_s = float(t.item())
    e2e_value = world * positions / e2e_s
    assert torch.equal(host_out["accept_len"], outs["accept_len"].cpu())
    # the same call asked for Algorithm 1's outputs only: it then copies just what the two-phase round reads
    e2e_alg1 = None
    if not args.lean:
        lean_host_out = {k: v for k, v in binding.alloc_outputs(spec.B, spec.K, "cpu", pin=True).items()
                         if k not in ("logp_plus", "logp_star", "log_z")}
        lean_hdesc = binding.make_desc(host_in, lean_host_out, flags=flags)
        for _ in range(2):
            ctx.round_host(lean_hdesc, stream)
        barrier()
        w0 = time.perf_counter()
        for _ in range(e2e_steps):
            ctx.round_host(lean_hdesc, stream)
        torch.cuda.synchronize(dev)
        w1 = time.perf_counter()
        sampler.window(w0, w1)
        lean_s = (w1 - w0) / e2e_steps
        if dist is not None:
            t = torch.tensor([lean_s], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            lean_s = float(t.item())
        n_acc = lean_host_out["accept_len"].to(torch.int64)
        dl = host_in["draft_len"].to(torch.int64)
        rows_copied = int(2 * spec.B * spec.K + (lean_host_out["rec_token"] >= 0).sum() + 2 * ((n_acc >= dl) & (lean_host_out["rec_token"] >= 0)).sum())
        e2e_alg1 = {"value": world * positions / lean_s, "unit": UNIT, "ms_per_step": 1e3 * lean_s, "steps": e2e_steps,
                    "h2d_bytes_per_step": rows_copied * spec.V * spec.elem_bytes + h2d - 3 * spec.rows * spec.V * spec.elem_bytes,
                    "same_accept_len_and_tokens": bool(torch.equal(lean_host_out["accept_len"], host_out["accept_len"]) and
                                                       torch.equal(lean_host_out["rec_token"], host_out["rec_token"]))}
    peak, peak_kind = _peaks()
    # ---- the largest configuration beside the headline (1 GPU runs of the default workload)
    largest = None
    if world == 1 and args.config == 3 and not args.requests and not args.lean and not args.no_extras:
        largest, wins = _largest_config(torch, binding, synth, dev, local_rank, stream, barrier, sampler, peak,
                                        max(10, min(args.steps, 100)))
        n0 = len(sampler.windows)
        for w in wins:
            sampler.window(*w)
        only = ClockSampler.__new__(ClockSampler)      # the clocks of those two timed regions alone
        only.samples, only.windows, only.max_mhz = sampler.samples, sampler.windows[n0:], sampler.max_mhz
        largest["clocks"] = only.summary()
    # ---- the measured special-function rate (the second ceiling of the streaming kernel)
    ex2_per_s, ex2_win, n_sm = _ex2_rate(torch, binding, dev, stream, sampler)
    probe_clk = ClockSampler.__new__(ClockSampler)
    probe_clk.samples, probe_clk.windows, probe_clk.max_mhz = sampler.samples, [ex2_win], sampler.max_mhz
    probe_clk = probe_clk.summary()
    # ---- several GPUs: the same configuration with the vocabulary split over the ranks
    sharded = None
    if dist is not None and (world > 1 or args.vocab_sharded) and args.config == 3 and not args.requests and not args.no_extras:
        from paper_2603_16219_b200 import sharding
        sharded = _vocab_sharded(torch, dist, binding, synth, sharding, dev, local_rank, rank, world, stream, barrier,
                                 max(10, min(args.steps, 100)))
    sampler.stop()

    if rank != 0:
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return

    achieved = logit_bytes / (kernel_ms * 1e-3) / 1e9
    traffic_ok = args.config in NCU_TRAFFIC_BYTES_PER_ROW and not args.requests and not args.lean and _traffic_still_valid()
    roofline = {
        "bound": "hbm", "kernel": "verify_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
        "frac": achieved / peak,
        "peak_source": "of " + peak_kind + " (a read+write copy: a read-only kernel can exceed it)",
        "traffic": (NCU_TRAFFIC_BYTES_PER_ROW[args.config] * rows if traffic_ok else None),
        "traffic_source": ("extrapolated: ncu dram bytes per row on a 32-request capture x rows of this launch"
                           if traffic_ok else "none: not captured for this workload, or the kernel's sources changed since"),
        "algorithmic_bytes_per_launch": logit_bytes, "kernel_ms": kernel_ms,
        "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
        "whole_step_gbs": logit_bytes / (ms_per_step * 1e-3) / 1e9,
        "whole_step_frac": logit_bytes / (ms_per_step * 1e-3) / 1e9 / peak,
        "whole_step_frac_of_nominal_8TBs": logit_bytes / (ms_per_step * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
    }
    # The second ceiling of the streaming kernel: one ex2.approx per normaliser and vocabulary entry on the
    # special-function unit, against the rate the probe kernel reached on this GPU a moment ago.
    clk = sampler.summary()
    if not args.lean:
        n_ex2 = 4.0 * rows * spec.V
        roofline["sfu"] = {"ex2_per_launch": n_ex2, "achieved": n_ex2 / (kernel_ms * 1e-3), "peak": ex2_per_s,
                           "unit": "ex2/s", "frac": n_ex2 / (kernel_ms * 1e-3) / ex2_per_s,
                           "peak_source": "measured: specsteer_probe_ex2, CUDA events",
                           "peak_per_clk_per_sm": (ex2_per_s / (probe_clk["sm_mhz"] * 1e6) / n_sm) if probe_clk.get("sm_mhz") else None,
                           "probe_sm_mhz": probe_clk.get("sm_mhz")}
    cpu = None
    if world == 1:
        import oracle
        oracle.build()
        cores = oracle.max_threads()
        probe = _sample_requests(spec, min(spec.B, cores))
        dt, pos, _ = _oracle_time(oracle, synth, inputs, probe, oracle.FLAG_BONUS, cores)
        n = int(min(spec.B, max(len(probe), 20.0 / max(dt / len(probe), 1e-9))))     # about 20 s of wall time at most
        sel = _sample_requests(spec, n)
        dt, pos, ora = _oracle_time(oracle, synth, inputs, sel, oracle.FLAG_BONUS, cores)
        got = outs["accept_len"].cpu().numpy()[sel]
        agree = int((got == ora["accept_len"]).sum())
        one = _sample_requests(spec, 2)
        dt1, pos1, _ = _oracle_time(oracle, synth, inputs, one, oracle.FLAG_BONUS, 1)
        cpu = {"value": pos / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": "%d of %d requests (evenly spaced over the batch), %.2f s wall on %d threads; "
                         "accept_len equal to the GPU's on %d of them" % (len(sel), spec.B, dt, cores, agree),
               "single_thread": {"value": pos1 / dt1, "unit": UNIT, "cores": 1,
                                 "sample": "%d requests, %.2f s wall" % (len(one), dt1)}}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": spec.dtype, "data": "synthetic",
        "config": {"workload": spec.name, "B": spec.B, "K": spec.K, "V": spec.V, "logit_dtype": spec.dtype,
                   "requests_per_gpu": spec.B, "rows_read_per_gpu": rows, "positions_per_step_per_gpu": positions,
                   "accept_mode": "ratio", "recover_mode": "steer", "bonus_row": True, "lambda": spec.lam,
                   "outputs": "Algorithm 1 only (no logp_plus, logp_star, log_z)" if args.lean else "all",
                   "acceptance_rate": float(outs["accept_len"].sum().item()) / max(1, positions),
                   "l2": ("inputs %.2f GB per step exceed L2" % (logit_bytes / 1e9)) if n_sets == 1 else
                         ("rotating %d input sets (%.2f GB) to exceed L2" % (n_sets, n_sets * logit_bytes / 1e9)),
                   "parallelism": "requests sharded over %d GPU(s), no collective" % world},
        "roofline": roofline,
        "cpu_baseline": cpu,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": 1e3 * e2e_s, "steps": e2e_steps, "api": "specsteer_round_host (pinned host buffers)",
                "algorithm1_outputs_only": e2e_alg1},
        "algorithm1_outputs_only": alg1,
        "largest_config": largest,
        "vocab_sharded": sharded,
        "gpu_launches": int(gpu_launches),
        "clocks": sampler.summary(),
    }
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def _tensor_peak():
    """Measured dense bf16 throughput (TFLOP/s): the sustained figure, since the kernel runs inside a long step."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            d = json.load(f)
        return float(d.get("bf16_tflops_sustained") or d["bf16_tflops"]), "measured (sustained)"
    except Exception:
        return FALLBACK_BF16_TFLOPS, "fallback"


def run_lmhead(args, local_rank):
    """The round with the LM heads fused in front (1 GPU): the hidden states and head weights of the benchmark
    shape go in, no logit is stored.  Beside it, the same work unfused: three library products into float32 logit
    tensors followed by the streaming round.  One short JSON line."""
    import dataclasses
    import torch
    from paper_2603_16219_b200 import binding, build, synth
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    build.build()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    spec = synth.CONFIGS[args.config]
    if args.requests:
        spec = dataclasses.replace(spec, B=args.requests, name="%s_first%d" % (spec.name, args.requests))
    dL, dS = args.d_llm, args.d_slm
    inputs = synth.make_lmhead_round(spec, dL, dS, device=dev, seed=0)
    B, K, V = spec.B, spec.K, spec.V
    rows = B * (K + 1)
    positions = int(inputs["draft_len"].sum().item())
    ctx = binding.Context(B, K, V, device=local_rank)
    outs = binding.alloc_outputs(B, K, dev)
    if args.lean:   # only Algorithm 1's outputs: the two-phase round (h_LLM and h_SLM- in verification, all three products
        # on the compacted recovery rows)
        for name in ("logp_plus", "logp_star", "log_z"):
            outs.pop(name)
    desc = binding.make_lmhead_desc(inputs, outs, flags=binding.FLAG_BONUS,
                                    recover_mode=binding.RECOVER_ARGMAX if args.greedy else binding.RECOVER_STEER)
    stream = torch.cuda.current_stream(dev)
    sampler = ClockSampler(local_rank)
    sampler.start()
    steps = min(args.steps, 50)
    for _ in range(max(3, min(args.warmup, 5))):
        ctx.lmhead_round(desc, stream)
    torch.cuda.synchronize(dev)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(min(steps, 16))]
    for a, b in evs:
        a.record(stream)
        b.record(stream)
    stride = max(1, steps // len(evs))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = ctx.launch_count
    torch.cuda.synchronize(dev)
    w0 = time.perf_counter()
    e0.record(stream)
    used = 0
    for i in range(steps):
        if i % stride == 0 and used < len(evs):
            ctx.time_streaming(*evs[used])
            ctx.lmhead_round(desc, stream)
            ctx.time_streaming(None, None)
            used += 1
        else:
            ctx.lmhead_round(desc, stream)
    e1.record(stream)
    torch.cuda.synchronize(dev)
    w1 = time.perf_counter()
    sampler.window(w0, w1)
    assert ctx.device_error() == 0
    fused_ms = e0.elapsed_time(e1) / steps
    kernel_ms = sum(a.elapsed_time(b) for a, b in evs[:used]) / used
    gpu_launches = ctx.launch_count - launches0
    fused_out = {k: v.clone() for k, v in outs.items()}

    # ---- the same work unfused: library products into float32 logits, then the streaming round
    h = {n: torch.empty(B, K + 1, V, dtype=torch.float32, device=dev) for n in ("h_llm", "h_slm_plus", "h_slm_minus")}
    li = {k: inputs[k] for k in ("draft_tokens", "draft_len", "lam", "beta", "temperature", "u_accept", "u_recover")}
    li.update(h)
    d2 = binding.make_desc(li, outs, flags=binding.FLAG_BONUS,
                           recover_mode=binding.RECOVER_ARGMAX if args.greedy else binding.RECOVER_STEER)
    pairs = (("h_llm", "x_llm", "w_llm"), ("h_slm_plus", "x_slm_plus", "w_slm_plus"), ("h_slm_minus", "x_slm_minus", "w_slm_minus"))

    def unfused():
        for hn, xn, wn in pairs:
            h[hn].view(rows, V).copy_(torch.matmul(inputs[xn].view(rows, -1), inputs[wn].t()))
        ctx.verify_round(d2, stream)
        ctx.recover_sample(d2, stream)

    for _ in range(3):
        unfused()
    torch.cuda.synchronize(dev)
    u0, u1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n_un = min(steps, 20)
    u0.record(stream)
    for _ in range(n_un):
        unfused()
    u1.record(stream)
    torch.cuda.synchronize(dev)
    unfused_ms = u0.elapsed_time(u1) / n_un
    same = float(((fused_out["accept_len"] == outs["accept_len"]) & (fused_out["rec_token"] == outs["rec_token"])).float().mean().item())
    sampler.stop()
    peak, peak_kind = _tensor_peak()
    flops = 2.0 * rows * V * (dL + 2 * dS)
    if args.lean:   # what the two tensor-core launches actually multiply: two products on every row, three on one row per request
        flops = 2.0 * rows * V * (dL + dS) + 2.0 * B * V * (dL + 2 * dS)
    achieved = flops / (kernel_ms * 1e-3) / 1e12
    line = {
        "workload": "%s_lmhead_dllm%d_dslm%d" % (spec.name, dL, dS), "metric": METRIC,
        "outputs": "Algorithm 1 only (two-phase: lmhead_ratio_kernel on every row, lmhead_kernel on the compacted recovery rows)" if args.lean else "all",
        "recovery": "greedy (argmax of h_rec)" if args.greedy else "sampled",
        "value": positions / (fused_ms * 1e-3), "unit": UNIT, "ms_per_step": fused_ms, "steps": steps, "dtype": "bf16",
        "roofline": {"bound": "tensor", "kernel": "lmhead_ratio_kernel + lmhead_kernel" if args.lean else "lmhead_kernel", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                     "frac": achieved / peak, "peak_source": "of " + peak_kind, "traffic": None,
                     "algorithmic_flops_per_launch": flops, "kernel_ms": kernel_ms},
        "unfused": {"ms_per_step": unfused_ms, "what": "three torch.matmul (library GEMM) products from the same bf16 operands, "
                    "copied into float32 logit tensors (bf16 product rounded once), then verify_round + recover_sample",
                    "requests_with_same_accept_len_and_token": same},
        "logit_bytes_never_stored": 3 * rows * V * 4,
        "gpu_launches": int(gpu_launches), "clocks": sampler.summary(),
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", type=int, default=3, help="index into the five benchmark configurations")
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--requests", type=int, default=0, help="override B (reduced batch for profiler captures)")
    ap.add_argument("--lean", action="store_true",
                    help="request only the outputs Algorithm 1 needs (no logp_plus, logp_star, log_z)")
    ap.add_argument("--topk", type=int, default=0,
                    help="with --kernels-only: also time the top-k split recovery (cloud + edge kernels) with this k")
    ap.add_argument("--kernels-only", action="store_true",
                    help="time only the device-resident steps and print a short line (profiling aid)")
    ap.add_argument("--separate", action="store_true",
                    help="keep verification and recovery in separate launches (small rounds otherwise run in one launch)")
    ap.add_argument("--one-launch", action="store_true",
                    help="take the one-launch round for a small batch of several requests too")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the blocks beside the headline (the largest configuration; the vocabulary-sharded rounds)")
    ap.add_argument("--vocab-sharded", action="store_true",
                    help="under torchrun with one rank: still time the vocabulary-sharded rounds (a check of that leg)")
    ap.add_argument("--greedy", action="store_true",
                    help="with --kernels-only: greedy recovery (the token of largest h_rec) instead of sampling")
    ap.add_argument("--lmhead", action="store_true",
                    help="time the round with the LM heads fused in front (hidden states and head weights in, 1 GPU)")
    ap.add_argument("--d-llm", type=int, default=5120, help="with --lmhead: hidden width of the Generalist")
    ap.add_argument("--d-slm", type=int, default=2048, help="with --lmhead: hidden width of the Specialist")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world == 1 and args.gpus > 1:
        # launched without torchrun: re-launch one process per GPU
        import subprocess
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
               "--master-addr", "127.0.0.1", "--master-port", str(29500 + os.getpid() % 1000), os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.call(cmd))
    if args.impl == "reference":
        run_reference(args, rank, world)
    elif args.lmhead:
        if rank == 0:
            run_lmhead(args, local_rank)
    else:
        run_cuda(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
