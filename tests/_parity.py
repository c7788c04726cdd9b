"""Shared helpers for the GPU-vs-oracle parity tests (test infrastructure; not collected by pytest).

The rule being checked: accepted lengths and recovered token ids are bit-exact except where the oracle's
acceptance margin or CDF margin is below 1e-5; log-probabilities (log_z included) agree within 1e-4 (float32
logits) or 2e-3 (bf16 logits) absolute.  Greedy recovery: the oracle orders h_rec (Eq. 8) in double; the GPU's token
must be that one wherever the gap to the runner-up exceeds what rounding h_rec to float32 can move, and must lie in
the set of such near-ties otherwise; for float32 / bf16 logits it must also be the token the library's documented
tie-break (h_rec formed in float32 with one fused multiply-add, lowest id among equals) picks.
"""
import numpy as np
import torch

MARGIN = 1e-5
TOL = {torch.float32: 1e-4, torch.bfloat16: 2e-3}


def to_np_inputs(inputs, sel=None):
    """Host numpy copies of (a subset of requests of) the round's inputs; bf16 logits as uint16 bits."""
    from paper_2603_16219_b200 import synth
    out = {}
    for k, v in inputs.items():
        v = v if sel is None else v[sel]
        out[k] = synth.to_numpy_bits(v) if k.startswith("h_") else v.detach().cpu().numpy()
    return out


def _f64(a):
    """Exact float64 values of a logit array (bf16 arrives as uint16 bit patterns)."""
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


def run_oracle(oracle, npin, accept_mode, recover_mode, flags, V=None, force=None, nthreads=None, margin=MARGIN,
               alg1=False):
    """alg1: the oracle round that reads only what Algorithm 1 reads (h_LLM, h_SLM- on drafted rows; all three on the
    recovery row): the reference for the library's two-phase round."""
    if nthreads is None:
        nthreads = max(1, min(oracle.max_threads(), 32))
    if alg1:
        flags = flags | oracle.FLAG_ALG1_READS
    return oracle.verify_recover_round(
        npin["h_llm"], npin["h_slm_plus"], npin["h_slm_minus"], npin["draft_tokens"], npin["draft_len"],
        npin["lam"], npin["beta"], npin["temperature"], npin["u_accept"], npin["u_recover"],
        accept_mode=accept_mode, recover_mode=recover_mode, flags=flags, force_accept=force,
        margin_tol=margin, nthreads=nthreads, V=V)


def run_gpu(ctx, inputs, accept_mode, recover_mode, flags, V=None):
    from paper_2603_16219_b200 import binding
    out = binding.verify_recover_round(ctx, inputs, accept_mode=accept_mode, recover_mode=recover_mode,
                                       flags=flags, V=V)
    torch.cuda.synchronize()
    assert ctx.device_error() == 0
    return {k: v.cpu().numpy() for k, v in out.items()}


def _slice(npin, b):
    return {k: v[b:b + 1] for k, v in npin.items()}


def compare(oracle, gpu, npin, accept_mode, recover_mode, flags, tol, V=None, sel=None, margin=MARGIN, alg1=False,
            keys=None):
    """Assert parity of GPU outputs (dict of numpy, all requests) with the oracle on the requests `sel`
    (indices into the GPU batch; npin holds exactly those requests, in order).  Returns statistics.
    `margin` is the width below which a decision may differ (then it is forced in the oracle and the rest
    of the request is compared on that branch).  `alg1`: compare with the oracle round that reads only what
    Algorithm 1 reads (the two-phase round); `keys`: the GPU outputs that exist (default: all)."""
    MARGIN = margin
    ora = run_oracle(oracle, npin, accept_mode, recover_mode, flags, V=V, margin=margin, alg1=alg1)
    have = (lambda k: True) if keys is None else (lambda k: k in keys)
    Vv = npin["h_llm"].shape[-1] if V is None else V
    B = npin["draft_len"].shape[0]
    K = npin["draft_tokens"].shape[1]
    sel = np.arange(B) if sel is None else np.asarray(sel)
    g = {k: v[sel] for k, v in gpu.items()}
    stats = {"excused_accept": 0, "excused_token": 0, "max_logp_err": 0.0, "max_logz_err": 0.0, "requests": int(B)}

    for b in range(B):
        ob = {k: v[b] for k, v in ora.items()}
        # ---- accepted length: bit-exact, or excused by a sub-margin decision which is then forced
        force = None
        for _ in range(K + 1):
            if g["accept_len"][b] == ob["accept_len"]:
                break
            t = min(int(g["accept_len"][b]), int(ob["accept_len"]))
            assert ob["accept_margin"][t] < MARGIN, (
                "request %d: accept_len gpu %d vs oracle %d with margin %.3g at position %d"
                % (b, g["accept_len"][b], ob["accept_len"], ob["accept_margin"][t], t))
            if force is None:
                force = np.full((1, K), -1, np.int8)
            force[0, t] = int(g["accept_flags"][b][t])
            stats["excused_accept"] += 1
            one = run_oracle(oracle, _slice(npin, b), accept_mode, recover_mode, flags, V=V, force=force, nthreads=1,
                             margin=margin, alg1=alg1)
            ob = {k: v[0] for k, v in one.items()}
        assert g["accept_len"][b] == ob["accept_len"]
        assert g["req_status"][b] == ob["req_status"], (b, g["req_status"][b], ob["req_status"])
        # ---- accept flags at every drafted position
        for t in range(K):
            if g["accept_flags"][b][t] != ob["accept_flags"][t]:
                assert ob["accept_margin"][t] < MARGIN or (force is not None and force[0, t] >= 0), (b, t)
        # ---- recovered token
        if recover_mode == 2 and ob["rec_token"] >= 0 and g["rec_token"][b] >= 0:
            # greedy recovery: the oracle's token is the maximiser of h_rec in double.  Forming h_rec in float32 moves a
            # value by at most bound(v) = 2^-23 (|h_LLM| + |beta| (|h_SLM+| + |h_SLM-|)) (two roundings of the three
            # terms); on the LM-head path the logits themselves carry `margin`.  A different token is admissible only
            # if the two values are closer than that; a gap above it therefore forces equality.
            n = int(ob["accept_len"])
            bt = float(npin["beta"][b])
            hl, hp, hm = (_f64(npin[k][b, n, :Vv]) for k in ("h_llm", "h_slm_plus", "h_slm_minus"))
            fuzzy = npin["h_llm"].dtype == np.float64
            gt, ot = int(g["rec_token"][b]), int(ob["rec_token"])
            if gt != ot:
                r = hl + bt * (hp - hm)
                bound = 2.0 ** -23 * (np.abs(hl) + abs(bt) * (np.abs(hp) + np.abs(hm))) + (margin if fuzzy else 0.0)
                assert ob["cdf_margin"] <= bound[gt] + bound[ot], (b, gt, ot, ob["cdf_margin"])
                assert r[gt] + bound[gt] >= r[ot] - bound[ot], (b, gt, ot, r[gt], r[ot])
                stats["excused_token"] += 1
            if not fuzzy:   # the documented tie-break: the float32 form of Eq. 8, lowest id among equals
                assert gt == int(ob["rec_token_lo"]), (b, gt, int(ob["rec_token_lo"]), ot)
            if gt == ot:
                assert abs(g["rec_logprob"][b] - ob["rec_logprob"]) <= tol, (b, g["rec_logprob"][b], ob["rec_logprob"])
        elif g["rec_token"][b] != ob["rec_token"]:
            lo, hi = int(ob["rec_token_lo"]), int(ob["rec_token_hi"])
            assert ob["rec_token"] >= 0 and g["rec_token"][b] >= 0, (b, g["rec_token"][b], ob["rec_token"])
            assert ob["cdf_margin"] < MARGIN and lo <= g["rec_token"][b] <= hi, (
                "request %d: token gpu %d vs oracle %d (admissible %d..%d), cdf margin %.3g"
                % (b, g["rec_token"][b], ob["rec_token"], lo, hi, ob["cdf_margin"]))
            n = int(ob["accept_len"])
            mode = recover_mode if n < npin["draft_len"][b] else 0
            if ob["req_status"] & 8:
                mode = 0
            r = oracle.row(npin["h_llm"][b, n, :V], npin["h_slm_plus"][b, n, :V], npin["h_slm_minus"][b, n, :V],
                           beta=float(npin["beta"][b]), temperature=float(npin["temperature"][b]), recover_mode=mode)
            assert r["weights"][g["rec_token"][b]] > 0.0
            stats["excused_token"] += 1
        else:
            if ob["rec_token"] >= 0:
                assert abs(g["rec_logprob"][b] - ob["rec_logprob"]) <= tol, (b, g["rec_logprob"][b], ob["rec_logprob"])
            else:
                assert np.isnan(g["rec_logprob"][b])
        # ---- emitted sequence is consistent with (accept_len, token)
        n = int(g["accept_len"][b])
        want = list(npin["draft_tokens"][b][:n]) + ([int(g["rec_token"][b])] if g["rec_token"][b] >= 0 else [])
        assert g["n_out"][b] == len(want) == ob["n_out"]
        assert list(g["out_tokens"][b][:len(want)]) == want and (g["out_tokens"][b][len(want):] == -1).all()
        # ---- floating-point outputs
        for key in ("logp_llm", "logp_minus", "logp_plus", "logp_star", "alpha"):
            if not have(key):
                continue
            a, o = g[key][b].astype(np.float64), ob[key]
            assert (np.isnan(a) == np.isnan(o)).all(), (key, b, a, o)
            fin = np.isfinite(o)
            assert (a[~fin & ~np.isnan(o)] == o[~fin & ~np.isnan(o)]).all(), (key, b)
            if fin.any():
                err = np.abs(a[fin] - o[fin]).max()
                stats["max_logp_err"] = max(stats["max_logp_err"], float(err))
                assert err <= tol, (key, b, err)
        if have("log_z"):
            a, o = g["log_z"][b].astype(np.float64), ob["log_z"]
            assert (np.isnan(a) == np.isnan(o)).all(), ("log_z", b, a, o)
            fin = np.isfinite(o)
            if fin.any():
                err = np.abs(a[fin] - o[fin]).max()
                stats["max_logz_err"] = max(stats["max_logz_err"], float(err))
                assert err <= tol, ("log_z", b, err)
    return stats


def invariants(gpu, inputs, flags, tol):
    """Properties that hold at any size, checked on every request of a full-size run."""
    K = inputs["draft_tokens"].shape[1]
    dl = inputs["draft_len"].cpu().numpy()
    n = gpu["accept_len"]
    assert ((n >= 0) & (n <= dl)).all()
    fl = gpu["accept_flags"]
    pos = np.arange(K)[None, :]
    first_rej = np.where((fl == 0) & (pos < dl[:, None]), pos, K).min(1)
    assert (np.minimum(first_rej, dl) == n).all()
    al = gpu["alpha"]
    assert ((al >= 0) & (al <= 1)).all()
    for key in ("logp_llm", "logp_minus", "logp_plus", "logp_star"):
        v = gpu[key][pos < dl[:, None]]
        assert (v <= tol).all(), key
    ok = gpu["req_status"] == 0
    assert ok.all()
    sampled = (n < dl) | bool(flags & 1)
    assert ((gpu["rec_token"] >= 0) == sampled).all()
    assert (gpu["n_out"] == n + sampled).all()
    assert (gpu["rec_logprob"][sampled] <= tol).all()
