"""ctypes access to the CPU oracle (``specsteer_oracle.c``).

TEST INFRASTRUCTURE ONLY.  The oracle is the slow float64 restatement of one
SpecSteer Draft-Verify-Recover round (Algorithm 1 phases 2-3, Eq. 6-8) that the
CUDA library is checked against.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this package; the product package never
does, and this package imports nothing from the product.

Inputs are numpy arrays (bf16 logits as ``uint16`` bit patterns); outputs come
back as a dict of numpy arrays, floating point in float64.

Also here: the top-k split recovery of the deployment appendix (``cloud_topk_row``,
``edge_resample_row``, ``topk_recover_round``) and the LM-head step in front of the
round (``lmhead_logits``: h = x W^T in float64 from bf16 operands;
``lmhead_verify_recover_round``).  Every function is pinned
(tests/test_oracle_pins.py, test_oracle_topk_pins.py, test_oracle_lmhead_pins.py).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "specsteer_oracle.c")
_SRC_TOPK = os.path.join(_HERE, "specsteer_oracle_topk.c")
_HDR = os.path.join(_HERE, "specsteer_oracle.h")
_LIB = os.path.join(_HERE, "libspecsteer_oracle.so")

DTYPE_F32, DTYPE_BF16, DTYPE_F64 = 0, 1, 2
ACCEPT_RATIO, ACCEPT_EXACT_Z = 0, 1
RECOVER_STEER, RECOVER_RESIDUAL, RECOVER_ARGMAX = 0, 1, 2
FLAG_BONUS = 1
FLAG_ALG1_READS = 2   # the round reading only what Algorithm 1 reads (see specsteer_oracle.h)
REQ_BAD_TOKEN, REQ_BAD_LEN, REQ_NONFINITE, REQ_RESIDUAL_EMPTY, REQ_BAD_PARAM = 1, 2, 4, 8, 16


def build(force: bool = False) -> str:
    """Compile the oracle into a shared object next to its source (gcc -O2 -fopenmp)."""
    stale = (not os.path.exists(_LIB)) or any(
        os.path.getmtime(p) > os.path.getmtime(_LIB) for p in (_SRC, _SRC_TOPK, _HDR))
    if force or stale:
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-std=c99", "-Wall", "-shared", "-fPIC",
                               "-o", tmp, _SRC, _SRC_TOPK, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Args(C.Structure):
    _fields_ = [
        ("B", C.c_int32), ("K", C.c_int32), ("V", C.c_int32),
        ("ld_row", C.c_int64), ("ld_req", C.c_int64),
        ("dtype", C.c_int32), ("accept_mode", C.c_int32), ("recover_mode", C.c_int32),
        ("flags", C.c_uint32), ("nthreads", C.c_int32), ("margin_tol", C.c_double),
        ("h_llm", C.c_void_p), ("h_slm_plus", C.c_void_p), ("h_slm_minus", C.c_void_p),
        ("draft_tokens", C.c_void_p), ("draft_len", C.c_void_p),
        ("lam", C.c_void_p), ("beta", C.c_void_p), ("temperature", C.c_void_p),
        ("u_accept", C.c_void_p), ("u_recover", C.c_void_p), ("force_accept", C.c_void_p),
        ("accept_len", C.c_void_p), ("accept_flags", C.c_void_p),
        ("alpha", C.c_void_p), ("logp_llm", C.c_void_p), ("logp_minus", C.c_void_p),
        ("logp_plus", C.c_void_p), ("logp_star", C.c_void_p), ("log_z", C.c_void_p),
        ("rec_token", C.c_void_p), ("rec_logprob", C.c_void_p), ("out_tokens", C.c_void_p),
        ("n_out", C.c_void_p), ("req_status", C.c_void_p),
        ("accept_margin", C.c_void_p), ("cdf_margin", C.c_void_p),
        ("rec_token_lo", C.c_void_p), ("rec_token_hi", C.c_void_p),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.specsteer_oracle_round.argtypes = [C.POINTER(_Args)]
        _lib.specsteer_oracle_round.restype = C.c_int
        _lib.specsteer_oracle_logsumexp.argtypes = [C.c_void_p, C.c_int64]
        _lib.specsteer_oracle_logsumexp.restype = C.c_double
        _lib.specsteer_oracle_row.argtypes = [C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                              C.c_double, C.c_double, C.c_int,
                                              C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        _lib.specsteer_oracle_row.restype = C.c_int
        _lib.specsteer_oracle_max_threads.restype = C.c_int
        _lib.specsteer_oracle_cloud_topk_row.argtypes = [C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_float, C.c_int,
                                                         C.c_void_p, C.c_void_p]
        _lib.specsteer_oracle_cloud_topk_row.restype = C.c_int
        _lib.specsteer_oracle_edge_resample_row.argtypes = [C.c_int, C.c_int, C.c_void_p, C.c_float, C.c_float, C.c_int,
                                                            C.c_void_p, C.c_void_p, C.c_double,
                                                            C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        _lib.specsteer_oracle_edge_resample_row.restype = C.c_int
    return _lib


def max_threads() -> int:
    return int(lib().specsteer_oracle_max_threads())


def _logits(a):
    a = np.ascontiguousarray(a)
    if a.dtype == np.float32:
        return a, DTYPE_F32
    if a.dtype == np.uint16:
        return a, DTYPE_BF16
    if a.dtype == np.float64:
        return a, DTYPE_F64
    raise TypeError("logits must be float32, float64 or uint16 (bf16 bit patterns), got %s" % a.dtype)


def _p(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def logsumexp(x) -> float:
    x = np.ascontiguousarray(x, dtype=np.float64)
    return float(lib().specsteer_oracle_logsumexp(_p(x), x.size))


def row(h_llm, h_plus, h_minus, beta=1.0, temperature=1.0, recover_mode=RECOVER_STEER):
    """One vocabulary row: the four normalisers, log Softmax(h_rec) and the recovery weights."""
    hl, dt = _logits(h_llm)
    hp, dt2 = _logits(h_plus)
    hm, dt3 = _logits(h_minus)
    assert dt == dt2 == dt3 and hl.ndim == 1 and hl.shape == hp.shape == hm.shape
    V = hl.shape[0]
    lse4 = np.empty(4); lps = np.empty(V); w = np.empty(V); W = np.empty(1)
    rc = lib().specsteer_oracle_row(V, dt, _p(hl), _p(hp), _p(hm), float(beta), float(temperature),
                                    int(recover_mode), _p(lse4), _p(lps), _p(w), _p(W))
    if rc != 0:
        raise RuntimeError("oracle row failed: %d" % rc)
    return {"lse": lse4, "logp_star": lps, "weights": w, "W": float(W[0])}


def verify_recover_round(h_llm, h_slm_plus, h_slm_minus, draft_tokens, draft_len, lam, beta, temperature,
                         u_accept, u_recover, accept_mode=ACCEPT_RATIO, recover_mode=RECOVER_STEER,
                         flags=0, force_accept=None, margin_tol=1e-5, nthreads=1, V=None):
    """One round for B requests.  Logits are [B, K+1, ld_row] (ld_row >= V; pass V if padded)."""
    hl, dt = _logits(h_llm)
    hp, dt2 = _logits(h_slm_plus)
    hm, dt3 = _logits(h_slm_minus)
    assert dt == dt2 == dt3 and hl.ndim == 3 and hl.shape == hp.shape == hm.shape
    B, K1, ld = hl.shape
    K = K1 - 1
    V = ld if V is None else int(V)
    tok = np.ascontiguousarray(draft_tokens, dtype=np.int32).reshape(B, K)
    dl = np.ascontiguousarray(draft_len, dtype=np.int32).reshape(B)
    lam = np.ascontiguousarray(lam, dtype=np.float32).reshape(B)
    beta = np.ascontiguousarray(beta, dtype=np.float32).reshape(B)
    tmp = np.ascontiguousarray(temperature, dtype=np.float32).reshape(B)
    ua = np.ascontiguousarray(u_accept, dtype=np.float32).reshape(B, K)
    ur = np.ascontiguousarray(u_recover, dtype=np.float32).reshape(B)
    fa = None if force_accept is None else np.ascontiguousarray(force_accept, dtype=np.int8).reshape(B, K)
    out = {
        "accept_len": np.empty(B, np.int32), "accept_flags": np.empty((B, K), np.uint8),
        "alpha": np.empty((B, K)), "logp_llm": np.empty((B, K)), "logp_minus": np.empty((B, K)),
        "logp_plus": np.empty((B, K)), "logp_star": np.empty((B, K)), "log_z": np.empty((B, K + 1)),
        "rec_token": np.empty(B, np.int32), "rec_logprob": np.empty(B),
        "out_tokens": np.empty((B, K + 1), np.int32), "n_out": np.empty(B, np.int32),
        "req_status": np.empty(B, np.int32), "accept_margin": np.empty((B, K)),
        "cdf_margin": np.empty(B), "rec_token_lo": np.empty(B, np.int32), "rec_token_hi": np.empty(B, np.int32),
    }
    a = _Args(B=B, K=K, V=V, ld_row=ld, ld_req=K1 * ld, dtype=dt, accept_mode=int(accept_mode),
              recover_mode=int(recover_mode), flags=int(flags), nthreads=int(nthreads),
              margin_tol=float(margin_tol),
              h_llm=_p(hl), h_slm_plus=_p(hp), h_slm_minus=_p(hm), draft_tokens=_p(tok), draft_len=_p(dl),
              lam=_p(lam), beta=_p(beta), temperature=_p(tmp), u_accept=_p(ua), u_recover=_p(ur),
              force_accept=_p(fa), **{k: _p(v) for k, v in out.items()})
    rc = lib().specsteer_oracle_round(C.byref(a))
    if rc != 0:
        raise RuntimeError("oracle round failed: %d" % rc)
    return out


def cloud_topk_row(h_llm, h_minus, beta, k):
    """Cloud half of the top-k split recovery on one row: (ids[k] int32, values[k] float32)."""
    hl, dt = _logits(h_llm)
    hm, dt2 = _logits(h_minus)
    assert dt == dt2 and dt != DTYPE_F64 and hl.ndim == 1 and hl.shape == hm.shape
    idx = np.empty(k, np.int32)
    val = np.empty(k, np.float32)
    rc = lib().specsteer_oracle_cloud_topk_row(hl.shape[0], dt, _p(hl), _p(hm), float(beta), int(k), _p(idx), _p(val))
    if rc != 0:
        raise RuntimeError("oracle cloud_topk_row failed: %d" % rc)
    return idx, val


def edge_resample_row(h_plus, beta, temperature, idx, val, u):
    """Edge half on one row: dict(token, logprob, probs[k], cdf_margin)."""
    hp, dt = _logits(h_plus)
    assert dt != DTYPE_F64
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    val = np.ascontiguousarray(val, dtype=np.float32)
    k = idx.shape[0]
    tok = np.empty(1, np.int32); lp = np.empty(1); probs = np.empty(k); mg = np.empty(1)
    rc = lib().specsteer_oracle_edge_resample_row(hp.shape[0], dt, _p(hp), float(beta), float(temperature), k,
                                                  _p(idx), _p(val), float(u), _p(tok), _p(lp), _p(probs), _p(mg))
    if rc != 0:
        raise RuntimeError("oracle edge_resample_row failed: %d" % rc)
    return {"token": int(tok[0]), "logprob": float(lp[0]), "probs": probs, "cdf_margin": float(mg[0])}


def topk_recover_round(h_llm, h_slm_plus, h_slm_minus, draft_len, beta, temperature, u_recover, accept_len, req_status,
                       k, flags=0):
    """Top-k split recovery for a verified batch: for every request that samples (accept_len < draft_len, or
    always with FLAG_BONUS; never after a BAD_PARAM / NONFINITE status) the cloud's list of row accept_len and the
    edge's token.  Returns dict(topk_idx[B,k], topk_val[B,k], rec_token[B], rec_logprob[B], cdf_margin[B])."""
    B = h_llm.shape[0]
    K = h_llm.shape[1] - 1
    out = {"topk_idx": np.full((B, k), -1, np.int32), "topk_val": np.full((B, k), -np.inf, np.float32),
           "rec_token": np.full(B, -1, np.int32), "rec_logprob": np.full(B, np.nan), "cdf_margin": np.full(B, np.inf)}
    for b in range(B):
        ln = int(draft_len[b])
        if ln < 0 or ln > K:
            ln = 0
        n = int(accept_len[b])
        bad = int(req_status[b]) & (REQ_BAD_PARAM | REQ_NONFINITE)
        if bad or not (n < ln or (flags & FLAG_BONUS)):
            continue
        idx, val = cloud_topk_row(h_llm[b, n], h_slm_minus[b, n], beta[b], k)
        r = edge_resample_row(h_slm_plus[b, n], beta[b], temperature[b], idx, val, float(u_recover[b]))
        out["topk_idx"][b], out["topk_val"][b] = idx, val
        out["rec_token"][b], out["rec_logprob"][b], out["cdf_margin"][b] = r["token"], r["logprob"], r["cdf_margin"]
    return out


# ---- the LM head in front of the round ------------------------------------------------------------------
def bf16_to_f64(bits):
    """Exact values of bf16 bit patterns (the upper half of an IEEE float32), as float64."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def lmhead_logits(x_bits, w_bits):
    """h = x W^T: the logits an LM head gives for hidden states x [..., d] and head weights W [V, d] (the h_LLM and
    h_SLM of Algorithm 1's verification and recovery steps), both bf16, every product and sum in float64."""
    x = bf16_to_f64(x_bits)
    w = bf16_to_f64(w_bits)
    assert x.shape[-1] == w.shape[1]
    return np.matmul(x, w.T)


def lmhead_verify_recover_round(x_llm, w_llm, x_plus, w_plus, x_minus, w_minus, draft_tokens, draft_len, lam, beta,
                                temperature, u_accept, u_recover, **kw):
    """The round of Algorithm 1 on logits that are first formed from hidden states [B, K+1, d] and head weights
    [V, d]: float64 logits, then `verify_recover_round` as it stands."""
    hl = lmhead_logits(x_llm, w_llm)
    hp = lmhead_logits(x_plus, w_plus)
    hm = lmhead_logits(x_minus, w_minus)
    return verify_recover_round(hl, hp, hm, draft_tokens, draft_len, lam, beta, temperature, u_accept, u_recover, **kw)
