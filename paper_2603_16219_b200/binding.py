"""Thin ctypes binding over ``libspecsteer.so`` (the C ABI declared in ``include/specsteer.h``).

Only argument marshalling lives here: torch tensors give device (or pinned-host) pointers and the
current CUDA stream; every step of the round runs inside the library's kernels.  There is no CPU
fallback: if the library has not been built, or no CUDA device is present, calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import torch

from . import build as _build

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_ORDER, ERR_TIMEOUT, ERR_STATIC_LIMIT = 1, 2, 3, 4, 5, 6, 7
F32, BF16 = 0, 1
ACCEPT_RATIO, ACCEPT_EXACT_Z = 0, 1
RECOVER_STEER, RECOVER_RESIDUAL, RECOVER_ARGMAX = 0, 1, 2
FLAG_BONUS = 1
FLAG_TWO_PHASE = 2
FLAG_SEPARATE_LAUNCHES = 4
FLAG_ONE_LAUNCH = 8
REQ_BAD_TOKEN, REQ_BAD_LEN, REQ_NONFINITE, REQ_RESIDUAL_EMPTY, REQ_BAD_PARAM = 1, 2, 4, 8, 16

EXPORTS = (
    "specsteer_ctx_create", "specsteer_ctx_destroy", "specsteer_verify_round", "specsteer_recover_sample",
    "specsteer_round_host", "specsteer_ctx_device_error", "specsteer_ctx_workspace_bytes",
    "specsteer_ctx_launch_count", "specsteer_status_string", "specsteer_version",
    "specsteer_verify_round_static", "specsteer_ctx_time_streaming",
    "specsteer_cloud_topk", "specsteer_edge_resample",
    "specsteer_shard_verify_local", "specsteer_shard_verify_combine", "specsteer_shard_recover_local",
    "specsteer_lmhead_round",
    "specsteer_lmhead_shard_local", "specsteer_lmhead_shard_combine", "specsteer_lmhead_shard_recover",
    "specsteer_shard_greedy_local", "specsteer_lmhead_shard_greedy_local", "specsteer_shard_greedy_finish",
    "specsteer_probe_ex2", "specsteer_ctx_set_wait_limit",
)
SHARD_PARTIAL_BYTES = 64
MAX_SHARDS = 32
TOPK_MAX = 32


class RoundDesc(C.Structure):
    """Mirror of ``specsteer_round_desc``."""
    _fields_ = [
        ("B", C.c_int32), ("K", C.c_int32), ("V", C.c_int32),
        ("ld_row", C.c_int64), ("ld_req", C.c_int64),
        ("dtype", C.c_int32), ("accept_mode", C.c_int32), ("recover_mode", C.c_int32), ("flags", C.c_uint32),
        ("h_llm", C.c_void_p), ("h_slm_plus", C.c_void_p), ("h_slm_minus", C.c_void_p),
        ("draft_tokens", C.c_void_p), ("draft_len", C.c_void_p),
        ("lam", C.c_void_p), ("beta", C.c_void_p), ("temperature", C.c_void_p),
        ("u_accept", C.c_void_p), ("u_recover", C.c_void_p),
        ("accept_len", C.c_void_p), ("accept_flags", C.c_void_p), ("alpha", C.c_void_p),
        ("logp_llm", C.c_void_p), ("logp_minus", C.c_void_p), ("logp_plus", C.c_void_p),
        ("logp_star", C.c_void_p), ("log_z", C.c_void_p),
        ("rec_token", C.c_void_p), ("rec_logprob", C.c_void_p), ("out_tokens", C.c_void_p),
        ("n_out", C.c_void_p), ("req_status", C.c_void_p),
    ]


class LmheadDesc(C.Structure):
    """Mirror of ``specsteer_lmhead_desc``."""
    _fields_ = [
        ("round", RoundDesc),
        ("x_llm", C.c_void_p), ("w_llm", C.c_void_p),
        ("x_slm_plus", C.c_void_p), ("w_slm_plus", C.c_void_p),
        ("x_slm_minus", C.c_void_p), ("w_slm_minus", C.c_void_p),
        ("d_llm", C.c_int32), ("d_slm", C.c_int32),
    ]


_lib = None


def load_library(path: Optional[str] = None):
    """dlopen the CUDA library (no CUDA call is made by loading it)."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or _build.LIB_PATH
    if not os.path.exists(path):
        raise RuntimeError(
            "libspecsteer.so is missing (%s): build it with `python -m paper_2603_16219_b200.build`; "
            "there is no CPU fallback" % path)
    lib = C.CDLL(path)
    lib.specsteer_ctx_create.argtypes = [C.POINTER(C.c_void_p), C.c_int, C.c_int32, C.c_int32, C.c_int32]
    lib.specsteer_ctx_create.restype = C.c_int
    lib.specsteer_ctx_destroy.argtypes = [C.c_void_p]
    lib.specsteer_ctx_destroy.restype = C.c_int
    for name in ("specsteer_verify_round", "specsteer_recover_sample", "specsteer_round_host"):
        fn = getattr(lib, name)
        fn.argtypes = [C.c_void_p, C.POINTER(RoundDesc), C.c_void_p]
        fn.restype = C.c_int
    lib.specsteer_verify_round_static.argtypes = [C.POINTER(RoundDesc), C.c_void_p]
    lib.specsteer_verify_round_static.restype = C.c_int
    lib.specsteer_ctx_device_error.argtypes = [C.c_void_p]
    lib.specsteer_ctx_device_error.restype = C.c_int
    lib.specsteer_ctx_workspace_bytes.argtypes = [C.c_void_p]
    lib.specsteer_ctx_workspace_bytes.restype = C.c_size_t
    lib.specsteer_cloud_topk.argtypes = [C.c_void_p, C.POINTER(RoundDesc), C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.specsteer_cloud_topk.restype = C.c_int
    lib.specsteer_edge_resample.argtypes = [C.c_void_p, C.POINTER(RoundDesc), C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.specsteer_edge_resample.restype = C.c_int
    lib.specsteer_shard_verify_local.argtypes = [C.c_void_p, C.POINTER(RoundDesc), C.c_int32, C.c_void_p, C.c_void_p]
    lib.specsteer_shard_verify_local.restype = C.c_int
    for name in ("specsteer_shard_verify_combine", "specsteer_shard_recover_local"):
        fn = getattr(lib, name)
        fn.argtypes = [C.c_void_p, C.POINTER(RoundDesc), C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]
        fn.restype = C.c_int
    lib.specsteer_lmhead_round.argtypes = [C.c_void_p, C.POINTER(LmheadDesc), C.c_void_p]
    lib.specsteer_lmhead_round.restype = C.c_int
    lib.specsteer_shard_greedy_local.argtypes = [C.c_void_p, C.POINTER(RoundDesc), C.c_int32, C.c_void_p, C.c_void_p]
    lib.specsteer_shard_greedy_local.restype = C.c_int
    lib.specsteer_lmhead_shard_greedy_local.argtypes = [C.c_void_p, C.POINTER(LmheadDesc), C.c_void_p, C.c_void_p]
    lib.specsteer_lmhead_shard_greedy_local.restype = C.c_int
    lib.specsteer_shard_greedy_finish.argtypes = [C.c_void_p, C.POINTER(RoundDesc), C.c_void_p, C.c_void_p]
    lib.specsteer_shard_greedy_finish.restype = C.c_int
    lib.specsteer_lmhead_shard_local.argtypes = [C.c_void_p, C.POINTER(LmheadDesc), C.c_int32, C.c_void_p, C.c_void_p]
    lib.specsteer_lmhead_shard_local.restype = C.c_int
    for fn in (lib.specsteer_lmhead_shard_combine, lib.specsteer_lmhead_shard_recover):
        fn.argtypes = [C.c_void_p, C.POINTER(LmheadDesc), C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]
        fn.restype = C.c_int
    lib.specsteer_ctx_set_wait_limit.argtypes = [C.c_void_p, C.c_int64]
    lib.specsteer_ctx_set_wait_limit.restype = C.c_int
    lib.specsteer_probe_ex2.argtypes = [C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
    lib.specsteer_probe_ex2.restype = C.c_int
    lib.specsteer_ctx_time_streaming.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
    lib.specsteer_ctx_time_streaming.restype = C.c_int
    lib.specsteer_ctx_launch_count.argtypes = [C.c_void_p]
    lib.specsteer_ctx_launch_count.restype = C.c_uint64
    lib.specsteer_status_string.argtypes = [C.c_int]
    lib.specsteer_status_string.restype = C.c_char_p
    lib.specsteer_version.restype = C.c_uint32
    _lib = lib
    return lib


class SpecSteerError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = load_library().specsteer_status_string(code).decode()
        super().__init__("%s failed: %s (%d)" % (where, msg, code))


def _check(code: int, where: str):
    if code != OK:
        raise SpecSteerError(code, where)


_OUT_SPECS = {
    # name: (dtype, per-request shape builder)
    "accept_len": (torch.int32, lambda K: ()), "accept_flags": (torch.uint8, lambda K: (K,)),
    "alpha": (torch.float32, lambda K: (K,)), "logp_llm": (torch.float32, lambda K: (K,)),
    "logp_minus": (torch.float32, lambda K: (K,)), "logp_plus": (torch.float32, lambda K: (K,)),
    "logp_star": (torch.float32, lambda K: (K,)), "log_z": (torch.float32, lambda K: (K + 1,)),
    "rec_token": (torch.int32, lambda K: ()), "rec_logprob": (torch.float32, lambda K: ()),
    "out_tokens": (torch.int32, lambda K: (K + 1,)), "n_out": (torch.int32, lambda K: ()),
    "req_status": (torch.int32, lambda K: ()),
}


def alloc_outputs(B: int, K: int, device, pin: bool = False) -> Dict[str, torch.Tensor]:
    """Caller-owned output tensors for one round (torch is only the allocator)."""
    out = {}
    for name, (dt, shp) in _OUT_SPECS.items():
        t = torch.empty((B,) + shp(K), dtype=dt, device=device)
        out[name] = t.pin_memory() if pin else t
    return out


def _fill_request_arrays(d: RoundDesc, inputs, outputs, B: int, K: int):
    """The per-request inputs and the outputs of a round descriptor (shared by both kinds of descriptor)."""
    def ptr(t, dt, n):
        if t.dtype != dt or not t.is_contiguous() or t.numel() != n:
            raise ValueError("bad auxiliary tensor: dtype %s, numel %d (want %s, %d)" % (t.dtype, t.numel(), dt, n))
        return t.data_ptr() if n else None

    d.draft_tokens = ptr(inputs["draft_tokens"], torch.int32, B * K)
    d.draft_len = ptr(inputs["draft_len"], torch.int32, B)
    d.lam = ptr(inputs["lam"], torch.float32, B)
    d.beta = ptr(inputs["beta"], torch.float32, B)
    d.temperature = ptr(inputs["temperature"], torch.float32, B)
    d.u_accept = ptr(inputs["u_accept"], torch.float32, B * K)
    d.u_recover = ptr(inputs["u_recover"], torch.float32, B)
    for name, (dt, shp) in _OUT_SPECS.items():
        t = outputs.get(name)
        n = B
        for s in shp(K):
            n *= s
        setattr(d, name, ptr(t, dt, n) if t is not None else None)


def make_desc(inputs: Dict[str, torch.Tensor], outputs: Dict[str, torch.Tensor], *, accept_mode=ACCEPT_RATIO,
              recover_mode=RECOVER_STEER, flags=0, V: Optional[int] = None) -> RoundDesc:
    """Fill a descriptor from tensors.  Logits: [B, K+1, ld_row] (last dim contiguous); pass V if ld_row > V."""
    hl, hp, hm = inputs["h_llm"], inputs["h_slm_plus"], inputs["h_slm_minus"]
    if hl.dim() != 3 or hl.shape != hp.shape or hl.shape != hm.shape or hl.dtype != hp.dtype or hl.dtype != hm.dtype:
        raise ValueError("logit tensors must share shape [B, K+1, V] and dtype")
    if hl.dtype not in (torch.float32, torch.bfloat16):
        raise ValueError("logits must be float32 or bfloat16")
    for t in (hl, hp, hm):
        if t.stride(2) != 1 or t.stride() != hl.stride():
            raise ValueError("logit tensors need a contiguous vocabulary axis and equal strides")
    B, K1, ld = hl.shape
    d = RoundDesc()
    d.B, d.K, d.V = B, K1 - 1, int(V if V is not None else ld)
    d.ld_row = hl.stride(1) if K1 > 1 else ld          # strides of size-1 axes carry no information
    d.ld_req = hl.stride(0) if B > 1 else K1 * d.ld_row
    d.dtype = F32 if hl.dtype == torch.float32 else BF16
    d.accept_mode, d.recover_mode, d.flags = int(accept_mode), int(recover_mode), int(flags)
    d.h_llm, d.h_slm_plus, d.h_slm_minus = hl.data_ptr(), hp.data_ptr(), hm.data_ptr()
    _fill_request_arrays(d, inputs, outputs, B, K1 - 1)
    return d


def make_lmhead_desc(inputs: Dict[str, torch.Tensor], outputs: Dict[str, torch.Tensor], *, accept_mode=ACCEPT_RATIO,
                     recover_mode=RECOVER_STEER, flags=0) -> LmheadDesc:
    """Descriptor of a round on hidden states and head weights: inputs hold x_llm [B, K+1, d_llm], w_llm [V, d_llm],
    x_slm_plus / x_slm_minus [B, K+1, d_slm], w_slm_plus / w_slm_minus [V, d_slm] (bf16, contiguous) and the
    per-request tensors of ``make_desc``."""
    xl, wl = inputs["x_llm"], inputs["w_llm"]
    xp, wp, xm, wm = inputs["x_slm_plus"], inputs["w_slm_plus"], inputs["x_slm_minus"], inputs["w_slm_minus"]
    for t in (xl, wl, xp, wp, xm, wm):
        if t.dtype != torch.bfloat16 or not t.is_contiguous():
            raise ValueError("hidden states and head weights must be contiguous bfloat16 tensors")
    B, K1, dL = xl.shape
    V, dS = wp.shape
    if wl.shape != (V, dL) or xp.shape != (B, K1, dS) or xm.shape != (B, K1, dS) or wm.shape != (V, dS):
        raise ValueError("operand shapes do not agree")
    K = K1 - 1
    ld = LmheadDesc()
    d = ld.round
    d.B, d.K, d.V = B, K, V
    d.ld_row, d.ld_req, d.dtype = V, K1 * V, F32
    d.accept_mode, d.recover_mode, d.flags = int(accept_mode), int(recover_mode), int(flags)
    _fill_request_arrays(d, inputs, outputs, B, K)
    ld.x_llm, ld.w_llm = xl.data_ptr(), wl.data_ptr()
    ld.x_slm_plus, ld.w_slm_plus = xp.data_ptr(), wp.data_ptr()
    ld.x_slm_minus, ld.w_slm_minus = xm.data_ptr(), wm.data_ptr()
    ld.d_llm, ld.d_slm = dL, dS
    return ld


def _check_topk(desc, topk_idx, topk_val) -> int:
    if topk_idx.dtype != torch.int32 or topk_val.dtype != torch.float32 or topk_idx.shape != topk_val.shape or \
            topk_idx.dim() != 2 or topk_idx.shape[0] != desc.B or not topk_idx.is_contiguous() or \
            not topk_val.is_contiguous():
        raise ValueError("top-k lists must be contiguous [B, k] int32 ids and float32 values")
    return int(topk_idx.shape[1])


class Context:
    """Owns one ``specsteer_ctx`` (device workspace sized for the given maxima)."""

    def __init__(self, max_B: int, max_K: int, max_V: int, device: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("specsteer needs a CUDA device; there is no CPU fallback")
        self._lib = load_library()
        h = C.c_void_p()
        _check(self._lib.specsteer_ctx_create(C.byref(h), int(device), int(max_B), int(max_K), int(max_V)),
               "specsteer_ctx_create")
        self._h = h
        self.device = int(device)

    def close(self):
        if getattr(self, "_h", None):
            self._lib.specsteer_ctx_destroy(self._h)
            self._h = None

    __del__ = close

    def _stream(self, stream):
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        return C.c_void_p(s.cuda_stream)

    def verify_round(self, desc: RoundDesc, stream=None):
        _check(self._lib.specsteer_verify_round(self._h, C.byref(desc), self._stream(stream)), "specsteer_verify_round")

    def recover_sample(self, desc: RoundDesc, stream=None):
        _check(self._lib.specsteer_recover_sample(self._h, C.byref(desc), self._stream(stream)),
               "specsteer_recover_sample")

    def lmhead_round(self, desc: LmheadDesc, stream=None):
        """Verification and recovery with the three LM heads fused in front: no logit tensor is ever stored."""
        _check(self._lib.specsteer_lmhead_round(self._h, C.byref(desc), self._stream(stream)), "specsteer_lmhead_round")

    def lmhead_shard_local(self, desc: LmheadDesc, vocab_offset: int, row_partials: torch.Tensor, stream=None):
        """Step 1 of the fused round with heads split along the vocabulary: this shard's 64-byte partial per row."""
        r = desc.round
        if row_partials.dtype != torch.uint8 or tuple(row_partials.shape) != (r.B, r.K + 1, SHARD_PARTIAL_BYTES) \
                or not row_partials.is_contiguous():
            raise ValueError("row_partials must be a contiguous uint8 tensor [B, K+1, 64]")
        _check(self._lib.specsteer_lmhead_shard_local(self._h, C.byref(desc), int(vocab_offset),
                                                      C.c_void_p(row_partials.data_ptr()), self._stream(stream)),
               "specsteer_lmhead_shard_local")

    def _lmhead_shard_call(self, fn, name, desc, gathered, shard_rank, vocab_offset, vocab_total, stream):
        r = desc.round
        if gathered.dtype != torch.uint8 or gathered.dim() != 4 or not gathered.is_contiguous() or \
                tuple(gathered.shape[1:]) != (r.B, r.K + 1, SHARD_PARTIAL_BYTES):
            raise ValueError("gathered must be a contiguous uint8 tensor [n_shards, B, K+1, 64]")
        _check(fn(self._h, C.byref(desc), C.c_void_p(gathered.data_ptr()), int(gathered.shape[0]), int(shard_rank),
                  int(vocab_offset), int(vocab_total), self._stream(stream)), name)

    def lmhead_shard_combine(self, desc, gathered, shard_rank, vocab_offset, vocab_total, stream=None):
        """Step 3: acceptance from the gathered partials of all shards."""
        self._lmhead_shard_call(self._lib.specsteer_lmhead_shard_combine, "specsteer_lmhead_shard_combine", desc, gathered,
                                shard_rank, vocab_offset, vocab_total, stream)

    def lmhead_shard_recover(self, desc, gathered, shard_rank, vocab_offset, vocab_total, stream=None):
        """Step 4: the shard that holds the CDF target recomputes its chunk and samples."""
        self._lmhead_shard_call(self._lib.specsteer_lmhead_shard_recover, "specsteer_lmhead_shard_recover", desc, gathered,
                                shard_rank, vocab_offset, vocab_total, stream)

    @staticmethod
    def _keys(best_keys: torch.Tensor, B: int):
        if best_keys.dtype != torch.int64 or tuple(best_keys.shape) != (B,) or not best_keys.is_contiguous():
            raise ValueError("best_keys must be a contiguous int64 tensor [B]")
        return C.c_void_p(best_keys.data_ptr())

    def shard_greedy_local(self, desc: RoundDesc, vocab_offset: int, best_keys: torch.Tensor, stream=None):
        """Greedy recovery in the vocabulary-sharded round: this shard's best key per request."""
        _check(self._lib.specsteer_shard_greedy_local(self._h, C.byref(desc), int(vocab_offset), self._keys(best_keys, desc.B),
                                                      self._stream(stream)), "specsteer_shard_greedy_local")

    def lmhead_shard_greedy_local(self, desc: LmheadDesc, best_keys: torch.Tensor, stream=None):
        """The same with the heads split along the vocabulary."""
        _check(self._lib.specsteer_lmhead_shard_greedy_local(self._h, C.byref(desc), self._keys(best_keys, desc.round.B),
                                                             self._stream(stream)), "specsteer_lmhead_shard_greedy_local")

    def shard_greedy_finish(self, desc, best_keys: torch.Tensor, stream=None):
        """Outputs from the keys reduced (MAX) over the shards; desc: a RoundDesc or an LmheadDesc."""
        r = desc.round if isinstance(desc, LmheadDesc) else desc
        _check(self._lib.specsteer_shard_greedy_finish(self._h, C.byref(r), self._keys(best_keys, r.B), self._stream(stream)),
               "specsteer_shard_greedy_finish")

    def cloud_topk(self, desc: RoundDesc, topk_idx: torch.Tensor, topk_val: torch.Tensor, stream=None):
        """Cloud half of the top-k split recovery: fills topk_idx [B, k] int32 and topk_val [B, k] float32."""
        k = _check_topk(desc, topk_idx, topk_val)
        _check(self._lib.specsteer_cloud_topk(self._h, C.byref(desc), k, C.c_void_p(topk_idx.data_ptr()),
                                              C.c_void_p(topk_val.data_ptr()), self._stream(stream)),
               "specsteer_cloud_topk")

    def edge_resample(self, desc: RoundDesc, topk_idx: torch.Tensor, topk_val: torch.Tensor, stream=None):
        """Edge half: samples one token per request among the k kept entries."""
        k = _check_topk(desc, topk_idx, topk_val)
        _check(self._lib.specsteer_edge_resample(self._h, C.byref(desc), k, C.c_void_p(topk_idx.data_ptr()),
                                                 C.c_void_p(topk_val.data_ptr()), self._stream(stream)),
               "specsteer_edge_resample")

    def shard_verify_local(self, desc: RoundDesc, vocab_offset: int, row_partials: torch.Tensor, stream=None):
        """Step 1 of a vocabulary-sharded round: this shard's 64-byte partial per row into row_partials
        (uint8 [B, K+1, 64])."""
        if row_partials.dtype != torch.uint8 or tuple(row_partials.shape) != (desc.B, desc.K + 1, SHARD_PARTIAL_BYTES) \
                or not row_partials.is_contiguous():
            raise ValueError("row_partials must be a contiguous uint8 tensor [B, K+1, 64]")
        _check(self._lib.specsteer_shard_verify_local(self._h, C.byref(desc), int(vocab_offset),
                                                      C.c_void_p(row_partials.data_ptr()), self._stream(stream)),
               "specsteer_shard_verify_local")

    def _shard_call(self, fn, name, desc, gathered, shard_rank, vocab_offset, vocab_total, stream):
        if gathered.dtype != torch.uint8 or gathered.dim() != 4 or not gathered.is_contiguous() or \
                tuple(gathered.shape[1:]) != (desc.B, desc.K + 1, SHARD_PARTIAL_BYTES):
            raise ValueError("gathered must be a contiguous uint8 tensor [n_shards, B, K+1, 64]")
        _check(fn(self._h, C.byref(desc), C.c_void_p(gathered.data_ptr()), int(gathered.shape[0]), int(shard_rank),
                  int(vocab_offset), int(vocab_total), self._stream(stream)), name)

    def shard_verify_combine(self, desc, gathered, shard_rank, vocab_offset, vocab_total, stream=None):
        """Step 3: acceptance from the gathered partials of all shards (same outputs as verify_round)."""
        self._shard_call(self._lib.specsteer_shard_verify_combine, "specsteer_shard_verify_combine", desc, gathered,
                         shard_rank, vocab_offset, vocab_total, stream)

    def shard_recover_local(self, desc, gathered, shard_rank, vocab_offset, vocab_total, stream=None):
        """Step 4: the shard that holds the CDF target samples; the others write values a MAX-reduce ignores."""
        self._shard_call(self._lib.specsteer_shard_recover_local, "specsteer_shard_recover_local", desc, gathered,
                         shard_rank, vocab_offset, vocab_total, stream)

    def round_host(self, desc: RoundDesc, stream=None):
        _check(self._lib.specsteer_round_host(self._h, C.byref(desc), self._stream(stream)), "specsteer_round_host")

    def time_streaming(self, ev_begin=None, ev_end=None):
        """Record two timing-enabled torch.cuda.Event objects around the streaming kernel of every later
        verify_round (None, None switches it off).  The events must have been recorded once already so that
        their CUDA handles exist."""
        a = C.c_void_p(ev_begin.cuda_event) if ev_begin is not None else None
        b = C.c_void_p(ev_end.cuda_event) if ev_end is not None else None
        _check(self._lib.specsteer_ctx_time_streaming(self._h, a, b), "specsteer_ctx_time_streaming")

    def set_wait_limit(self, sm_clocks: int):
        """Give-up limit of the streaming kernel's bounded waits, in SM clocks (0 = the default of a few seconds).
        A test hook: see specsteer_ctx_set_wait_limit."""
        _check(self._lib.specsteer_ctx_set_wait_limit(self._h, int(sm_clocks)), "specsteer_ctx_set_wait_limit")

    def device_error(self) -> int:
        return int(self._lib.specsteer_ctx_device_error(self._h))

    @property
    def workspace_bytes(self) -> int:
        return int(self._lib.specsteer_ctx_workspace_bytes(self._h))

    @property
    def launch_count(self) -> int:
        return int(self._lib.specsteer_ctx_launch_count(self._h))


def probe_ex2(n_ctas: int, iters: int, sink: torch.Tensor, stream=None) -> int:
    """Launch the ex2.approx rate probe (a measurement aid) on the current stream; returns the evaluations it makes."""
    if not torch.cuda.is_available():
        raise RuntimeError("specsteer needs a CUDA device; there is no CPU fallback")
    if sink.dtype != torch.float32 or not sink.is_contiguous() or sink.numel() < n_ctas * 1024:
        raise ValueError("sink must be a contiguous float32 tensor of at least n_ctas * 1024 elements")
    s = stream if stream is not None else torch.cuda.current_stream()
    _check(load_library().specsteer_probe_ex2(int(n_ctas), int(iters), C.c_void_p(sink.data_ptr()), C.c_void_p(s.cuda_stream)),
           "specsteer_probe_ex2")
    return int(n_ctas) * 1024 * 8 * int(iters)


def verify_round_static(desc: RoundDesc, stream=None):
    """Verification through the entry point that allocates nothing (fixed scratch inside the library).

    For hosts that cannot allocate device memory; runs on the current CUDA device and needs no Context.
    Raises SpecSteerError(ERR_STATIC_LIMIT) when the shape does not fit the fixed scratch.
    """
    if not torch.cuda.is_available():
        raise RuntimeError("specsteer needs a CUDA device; there is no CPU fallback")
    s = stream if stream is not None else torch.cuda.current_stream()
    _check(load_library().specsteer_verify_round_static(C.byref(desc), C.c_void_p(s.cuda_stream)),
           "specsteer_verify_round_static")


def verify_recover_round(ctx: Context, inputs, *, accept_mode=ACCEPT_RATIO, recover_mode=RECOVER_STEER, flags=0,
                         V=None, outputs=None, stream=None) -> Dict[str, torch.Tensor]:
    """Convenience: allocate outputs if needed, run verification then recovery on the current stream."""
    hl = inputs["h_llm"]
    if outputs is None:
        outputs = alloc_outputs(hl.shape[0], hl.shape[1] - 1, hl.device)
    desc = make_desc(inputs, outputs, accept_mode=accept_mode, recover_mode=recover_mode, flags=flags, V=V)
    ctx.verify_round(desc, stream)
    ctx.recover_sample(desc, stream)
    return outputs
