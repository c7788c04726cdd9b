"""Seeded synthetic inputs for one SpecSteer verify/recover round.

This module only manufactures inputs: logit tensors shaped like the paper's
workloads (Qwen-size and Llama-3-size vocabularies, draft horizon K, per-request
lambda / beta / temperature), drafted tokens and the uniforms the round
consumes.  It contains none of the verification or recovery arithmetic and is
imported by neither the CUDA binding nor the CPU oracle; tests and the
benchmark feed the same tensors to both.

Recipe (per vocabulary row):
  generalist   G(v) = g * z_v - s * ln(rank_pi(v)),   z ~ N(0,1) (or 3 * Student-t(3)),
               pi a fresh uniform permutation of the vocabulary, g = 2, s = 1.1
  specialist+  P = G + sigma_plus  * N(0,1)
  specialist-  M = G + sigma_minus * N(0,1),  sigma_minus = sigma_plus / 2
Logits are rounded to the storage dtype first; drafted tokens are then sampled
from Softmax(P / T) of the rounded values (the drafting step, Eq. 5).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Sequence, Tuple

import torch

ZIPF_S = 1.1
GAUSS_G = 2.0
SLAB_ROWS = 32  # rows generated at a time (bounds temporary memory); part of the recipe


@dataclasses.dataclass(frozen=True)
class RoundSpec:
    name: str
    B: int
    K: int
    V: int
    dtype: str = "f32"                        # "f32" | "bf16"
    sigma_plus: Tuple[Tuple[float, float], ...] = ((1.0, 1.0),)   # (fraction of requests, sigma+) blocks, in order
    heavy_tail: bool = False                  # generalist noise 3 * Student-t(nu=3) instead of 2 * N(0,1)
    ragged: bool = False                      # draft_len uniform in [1, K] instead of K
    beta_choices: Tuple[float, ...] = (1.0,)  # per-request uniform choice
    beta_uniform: Tuple[float, float] = None  # or U(lo, hi)
    temp_choices: Tuple[float, ...] = (1.0,)
    lam: float = 0.5

    @property
    def rows(self) -> int:
        return self.B * (self.K + 1)

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def logit_bytes(self, rows: int) -> int:
        return 3 * rows * self.V * self.elem_bytes


# The five benchmark configurations.
CONFIGS: Sequence[RoundSpec] = (
    RoundSpec("cfg0_B1_K4_V32000_f32", 1, 4, 32000, "f32"),
    RoundSpec("cfg1_B16_K5_V128256_bf16", 16, 5, 128256, "bf16", sigma_plus=((1.0, 1.5),),
              beta_choices=(0.5, 1.0, 2.0), temp_choices=(0.7,)),
    RoundSpec("cfg2_B64_K8_V151936_bf16_ragged", 64, 8, 151936, "bf16", ragged=True),
    RoundSpec("cfg3_B256_K4_V151936_f32", 256, 4, 151936, "f32", sigma_plus=((0.5, 0.3), (0.5, 3.0))),
    RoundSpec("cfg4_B512_K6_V256000_bf16", 512, 6, 256000, "bf16", heavy_tail=True,
              beta_uniform=(0.0, 3.0), temp_choices=(0.3, 1.0, 1.5)),
)


def _torch_dtype(spec: RoundSpec):
    return torch.float32 if spec.dtype == "f32" else torch.bfloat16


def _sigma_per_request(spec: RoundSpec) -> torch.Tensor:
    out = torch.empty(spec.B, dtype=torch.float32)
    start = 0
    for i, (frac, s) in enumerate(spec.sigma_plus):
        end = spec.B if i == len(spec.sigma_plus) - 1 else min(spec.B, start + int(round(frac * spec.B)))
        out[start:end] = s
        start = end
    return out


def make_round(spec: RoundSpec, device="cpu", seed: int = 0) -> Dict[str, torch.Tensor]:
    """All inputs of one round, on ``device``, deterministic for (spec, seed, device type)."""
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    B, K, V = spec.B, spec.K, spec.V
    K1 = K + 1
    dt = _torch_dtype(spec)

    # per-request parameters first (tiny), so that the drafting temperature is known per slab
    cgen = torch.Generator(device="cpu")
    cgen.manual_seed(seed + 1)
    if spec.beta_uniform is not None:
        lo, hi = spec.beta_uniform
        beta = lo + (hi - lo) * torch.rand(B, generator=cgen)
    else:
        beta = torch.tensor(spec.beta_choices)[torch.randint(len(spec.beta_choices), (B,), generator=cgen)]
    temp = torch.tensor(spec.temp_choices)[torch.randint(len(spec.temp_choices), (B,), generator=cgen)]
    lam = torch.full((B,), spec.lam)
    if spec.ragged:
        draft_len = torch.randint(1, K + 1, (B,), generator=cgen, dtype=torch.int32)
    else:
        draft_len = torch.full((B,), K, dtype=torch.int32)
    u_accept = torch.rand(B, K, generator=cgen, dtype=torch.float32)
    u_recover = torch.rand(B, generator=cgen, dtype=torch.float32)
    sigma = _sigma_per_request(spec)

    h_llm = torch.empty(B, K1, V, dtype=dt, device=dev)
    h_plus = torch.empty_like(h_llm)
    h_minus = torch.empty_like(h_llm)
    draft = torch.zeros(B, K, dtype=torch.int32, device=dev)

    rows = B * K1
    fl, fp, fm = h_llm.view(rows, V), h_plus.view(rows, V), h_minus.view(rows, V)
    sig_row = sigma.repeat_interleave(K1).to(dev)
    temp_row = temp.repeat_interleave(K1).to(dev)
    tok_row = torch.zeros(rows, dtype=torch.int64, device=dev)
    for r0 in range(0, rows, SLAB_ROWS):
        r1 = min(rows, r0 + SLAB_ROWS)
        n = r1 - r0
        z = torch.randn(n, V, generator=gen, device=dev, dtype=torch.float32)
        if spec.heavy_tail:
            chi = torch.randn(n, V, 3, generator=gen, device=dev, dtype=torch.float32).square_().sum(-1)
            z = 3.0 * z / torch.sqrt(chi / 3.0)
            del chi
        else:
            z = GAUSS_G * z
        rank = torch.argsort(torch.rand(n, V, generator=gen, device=dev), dim=1).to(torch.float32) + 1.0
        G = z - ZIPF_S * torch.log(rank)
        del z, rank
        sp = sig_row[r0:r1, None]
        P = G + sp * torch.randn(n, V, generator=gen, device=dev, dtype=torch.float32)
        M = G + (0.5 * sp) * torch.randn(n, V, generator=gen, device=dev, dtype=torch.float32)
        fl[r0:r1] = G.to(dt)
        fp[r0:r1] = P.to(dt)
        fm[r0:r1] = M.to(dt)
        del G, P, M
        q = torch.softmax(fp[r0:r1].to(torch.float64) / temp_row[r0:r1, None].to(torch.float64), dim=1)
        tok_row[r0:r1] = torch.multinomial(q, 1, generator=gen).squeeze(1)
        del q
    draft.copy_(tok_row.view(B, K1)[:, :K].to(torch.int32))

    return {
        "h_llm": h_llm, "h_slm_plus": h_plus, "h_slm_minus": h_minus,
        "draft_tokens": draft, "draft_len": draft_len.to(dev),
        "lam": lam.to(dev), "beta": beta.to(torch.float32).to(dev), "temperature": temp.to(torch.float32).to(dev),
        "u_accept": u_accept.to(dev), "u_recover": u_recover.to(dev),
    }


def make_lmhead_round(spec: RoundSpec, d_llm: int, d_slm: int, device="cpu", seed: int = 0) -> Dict[str, torch.Tensor]:
    """Inputs of one round on hidden states and LM heads instead of logits (bf16), deterministic for
    (spec, d_llm, d_slm, seed, device type); needs d_slm < d_llm.

    The three logit tensors x W^T have the structure of ``make_round``'s: the Specialist's head is the first d_slm
    columns of the Generalist's, the Generalist's hidden state is the Specialist's clean state s followed by extra
    dimensions, and the Specialist's two states are s plus noise (twice as much with the context as without).  The
    first hidden dimension is the constant 1 and carries a per-token bias with the Zipf profile over one random
    permutation of the vocabulary.  Draft tokens are sampled from Softmax(h_SLM+ / T) formed with a float32 product.
    """
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    cgen = torch.Generator(device="cpu")
    cgen.manual_seed(seed + 1)
    B, K, V = spec.B, spec.K, spec.V
    K1 = K + 1
    if spec.beta_uniform is not None:
        lo, hi = spec.beta_uniform
        beta = lo + (hi - lo) * torch.rand(B, generator=cgen)
    else:
        beta = torch.tensor(spec.beta_choices)[torch.randint(len(spec.beta_choices), (B,), generator=cgen)]
    temp = torch.tensor(spec.temp_choices)[torch.randint(len(spec.temp_choices), (B,), generator=cgen)]
    lam = torch.full((B,), spec.lam)
    if spec.ragged:
        draft_len = torch.randint(1, K + 1, (B,), generator=cgen, dtype=torch.int32)
    else:
        draft_len = torch.full((B,), K, dtype=torch.int32)
    u_accept = torch.rand(B, K, generator=cgen, dtype=torch.float32)
    u_recover = torch.rand(B, generator=cgen, dtype=torch.float32)
    sigma = _sigma_per_request(spec).to(dev)          # noise of h_SLM+ in logit units; h_SLM- gets half

    # heads: entries N(0, g^2 / d_slm) on the shared columns, so that s W^T has standard deviation g for |s_i| ~ 1
    w_llm = torch.randn(V, d_llm, generator=gen, device=dev) * (GAUSS_G / d_slm ** 0.5)
    w_llm[:, d_slm:] *= 0.3 * (d_slm / max(1, d_llm - d_slm)) ** 0.5   # the extra dimensions add a tenth of the variance
    rank = torch.argsort(torch.rand(V, generator=gen, device=dev)).to(torch.float32) + 1.0
    w_llm[:, 0] = -ZIPF_S * torch.log(rank)
    w_llm = w_llm.to(torch.bfloat16)
    w_slm = w_llm[:, :d_slm].contiguous()
    s = torch.randn(B, K1, d_slm, generator=gen, device=dev)
    s[..., 0] = 1.0
    extra = torch.randn(B, K1, d_llm - d_slm, generator=gen, device=dev)
    x_llm = torch.cat([s, extra], dim=2).to(torch.bfloat16)
    sg = (sigma / GAUSS_G)[:, None, None]
    x_plus = s + sg * torch.randn(B, K1, d_slm, generator=gen, device=dev)
    x_minus = s + 0.5 * sg * torch.randn(B, K1, d_slm, generator=gen, device=dev)
    x_plus[..., 0] = 1.0
    x_minus[..., 0] = 1.0
    x_plus, x_minus = x_plus.to(torch.bfloat16), x_minus.to(torch.bfloat16)

    draft = torch.zeros(B, K, dtype=torch.int32, device=dev)
    wf = w_slm.to(torch.float32)
    for b0 in range(0, B, 32):
        b1 = min(B, b0 + 32)
        hp = torch.matmul(x_plus[b0:b1, :K].to(torch.float32), wf.t())
        q = torch.softmax(hp.to(torch.float64) / temp[b0:b1, None, None].to(dev).to(torch.float64), dim=2)
        if K > 0:
            draft[b0:b1] = torch.multinomial(q.view(-1, V), 1, generator=gen).view(b1 - b0, K).to(torch.int32)
        del hp, q
    return {
        "x_llm": x_llm, "w_llm": w_llm, "x_slm_plus": x_plus, "w_slm_plus": w_slm, "x_slm_minus": x_minus,
        "w_slm_minus": w_slm,
        "draft_tokens": draft, "draft_len": draft_len.to(dev),
        "lam": lam.to(dev), "beta": beta.to(torch.float32).to(dev), "temperature": temp.to(torch.float32).to(dev),
        "u_accept": u_accept.to(dev), "u_recover": u_recover.to(dev),
    }


def used_rows(spec: RoundSpec, draft_len: torch.Tensor, bonus: bool) -> int:
    """Rows the round must read: the drafted rows plus, with the bonus flag, the row after them."""
    return int(draft_len.to(torch.int64).sum().item()) + (spec.B if bonus else 0)


def to_numpy_bits(t: torch.Tensor):
    """Host numpy view of a logit tensor: float32 as is, bf16 as uint16 bit patterns."""
    import numpy as np
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()
