"""Host-side helpers for running rounds on several GPUs.

Requests of a round are independent, so the path shards by request: every rank verifies its own
contiguous block and no collective touches the logits.  These helpers hold the shard arithmetic and the
two tiny collectives a job needs around the kernels (gathering per-request results, and the
max-over-ranks of a timing).  They work with any torch.distributed backend (NCCL on GPUs, gloo in tests).

When the logits arrive split along the vocabulary instead (a tensor-parallel LM head), `sharded_vocab_round`
runs the round with one exchange step: an all-gather of 64 bytes per row and rank, and a MAX all-reduce of the
per-request results.  The arithmetic stays in the library's kernels; only the two collectives live here.
"""
from __future__ import annotations

from typing import Dict, Tuple

import torch


def request_range(B: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous block [lo, hi) of the B requests owned by `rank`; sizes differ by at most one."""
    if world <= 0 or not (0 <= rank < world) or B < 0:
        raise ValueError("bad shard arguments")
    base, rem = divmod(B, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def gather_by_request(local: Dict[str, torch.Tensor], B: int, dist) -> Dict[str, torch.Tensor]:
    """All-gather per-request outputs (first axis = this rank's requests) into full-batch tensors."""
    world, rank = dist.get_world_size(), dist.get_rank()
    sizes = [request_range(B, r, world) for r in range(world)]
    pad = max(hi - lo for lo, hi in sizes)
    out = {}
    for name, t in local.items():
        lo, hi = sizes[rank]
        if t.shape[0] != hi - lo:
            raise ValueError("%s: first axis %d is not this rank's %d requests" % (name, t.shape[0], hi - lo))
        buf = torch.zeros((pad,) + tuple(t.shape[1:]), dtype=t.dtype, device=t.device)
        buf[: hi - lo] = t
        parts = [torch.empty_like(buf) for _ in range(world)]
        dist.all_gather(parts, buf)
        out[name] = torch.cat([parts[r][: sizes[r][1] - sizes[r][0]] for r in range(world)], 0)
    return out


def max_over_ranks(value: float, device, dist) -> float:
    """The slowest rank's time: what a multi-GPU throughput figure has to be divided by."""
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def vocab_range(V: int, rank: int, world: int, align: int = 8) -> Tuple[int, int]:
    """Contiguous block [lo, hi) of the V token ids owned by `rank`: equal blocks rounded up to `align` ids
    (16-byte rows for 16-bit logits), the last rank taking what is left."""
    if world <= 0 or not (0 <= rank < world) or V < 0 or align <= 0:
        raise ValueError("bad shard arguments")
    per = -(-V // world)
    per = -(-per // align) * align
    lo = min(rank * per, V)
    return lo, min(lo + per, V)


def gather_partials(row_partials: torch.Tensor, dist) -> torch.Tensor:
    """All-gather the [B, K+1, 64] uint8 partials of every rank into [world, B, K+1, 64], rank-major."""
    world = dist.get_world_size()
    out = torch.empty((world,) + tuple(row_partials.shape), dtype=row_partials.dtype, device=row_partials.device)
    dist.all_gather(list(out.unbind(0)), row_partials.contiguous())
    return out


def reduce_recovered(outputs: Dict[str, torch.Tensor], dist) -> None:
    """Element-wise MAX over ranks of the four arrays the owning shard fills (in place)."""
    for name in ("rec_token", "rec_logprob", "out_tokens", "n_out"):
        t = outputs.get(name)
        if t is not None:
            dist.all_reduce(t, op=dist.ReduceOp.MAX)


def reduce_keys(best_keys: torch.Tensor, dist) -> None:
    """Element-wise MAX over ranks of the shards' best keys of a greedy round (int64 [B], in place)."""
    dist.all_reduce(best_keys, op=dist.ReduceOp.MAX)


def sharded_vocab_round(ctx, desc, outputs: Dict[str, torch.Tensor], vocab_offset: int, vocab_total: int, dist,
                        stream=None) -> torch.Tensor:
    """One verify + recover round over a vocabulary split across the ranks of `dist`.

    `desc` describes this rank's shard (V = local width; draft_tokens hold global ids) and points at `outputs`.
    Returns the gathered partials.  Every rank ends with identical outputs.
    """
    rank = dist.get_rank()
    parts = torch.empty((desc.B, desc.K + 1, 64), dtype=torch.uint8, device=outputs["accept_len"].device)
    ctx.shard_verify_local(desc, vocab_offset, parts, stream)
    gathered = gather_partials(parts, dist)
    ctx.shard_verify_combine(desc, gathered, rank, vocab_offset, vocab_total, stream)
    if getattr(desc, "recover_mode", 0) == 2:     # greedy: every shard's best key, MAX over shards, then the outputs
        keys = torch.empty(desc.B, dtype=torch.int64, device=outputs["accept_len"].device)
        ctx.shard_greedy_local(desc, vocab_offset, keys, stream)
        reduce_keys(keys, dist)
        ctx.shard_greedy_finish(desc, keys, stream)
        return gathered
    ctx.shard_recover_local(desc, gathered, rank, vocab_offset, vocab_total, stream)
    reduce_recovered(outputs, dist)
    return gathered


def sharded_lmhead_round(ctx, desc, outputs: Dict[str, torch.Tensor], vocab_offset: int, vocab_total: int, dist,
                         stream=None) -> torch.Tensor:
    """One verify + recover round on hidden states and heads whose rows (the vocabulary) are split across the ranks
    of `dist`: `desc` (an LM-head descriptor) describes this rank's rows of the heads (round.V = local count;
    draft_tokens hold global ids) and points at `outputs`.  Same collectives as `sharded_vocab_round`; every rank
    ends with identical outputs.  Returns the gathered partials."""
    rank = dist.get_rank()
    r = desc.round
    parts = torch.empty((r.B, r.K + 1, 64), dtype=torch.uint8, device=outputs["accept_len"].device)
    ctx.lmhead_shard_local(desc, vocab_offset, parts, stream)
    gathered = gather_partials(parts, dist)
    ctx.lmhead_shard_combine(desc, gathered, rank, vocab_offset, vocab_total, stream)
    if getattr(r, "recover_mode", 0) == 2:
        keys = torch.empty(r.B, dtype=torch.int64, device=outputs["accept_len"].device)
        ctx.lmhead_shard_greedy_local(desc, keys, stream)
        reduce_keys(keys, dist)
        ctx.shard_greedy_finish(desc, keys, stream)
        return gathered
    ctx.lmhead_shard_recover(desc, gathered, rank, vocab_offset, vocab_total, stream)
    reduce_recovered(outputs, dist)
    return gathered
