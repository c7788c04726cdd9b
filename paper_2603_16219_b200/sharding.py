"""Host-side helpers for running rounds on several GPUs.

Requests of a round are independent, so the path shards by request: every rank verifies its own
contiguous block and no collective touches the logits.  These helpers hold the shard arithmetic and the
two tiny collectives a job needs around the kernels (gathering per-request results, and the
max-over-ranks of a timing).  They work with any torch.distributed backend (NCCL on GPUs, gloo in tests).
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
