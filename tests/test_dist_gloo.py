"""The multi-GPU host logic on two gloo ranks (CPU): request sharding, result gathering, max-over-ranks."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, B, K, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2603_16219_b200 import sharding
        lo, hi = sharding.request_range(B, rank, world)
        ids = torch.arange(lo, hi)
        local = {"accept_len": (ids % (K + 1)).to(torch.int32),
                 "out_tokens": (ids[:, None] * 10 + torch.arange(K + 1)[None, :]).to(torch.int32),
                 "rec_logprob": -ids.to(torch.float32)}
        full = sharding.gather_by_request(local, B, dist)
        slow = sharding.max_over_ranks(1.0 + rank, "cpu", dist)
        ok = (torch.equal(full["accept_len"], (torch.arange(B) % (K + 1)).to(torch.int32))
              and torch.equal(full["out_tokens"][:, 1], (torch.arange(B) * 10 + 1).to(torch.int32))
              and torch.equal(full["rec_logprob"], -torch.arange(B, dtype=torch.float32))
              and slow == float(world))
        q.put((rank, bool(ok), (lo, hi)))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("B", [7, 8, 1])
def test_request_sharding_and_gather_on_two_ranks(B):
    world, K = 2, 3
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, B, K, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert all(ok for _, ok, _ in res)
    assert res[0][2][0] == 0 and res[0][2][1] == res[1][2][0] and res[1][2][1] == B


def test_request_range_covers_every_request_once():
    from paper_2603_16219_b200 import sharding
    for B in (0, 1, 5, 256, 1000):
        for world in (1, 2, 3, 8):
            got = []
            for r in range(world):
                lo, hi = sharding.request_range(B, r, world)
                got += list(range(lo, hi))
            assert got == list(range(B))
    with pytest.raises(ValueError):
        sharding.request_range(4, 2, 2)
