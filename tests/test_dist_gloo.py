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


def _vocab_worker(rank, world, port, q):
    import torch.distributed as dist
    from paper_2603_16219_b200 import sharding
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % port, rank=rank, world_size=world)
    try:
        B, K1 = 3, 4
        parts = torch.full((B, K1, 64), rank + 1, dtype=torch.uint8)
        parts[:, :, 0] = torch.arange(B * K1, dtype=torch.uint8).reshape(B, K1)
        gathered = sharding.gather_partials(parts, dist)
        ok = tuple(gathered.shape) == (world, B, K1, 64)
        for r in range(world):                                  # rank-major, every rank sees the same thing
            ok = ok and bool((gathered[r, :, :, 1:] == r + 1).all()) and bool((gathered[r, :, :, 0] == parts[:, :, 0]).all())
        # the owner of each request's target fills the results, the others leave -1 / -inf / the accepted length
        outs = {"rec_token": torch.tensor([7 if rank == 0 else -1, 9 if rank == 1 else -1, -1], dtype=torch.int32),
                "rec_logprob": torch.tensor([-0.5 if rank == 0 else float("-inf"), -2.0 if rank == 1 else float("-inf"),
                                             float("-inf")]),
                "out_tokens": torch.tensor([[3, 7 if rank == 0 else -1], [9 if rank == 1 else -1, -1], [-1, -1]], dtype=torch.int32),
                "n_out": torch.tensor([2 if rank == 0 else 1, 1 if rank == 1 else 0, 0], dtype=torch.int32)}
        sharding.reduce_recovered(outs, dist)
        ok = ok and outs["rec_token"].tolist() == [7, 9, -1] and outs["n_out"].tolist() == [2, 1, 0]
        ok = ok and outs["out_tokens"].tolist() == [[3, 7], [9, -1], [-1, -1]]
        ok = ok and outs["rec_logprob"][:2].tolist() == [-0.5, -2.0]
        q.put((rank, ok))
    finally:
        dist.destroy_process_group()


def test_vocab_shard_collectives_on_two_ranks():
    """The two collectives of the vocabulary-sharded round (all-gather of row partials, MAX all-reduce of results)."""
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_vocab_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
    assert res == [(0, True), (1, True)]


def test_vocab_range_covers_every_id_once():
    from paper_2603_16219_b200 import sharding
    for V, world, align in ((151936, 8, 8), (4096, 7, 1024), (10, 4, 8), (128256, 3, 8), (5, 2, 1)):
        spans = [sharding.vocab_range(V, r, world, align) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == V
        assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
        assert all(lo % align == 0 for lo, hi in spans if hi > lo)


class _FakeShardCtx:
    """Stands in for the CUDA context in the sharded-round helpers: records the order of the calls and plays the
    kernels' part on CPU tensors (rank r's partial is filled with r + 1; rank 0 owns the targets)."""

    def __init__(self, rank, outputs, prefix):
        self.rank, self.outputs, self.prefix, self.calls = rank, outputs, prefix, []

    def _local(self, desc, vocab_offset, parts, stream=None):
        self.calls.append(("local", vocab_offset))
        parts.fill_(self.rank + 1)

    def _combine(self, desc, gathered, rank, vocab_offset, vocab_total, stream=None):
        self.calls.append(("combine", rank, vocab_offset, vocab_total, tuple(gathered.shape)))
        self.outputs["accept_len"].fill_(int(gathered[:, 0, 0, 0].sum()))     # the same on every rank

    def _recover(self, desc, gathered, rank, vocab_offset, vocab_total, stream=None):
        self.calls.append(("recover", rank))
        own = rank == 0
        self.outputs["rec_token"].fill_(11 if own else -1)
        self.outputs["rec_logprob"].fill_(-1.5 if own else float("-inf"))
        self.outputs["out_tokens"].fill_(11 if own else -1)
        self.outputs["n_out"].fill_(1 if own else 0)

    _NAMES = {"shard_verify_local": "_local", "shard_verify_combine": "_combine", "shard_recover_local": "_recover",
              "lmhead_shard_local": "_local", "lmhead_shard_combine": "_combine", "lmhead_shard_recover": "_recover"}

    def shard_greedy_local(self, desc, vocab_offset, keys, stream=None):
        self.calls.append(("greedy_local", vocab_offset))
        keys.copy_(torch.tensor([100 + self.rank, 7 - self.rank], dtype=torch.int64))   # rank 1 wins request 0, rank 0 request 1

    def lmhead_shard_greedy_local(self, desc, keys, stream=None):
        self.shard_greedy_local(desc, None, keys)

    def shard_greedy_finish(self, desc, keys, stream=None):
        self.calls.append(("greedy_finish", keys.tolist()))

    def __getattr__(self, name):
        if name in self._NAMES and name.startswith(self.prefix):
            return getattr(self, self._NAMES[name])
        raise AttributeError(name)


def _round_worker(rank, world, port, q):
    import types
    import torch.distributed as dist
    from paper_2603_16219_b200 import sharding
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % port, rank=rank, world_size=world)
    try:
        ok = True
        for helper, prefix, desc in (
                (sharding.sharded_vocab_round, "shard", types.SimpleNamespace(B=2, K=3)),
                (sharding.sharded_lmhead_round, "lmhead_shard", types.SimpleNamespace(round=types.SimpleNamespace(B=2, K=3)))):
            outs = {"accept_len": torch.zeros(2, dtype=torch.int32), "rec_token": torch.zeros(2, dtype=torch.int32),
                    "rec_logprob": torch.zeros(2), "out_tokens": torch.zeros(2, 4, dtype=torch.int32),
                    "n_out": torch.zeros(2, dtype=torch.int32)}
            fake = _FakeShardCtx(rank, outs, prefix)
            gathered = helper(fake, desc, outs, 100 * rank, 200, dist)
            ok = ok and tuple(gathered.shape) == (world, 2, 4, 64) and [c[0] for c in fake.calls] == ["local", "combine", "recover"]
            ok = ok and fake.calls[0][1] == 100 * rank and fake.calls[1][1:4] == (rank, 100 * rank, 200)
            ok = ok and outs["accept_len"].tolist() == [3, 3]            # partials of rank 0 (1) and rank 1 (2)
            ok = ok and outs["rec_token"].tolist() == [11, 11] and outs["n_out"].tolist() == [1, 1]
            ok = ok and outs["rec_logprob"].tolist() == [-1.5, -1.5] and bool((outs["out_tokens"] == 11).all())
        # greedy rounds: local keys, their MAX over the ranks, the common last step
        for helper, prefix, desc in (
                (sharding.sharded_vocab_round, "shard", types.SimpleNamespace(B=2, K=3, recover_mode=2)),
                (sharding.sharded_lmhead_round, "lmhead_shard",
                 types.SimpleNamespace(round=types.SimpleNamespace(B=2, K=3, recover_mode=2)))):
            outs = {"accept_len": torch.zeros(2, dtype=torch.int32)}
            fake = _FakeShardCtx(rank, outs, prefix)
            helper(fake, desc, outs, 100 * rank, 200, dist)
            ok = ok and [c[0] for c in fake.calls] == ["local", "combine", "greedy_local", "greedy_finish"]
            ok = ok and fake.calls[-1][1] == [101, 7]
        q.put((rank, ok))
    finally:
        dist.destroy_process_group()


def test_sharded_round_helpers_call_order_and_collectives_on_two_ranks():
    """Both sharded rounds (logit shards, fused LM-head shards): local pass, all-gather, combine, recover, MAX
    all-reduce - with the kernels replaced by a stand-in, on two gloo ranks."""
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_round_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
    assert res == [(0, True), (1, True)]
