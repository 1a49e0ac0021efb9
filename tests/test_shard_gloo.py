"""Multi-rank host logic on CPU: two gloo ranks shard a batch, and the reductions used for
reporting (slowest rank, total units) agree on every rank."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2603_12617_b200 import shard


@pytest.mark.parametrize("B,world", [(256, 1), (256, 2), (7, 2), (5, 4), (3, 8), (0, 2)])
def test_shard_ranges_tile_the_batch(B, world):
    ranges = [shard.shard_range(B, r, world) for r in range(world)]
    assert ranges[0][0] == 0 and ranges[-1][1] == B
    for (a0, a1), (b0, b1) in zip(ranges, ranges[1:]):
        assert a1 == b0
    sizes = [b - a for a, b in ranges]
    assert max(sizes) - min(sizes) <= 1


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, B, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        b0, b1 = shard.shard_range(B, rank, world)
        # every rank learns every range and checks the tiling
        mine = torch.tensor([b0, b1], dtype=torch.int64)
        got = [torch.zeros(2, dtype=torch.int64) for _ in range(world)]
        dist.all_gather(got, mine)
        ok = got[0][0].item() == 0 and got[-1][1].item() == B and all(
            got[i][1].item() == got[i + 1][0].item() for i in range(world - 1))
        slowest = shard.max_over_ranks(10.0 + rank)
        total = shard.sum_over_ranks(float(b1 - b0))
        q.put((rank, ok, slowest, total))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_agree():
    world, B = 2, 37
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, B, q)) for r in range(world)]
    for p in procs:
        p.start()
    results = [q.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ok, slowest, total in results:
        assert ok
        assert slowest == 10.0 + (world - 1)
        assert total == float(B)
