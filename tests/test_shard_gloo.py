"""The multi-rank host logic on CPU: batch sharding covers the batch exactly once, and the time
reduction takes the maximum over ranks (world size 2, gloo)."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2510_05688_b200.shard import max_over_ranks, shard_batch


def test_shard_batch_partitions_exactly():
    for batch in (0, 1, 7, 8, 32, 33):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                lo, hi = shard_batch(batch, r, world)
                assert 0 <= lo <= hi <= batch
                seen += list(range(lo, hi))
            assert seen == list(range(batch))
            sizes = [shard_batch(batch, r, world)[1] - shard_batch(batch, r, world)[0] for r in range(world)]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard_batch(4, 2, 2)


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    got = max_over_ranks(1.5 + rank, world)
    lo, hi = shard_batch(5, rank, world)
    rows = torch.zeros(5)
    rows[lo:hi] = 1
    dist.all_reduce(rows)
    q.put((rank, got, rows.tolist()))
    dist.destroy_process_group()


def test_max_over_ranks_world2_gloo():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, rows in res:
        assert got == 2.5                      # the slower rank's time
        assert rows == [1.0] * 5               # every batch row owned by exactly one rank
    assert max_over_ranks(3.25, 1) == 3.25
