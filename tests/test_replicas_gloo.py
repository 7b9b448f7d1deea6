"""The N > 1 path on CPU: two gloo ranks reduce their timings with a max and own disjoint shards."""
import os

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_37852_b200 import replicas


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    times = [10.0 + rank, 5.0 - rank]                      # rank 1 is slower on the first, faster on the second
    red = replicas.max_over_ranks(times)
    b, e = replicas.shard_units(8 * 2, world, rank)        # 2 batches x 8 KV heads
    out[rank] = (red, (b, e))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_max_and_shards():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, 29641, out), nprocs=world, join=True)
    assert out[0][0] == [11.0, 5.0] and out[1][0] == [11.0, 5.0]
    (b0, e0), (b1, e1) = out[0][1], out[1][1]
    assert (b0, e0, b1, e1) == (0, 8, 8, 16)
    assert replicas.aggregate_rate(3.0, 2, 1.5) == 4.0


def test_shard_units_cover_everything_once():
    for n in (1, 7, 16, 33):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                b, e = replicas.shard_units(n, world, r)
                seen += list(range(b, e))
            assert seen == list(range(n))
    with pytest.raises(ValueError):
        replicas.shard_units(4, 2, 2)
    assert replicas.max_over_ranks([1.0, 2.0]) == [1.0, 2.0]   # no process group: identity
