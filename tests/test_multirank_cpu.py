"""The N > 1 path on CPU: two gloo ranks shard layers round-robin, agree on the slowest rank's time
and on the aggregate throughput.  (The data path itself has no collective.)"""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2410_13056_b200 import sharding


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = sharding.layers_of_rank(7, rank, world)
    fake_seconds = 1.0 + rank          # rank 1 is the slower one
    slowest = sharding.max_over_ranks(fake_seconds)
    counts = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
    dist.all_gather(counts, torch.tensor([len(mine)], dtype=torch.int64))
    dist.barrier()
    out[rank] = (mine, slowest, [int(c.item()) for c in counts])
    dist.destroy_process_group()


def test_two_ranks_shard_layers_and_agree_on_time():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    assert out[0][0] == [0, 2, 4, 6] and out[1][0] == [1, 3, 5]
    assert sorted(out[0][0] + out[1][0]) == list(range(7))           # every layer exactly once
    assert out[0][1] == out[1][1] == 2.0                              # max over ranks
    assert out[0][2] == out[1][2] == [4, 3]
    assert sharding.aggregate_throughput([4 * 10.0, 3 * 10.0], out[0][1]) == 35.0


def test_single_process_helpers():
    assert sharding.layers_of_rank(5, 0, 1) == [0, 1, 2, 3, 4]
    assert sharding.layers_of_rank(2, 3, 4) == []
    assert sharding.max_over_ranks(3.5) == 3.5
    with pytest.raises(ValueError):
        sharding.layers_of_rank(5, 2, 2)
