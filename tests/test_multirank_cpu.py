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


class _StubQuantizer:
    """Stands in for LayerQuantizer on a machine without a GPU: records what it was asked to do."""
    log = []

    def __init__(self, d_in, d_out):
        self.shape = (d_in, d_out)

    def run(self, X, W, avg_bits, lloyd_iters):
        assert X.shape[1] == self.shape[0] and tuple(W.shape) == self.shape
        _StubQuantizer.log.append((self.shape, float(W.sum())))
        return {"shape": self.shape, "checksum": float(W.sum())}


def _stack_worker(rank, world, port, out):
    from paper_2410_13056_b200.pipeline import StackQuantizer

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    shapes = [(4, 6), (4, 6), (8, 4), (4, 6), (8, 4)] * 2          # two blocks of five layers
    stack = StackQuantizer(shapes, rank, world, quantizer_factory=_StubQuantizer)

    def inputs_of(k):
        d_in, d_out = shapes[k]
        return torch.zeros(3, d_in), torch.full((d_in, d_out), float(k))

    seen = []
    res = stack.run(inputs_of, 3.0, 5, on_result=lambda k, r: seen.append((k, r["checksum"])))
    total = torch.tensor([float(res["params"])], dtype=torch.float64)
    dist.all_reduce(total)
    out[rank] = (stack.mine, seen, res["layers"], res["params"], float(total.item()), len(stack._quantizers))
    dist.destroy_process_group()


def test_two_ranks_drive_the_stack_quantizer_over_disjoint_layers():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_stack_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    mine0, seen0, n0, p0, total0, nq0 = out[0]
    mine1, seen1, n1, p1, total1, nq1 = out[1]
    assert mine0 == [0, 2, 4, 6, 8] and mine1 == [1, 3, 5, 7, 9]
    assert [k for k, _ in seen0] == mine0 and [k for k, _ in seen1] == mine1     # in order, each once
    shapes = [(4, 6), (4, 6), (8, 4), (4, 6), (8, 4)] * 2
    for k, checksum in seen0 + seen1:                                             # the layer's own weights
        assert checksum == k * shapes[k][0] * shapes[k][1]
    assert (n0, n1) == (5, 5) and p0 + p1 == total0 == total1 == sum(a * b for a, b in shapes)
    assert nq0 == 2 and nq1 == 2                                                  # one quantizer per shape


def test_single_process_helpers():
    assert sharding.layers_of_rank(5, 0, 1) == [0, 1, 2, 3, 4]
    assert sharding.layers_of_rank(2, 3, 4) == []
    assert sharding.max_over_ranks(3.5) == 3.5
    with pytest.raises(ValueError):
        sharding.layers_of_rank(5, 2, 2)
