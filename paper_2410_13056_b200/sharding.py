"""Multi-GPU plumbing: the pass shards by layer, with no collective on the data path.

Every linear layer is quantized independently of every other (Section 3.2.1 of the paper works
layer by layer), so N ranks simply take different layers.  torch.distributed is used only to agree
on timings: a barrier around the timed region and the maximum over ranks of the measured time.
"""
from typing import List, Sequence

import torch
import torch.distributed as dist


def layers_of_rank(n_layers: int, rank: int, world: int) -> List[int]:
    """Round-robin assignment of layer indices to ranks."""
    if world < 1 or not (0 <= rank < world):
        raise ValueError("bad rank/world")
    return list(range(rank, n_layers, world))


def max_over_ranks(value: float, device="cpu") -> float:
    """Largest `value` of any rank (the job is as slow as its slowest rank)."""
    if not dist.is_available() or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: Sequence[float], seconds: float) -> float:
    """Whole-job throughput: all units processed by all ranks over the slowest rank's time."""
    return float(sum(units_per_rank)) / seconds
