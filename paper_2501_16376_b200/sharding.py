"""Multi-GPU host logic.  The pruning pass shards without any data-path exchange: rows, layers
and whole models are independent problems (the paper prunes every row on its own), so each rank
works on its own units and the only communication is the reduction of the timing."""
from __future__ import annotations

import torch
import torch.distributed as dist


def unit_of_rank(rank: int, world: int) -> int:
    """Weak scaling: rank r owns model number r (used as a seed offset)."""
    if not 0 <= rank < max(world, 1):
        raise ValueError("rank out of range")
    return rank


def assign_units(n_units: int, world: int, rank: int) -> range:
    """Strong-scaling split of n_units independent units (blocks, layers) into contiguous,
    balanced shares: the first n_units % world ranks get one extra unit."""
    if world < 1 or not 0 <= rank < world or n_units < 0:
        raise ValueError("bad partition arguments")
    base, extra = divmod(n_units, world)
    begin = rank * base + min(rank, extra)
    return range(begin, begin + base + (1 if rank < extra else 0))


def max_over_ranks(value: float, world: int, device=None) -> float:
    """Max of a per-rank number (the step time) over the process group."""
    if world <= 1 or not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64,
                     device=device if dist.get_backend() == "nccl" else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, world: int, device=None) -> float:
    if world <= 1 or not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64,
                     device=device if dist.get_backend() == "nccl" else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
