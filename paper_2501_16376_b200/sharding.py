"""Multi-GPU host logic.  The pruning pass shards without any data-path exchange: rows, layers
and whole models are independent problems (the paper prunes every row on its own), so each rank
works on its own units and the only communication is the reduction of the timing.

One optional exchange exists: when the calibration TOKENS of one layer input are split over
ranks, the per-channel sums of squares are additive, so one all-reduce of d_in doubles (plus the
token count) gives every rank the statistics of all tokens (``allreduce_colsq``,
``merge_calibration``)."""
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


def token_share(n_tokens: int, world: int, rank: int, align: int = 1) -> range:
    """Token-sharded calibration: the contiguous share of the calibration tokens that `rank`
    accumulates; shares are balanced in units of `align` tokens (e.g. one sequence)."""
    if align < 1 or n_tokens < 0:
        raise ValueError("bad partition arguments")
    units = assign_units((n_tokens + align - 1) // align, world, rank)
    return range(min(units.start * align, n_tokens), min(units.stop * align, n_tokens))


def row_share(n_rows: int, world: int, rank: int) -> range:
    """Row-sharded selection: the contiguous rows of a layer that `rank` prunes (rows are
    independent problems: the row loop of Algorithm 1 is parallel)."""
    return assign_units(n_rows, world, rank)


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


def allreduce_colsq(colsq: torch.Tensor, n_tokens: int, world: int, device=None):
    """Sums per-rank column sums of squares (fp64 [d_in]) and token counts over the process group.
    Returns (colsq_sum as a CPU fp64 tensor, total token count)."""
    if colsq.dtype != torch.float64 or colsq.dim() != 1:
        raise ValueError("colsq must be a 1-D float64 tensor")
    if world <= 1 or not dist.is_initialized():
        return colsq.detach().cpu().clone(), int(n_tokens)
    on = device if dist.get_backend() == "nccl" else "cpu"
    buf = torch.empty(colsq.numel() + 1, dtype=torch.float64, device=on)
    buf[:-1] = colsq.to(on)
    buf[-1] = float(n_tokens)          # exact in fp64 for any realistic token count
    dist.all_reduce(buf, op=dist.ReduceOp.SUM)
    buf = buf.cpu()
    return buf[:-1].clone(), int(round(float(buf[-1])))


def merge_calibration(ctx, world: int, device=None, stream=None) -> int:
    """Token-sharded calibration: every rank has accumulated its share of the tokens of the same
    layer input into its own context; afterwards every context holds the statistics of all
    tokens.  Returns the total token count.  (ctx is a binding.Context.)"""
    colsq, _S, _factor, n_tokens = ctx.sp_get_stats(stream)
    total, n_all = allreduce_colsq(colsq, n_tokens, world, device)
    ctx.sp_set_stats(total, n_all, stream)
    return n_all
