"""Host logic of the multi-GPU path, run as two gloo ranks on the CPU."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2501_16376_b200 import sharding


def test_assign_units_is_a_balanced_partition():
    for n in (0, 1, 7, 32, 40, 224):
        for world in (1, 2, 3, 8):
            shares = [sharding.assign_units(n, world, r) for r in range(world)]
            flat = [u for s in shares for u in s]
            assert flat == list(range(n))
            sizes = [len(s) for s in shares]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.assign_units(4, 2, 2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        unit = sharding.unit_of_rank(rank, world)
        # every rank prunes its own unit; rank 1 is "slower"
        step_ms = 10.0 + 5.0 * rank
        slowest = sharding.max_over_ranks(step_ms, world)
        total = sharding.sum_over_ranks(1000.0 * (unit + 1), world)
        blocks = list(sharding.assign_units(7, world, rank))
        gathered = [None] * world
        dist.all_gather_object(gathered, blocks)
        # token-sharded calibration: per-rank column sums of squares add up
        colsq = torch.arange(5, dtype=torch.float64) * (rank + 1) + 0.25
        merged, tokens = sharding.allreduce_colsq(colsq, 100 + rank, world)
        if rank == 0:
            out.put((slowest, total, gathered, merged.tolist(), tokens))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_reduce_timing_and_partition_units():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    slowest, total, gathered, merged, tokens = out.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert slowest == 15.0                 # value = total work / slowest rank's time
    assert total == 3000.0
    assert gathered == [[0, 1, 2, 3], [4, 5, 6]]
    assert merged == [0.5 + 3.0 * k for k in range(5)]     # (k + 0.25) + (2k + 0.25)
    assert tokens == 201


def test_single_process_reductions_are_identity():
    assert sharding.max_over_ranks(3.5, 1) == 3.5
    assert sharding.sum_over_ranks(3.5, 1) == 3.5
    assert sharding.unit_of_rank(0, 1) == 0
    c = torch.tensor([1.0, 2.0], dtype=torch.float64)
    merged, tokens = sharding.allreduce_colsq(c, 7, 1)
    assert merged.tolist() == [1.0, 2.0] and tokens == 7
    with pytest.raises(ValueError):
        sharding.allreduce_colsq(c.float(), 7, 1)
