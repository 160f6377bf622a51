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


def test_token_and_row_shares_partition_their_ranges():
    for n, align in ((0, 1), (262144, 2048), (65536, 512), (1000, 64), (7, 3)):
        for world in (1, 2, 3, 8):
            shares = [sharding.token_share(n, world, r, align) for r in range(world)]
            assert [t for s in shares for t in s] == list(range(n))
            for s in shares[:-1]:
                assert s.stop % align == 0 or s.stop == n
    assert [list(sharding.row_share(10, 4, r)) for r in range(4)] == [[0, 1, 2], [3, 4, 5], [6, 7], [8, 9]]
    with pytest.raises(ValueError):
        sharding.token_share(8, 2, 0, align=0)


def _split_worker(rank, world, port, out):
    """One model shared by two ranks, by tokens and rows: each rank accumulates its token share
    (here with the CPU oracle standing in for the GPU kernel), the shares are merged with one
    all-reduce, and each rank selects its share of the rows."""
    import numpy as np
    from oracle import swiftprune_oracle as so
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        rng = np.random.default_rng(5)                      # the same data on every rank
        T, n, R = 96, 40, 10
        X = rng.standard_normal((T, n)).astype(np.float16).view(np.uint16)
        W = (rng.standard_normal((R, n)) * 0.02).astype(np.float16).view(np.uint16)
        share = sharding.token_share(T, world, rank, align=8)
        st = so.colsq_accumulate(so.new_stats(n), X[share.start:share.stop], so.F16)
        merged, tokens = sharding.allreduce_colsq(torch.from_numpy(st.colsq), st.n_tokens, world)
        stats = so.Stats(merged.numpy().copy(), tokens)
        rows = sharding.row_share(R, world, rank)
        sel = so.select_nm(W[rows.start:rows.stop], so.F16, stats, 2, 4)
        gathered = [None] * world
        dist.all_gather_object(gathered, (list(rows), sel.mask.tolist(), tokens))
        if rank == 0:
            whole = so.colsq_accumulate(so.new_stats(n), X, so.F16)
            ref = so.select_nm(W, so.F16, whole, 2, 4)
            out.put((gathered, ref.mask.tolist(), np.array_equal(stats.colsq, whole.colsq)))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_share_one_model_by_tokens_and_rows():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_split_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    gathered, ref_mask, same_stats = out.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert same_stats                                   # fp64 sums of exact squares: additive
    assert [t for _, _, t in gathered] == [96, 96]
    rows = [r for part, _, _ in gathered for r in part]
    masks = [m for _, part, _ in gathered for m in part]
    assert rows == list(range(10)) and masks == ref_mask
