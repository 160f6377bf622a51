"""The allocation-free statistics call, checked against the ordinary context path.

Some users of the library run where device memory must not be allocated while they work:
inside a framework that has taken the whole memory pool for itself, in a service that has
given every spare byte to its caches, or in a latency-critical loop where the device-wide
synchronisation hidden in cudaMalloc/cudaFree is not acceptable.  For them
``sp_calib_stats_noalloc`` keeps its working memory in a fixed array inside the library.
This file is named so that it is collected after every other test."""
import pytest
import torch

pytestmark = pytest.mark.gpu

RTOL = 1e-6   # same bound the statistics tests use (fp32 sums of 8 squares, fp64 beyond)


def _batch(seed, T, n, dtype):
    g = torch.Generator(device="cuda").manual_seed(seed)
    X = torch.randn(T, n, generator=g, device="cuda")
    X[:, :: max(1, n // 4)] *= 20.0
    return X.to(dtype)


def _reference(sp, X):
    with sp.Context(X.shape[1]) as ctx:
        ctx.sp_calib_accumulate(X)
        colsq, S, factor, _ = ctx.sp_get_stats()
    return colsq, S, factor


def _rel(a, b):
    return ((a - b).abs() / b.abs().clamp_min(1e-300)).max().item()


def test_noalloc_statistics_match_the_context_path_on_two_calls_in_a_row():
    from paper_2501_16376_b200 import binding as sp
    # caller-owned outputs, allocated before the calls under test (sized for the larger case)
    colsq_out = torch.full((4096,), -1.0, dtype=torch.float64, device="cuda")
    factor_out = torch.full((4096,), -1.0, dtype=torch.float32, device="cuda")
    S_out = torch.full((1,), -1.0, dtype=torch.float64, device="cuda")
    # second call: narrower, ragged, other dtype - stale contents of the shared array must not leak
    cases = [(_batch(1, 3000, 4096, torch.float16)), (_batch(2, 777, 520, torch.bfloat16))]
    for X in cases:
        n = X.shape[1]
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated()
        sp.sp_calib_stats_noalloc(X, colsq_out, factor_out, S_out)
        assert torch.cuda.memory_allocated() == before      # the wrapper allocates nothing either
        torch.cuda.synchronize()
        colsq, S, factor = _reference(sp, X)
        assert _rel(colsq_out[:n].cpu(), colsq) <= RTOL
        assert abs(S_out.item() - S) <= RTOL * S
        assert _rel(factor_out[:n].cpu().double(), factor.double()) <= RTOL
    # the same input twice gives the same bits
    X = cases[0]
    sp.sp_calib_stats_noalloc(X, colsq_out, factor_out, S_out)
    first = colsq_out.clone()
    sp.sp_calib_stats_noalloc(X, colsq_out, factor_out, S_out)
    assert torch.equal(first, colsq_out)


def test_noalloc_rejects_sizes_beyond_its_fixed_array():
    from paper_2501_16376_b200 import binding as sp
    X = torch.zeros(8, 16392, dtype=torch.float16, device="cuda")
    with pytest.raises(sp.SpError) as e:
        sp.sp_calib_stats_noalloc(X)
    assert e.value.status == sp.SP_ERR_SHAPE
    with pytest.raises(sp.SpError) as e:
        sp.sp_calib_stats_noalloc(X[:0, :64])
    assert e.value.status == sp.SP_ERR_INVALID_ARG
