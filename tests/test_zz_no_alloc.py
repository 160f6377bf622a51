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


@pytest.mark.parametrize("T,n,ld,dtype", [
    (4096, 16384, 16384, torch.float16),     # the widest input: the fixed partial-sum area is full
    (1500, 16376, 16384, torch.bfloat16),    # padded row stride
    (900, 1001, 1001, torch.float16),        # odd width: element-wise loads
])
def test_noalloc_statistics_match_the_oracle_at_the_limits(T, n, ld, dtype):
    """Against the CPU oracle and the context path; checks as well that the call launches exactly
    its two kernels and leaves the device's free memory as it found it."""
    import numpy as np
    from oracle import swiftprune_oracle as so
    from paper_2501_16376_b200 import binding as sp
    from tests import parity as P
    buf = _batch(7, T, ld, dtype)
    X = buf[:, :n]
    colsq_out = torch.empty(n, dtype=torch.float64, device="cuda")
    factor_out = torch.empty(n, dtype=torch.float32, device="cuda")
    S_out = torch.empty(1, dtype=torch.float64, device="cuda")
    sp.sp_calib_stats_noalloc(X, colsq_out, factor_out, S_out)       # first call on the device
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    launches_before = sp.sp_launch_count()
    sp.sp_calib_stats_noalloc(X, colsq_out, factor_out, S_out)
    torch.cuda.synchronize()
    assert sp.sp_launch_count() - launches_before == 2
    assert torch.cuda.mem_get_info()[0] == free_before
    st = so.colsq_accumulate(so.new_stats(n), P.bits(X), P.odtype(X), threads=so.max_threads())
    assert P.rel_err(colsq_out.cpu().numpy(), st.colsq) <= P.SCORE_RTOL
    assert abs(S_out.item() - st.S) <= P.SCORE_RTOL * st.S
    assert P.rel_err(factor_out.cpu().numpy(), st.channel_factor32()) <= P.SCORE_RTOL
    colsq, S, factor = _reference(sp, X)
    assert _rel(colsq_out.cpu(), colsq) <= RTOL and abs(S_out.item() - S) <= RTOL * S
    assert np.isfinite(factor_out.cpu().numpy()).all()


def test_noalloc_rejects_sizes_beyond_its_fixed_array():
    from paper_2501_16376_b200 import binding as sp
    X = torch.zeros(8, 16392, dtype=torch.float16, device="cuda")
    with pytest.raises(sp.SpError) as e:
        sp.sp_calib_stats_noalloc(X)
    assert e.value.status == sp.SP_ERR_SHAPE
    with pytest.raises(sp.SpError) as e:
        sp.sp_calib_stats_noalloc(X[:0, :64])
    assert e.value.status == sp.SP_ERR_INVALID_ARG
