"""The 16-byte-access kernels on widths that are not whole tiles or strips: every aligned width
around the 256-column strip of the N:M kernel and the 512-column tile of the EWMA kernel, with
row counts that leave CTAs partly empty, both 16-bit types, with and without counters, in place
and out of place - each case against the oracle fed with the same statistics."""
import numpy as np
import pytest
import torch

from oracle import swiftprune_oracle as so
from tests import parity as P

pytestmark = pytest.mark.gpu

WIDTHS = [8, 16, 248, 256, 264, 504, 512, 520, 768, 1016, 1024, 1032, 1544, 2048 + 8]
ROWS = [1, 3, 4, 5, 33]


@pytest.fixture(scope="module")
def sp():
    from paper_2501_16376_b200 import binding
    return binding


def _inputs(seed, R, n, dtype):
    g = torch.Generator(device="cuda").manual_seed(seed)
    W = (torch.randn(R, n, generator=g, device="cuda") * 0.02).to(dtype)
    assert W.data_ptr() % 16 == 0
    rng = np.random.default_rng(seed)
    colsq = rng.uniform(0.5, 2.0, n) * 1e4
    colsq[rng.integers(0, n)] *= 300.0
    return W, colsq


@pytest.mark.parametrize("n", WIDTHS)
@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_nm_stream_kernel_on_partial_strips(sp, n, dtype):
    for k, R in enumerate(ROWS):
        for (N, M) in [(2, 4), (4, 8)]:
            W, colsq = _inputs(31 * n + R, R, n, dtype)
            W_ref = W.clone()
            with sp.Context(n) as ctx:
                ctx.sp_set_stats(torch.from_numpy(colsq), 5)
                sel = so.select_nm(P.bits(W_ref), P.odtype(W_ref), so.Stats(colsq.copy(), 5), N, M)
                # both outputs, mask only, weights only (the kernel is specialised on them)
                mask, out = ctx.sp_select_nm(W, N, M, inplace=(k % 2 == 1))
                P.check_selection(mask, out, W_ref, sel, None, strict=True)
                _, out_only = ctx.sp_select_nm(W_ref, N, M, want_mask=False)
                assert np.array_equal(P.bits(out_only), sel.W_out)
                mask_only = torch.full_like(mask, -1)
                st = sp.lib.sp_select_nm(ctx._h, W_ref.data_ptr(), sp.SP_F16 if dtype == torch.float16
                                         else sp.SP_BF16, R, W_ref.stride(0) if R > 1 else n, N, M,
                                         mask_only.data_ptr(), None, n,
                                         torch.cuda.current_stream().cuda_stream)
                assert st == sp.SP_OK
                assert np.array_equal(P.mask_np(mask_only), P.mask_np(mask))
                if (N, M) == (2, 4):  # the same selection, emitted as values + index records
                    values, meta = ctx.sp_select_24_compressed(W_ref)
                    v, m = so.compress_24(P.bits(W_ref), sel.keep_bool(n))
                    assert np.array_equal(P.bits(values), v)
                    assert np.array_equal(P.mask_np(meta), m)

@pytest.mark.parametrize("n", WIDTHS)
@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_ewma_pair_kernel_on_partial_tiles(sp, n, dtype):
    for k, R in enumerate(ROWS):
        W, colsq = _inputs(77 * n + R, R, n, dtype)
        W_ref = W.clone()
        la = [0.5, -0.2, 2.0, -0.9, 0.2][k]
        counters = sp.new_counters() if k % 2 == 0 else None
        with sp.Context(n) as ctx:
            ctx.sp_set_stats(torch.from_numpy(colsq), 5)
            params = sp.EwmaParams(0.125, 0.125, la, 0)
            mask, out = ctx.sp_select_unstructured(W, params=params, inplace=(k == 3),
                                                   counters=counters)
            sel = so.select_ewma(P.bits(W_ref), P.odtype(W_ref), so.Stats(colsq.copy(), 5), la,
                                 0.125, 0.125, s_update=so.S_FROZEN, want_trace=True)
            keep = so.unpack_mask(P.mask_np(mask), n)
            want = sel.keep_bool(n)
            diff = keep != want
            assert not (diff & ~P.ewma_allowed_flips(sel)).any()
            assert diff.sum() <= 1           # tiny matrices: at most one in-band entry
            assert keep[:, 0].all()          # column 0 is never pruned (Table 2)
            assert np.array_equal(P.bits(out), np.where(keep, P.bits(W_ref), 0))
            # bits past d_in in the last mask word are zero
            words = P.mask_np(mask)
            if n % 32:
                assert not (words[:, -1] >> np.uint32(n % 32)).any()
            if counters is not None:
                assert int(counters[sp.SP_COUNTER_KEPT]) == int(keep.sum())


@pytest.mark.parametrize("alpha,beta", [(1.0, 1.0), (1.0, 0.125), (0.01, 0.02), (0.5, 0.03125)])
def test_ewma_pair_kernel_parameter_extremes(sp, alpha, beta):
    # a = 1 - alpha = 0 makes every power in the lane scans vanish; a small alpha gives the state
    # a memory of hundreds of columns, i.e. many tiles
    R, n = 24, 2048
    W, colsq = _inputs(4242, R, n, torch.bfloat16)
    for la in (0.5, -0.9):
        with sp.Context(n) as ctx:
            ctx.sp_set_stats(torch.from_numpy(colsq), 5)
            mask, out = ctx.sp_select_unstructured(W, params=sp.EwmaParams(alpha, beta, la, 0))
            sel = so.select_ewma(P.bits(W), P.odtype(W), so.Stats(colsq.copy(), 5), la, alpha, beta,
                                 s_update=so.S_FROZEN, want_trace=True)
            keep = so.unpack_mask(P.mask_np(mask), n)
            diff = keep != sel.keep_bool(n)
            assert not (diff & ~P.ewma_allowed_flips(sel)).any()
            assert diff.sum() <= 1
            assert np.array_equal(P.bits(out), np.where(keep, P.bits(W), 0))


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_fast_kernels_with_padded_row_strides(sp, dtype):
    # rows that allow 16-byte access but are not contiguous: input and output are column slices of
    # wider matrices with different (aligned) leading dimensions
    R, n = 37, 1032
    g = torch.Generator(device="cuda").manual_seed(99)
    big_in = (torch.randn(R, n + 24, generator=g, device="cuda") * 0.02).to(dtype)
    W = big_in[:, 8:8 + n]
    big_out = torch.full((R, n + 40), 7.0, device="cuda").to(dtype)
    W_out = big_out[:, 16:16 + n]
    assert W.data_ptr() % 16 == 0 and W_out.data_ptr() % 16 == 0
    rng = np.random.default_rng(5)
    colsq = rng.uniform(0.5, 2.0, n) * 1e4
    W_ref = W.clone()
    with sp.Context(n) as ctx:
        ctx.sp_set_stats(torch.from_numpy(colsq), 5)
        st = so.Stats(colsq.copy(), 5)
        mask, out = ctx.sp_select_nm(W, 2, 4, W_out=W_out)
        sel = so.select_nm(P.bits(W_ref), P.odtype(W_ref), st, 2, 4)
        P.check_selection(mask, out, W_ref, sel, None, strict=True)
        values, meta = ctx.sp_select_24_compressed(W)
        v, m = so.compress_24(P.bits(W_ref), sel.keep_bool(n))
        assert np.array_equal(P.bits(values), v) and np.array_equal(P.mask_np(meta), m)
        for literal in (0, 1):
            big_out.fill_(7.0)
            mask, out = ctx.sp_select_unstructured(W, params=sp.EwmaParams(0.125, 0.125, 0.5, literal),
                                                   W_out=W_out)
            sel = so.select_ewma(P.bits(W_ref), P.odtype(W_ref), st, 0.5, 0.125, 0.125,
                                 s_update=so.S_LITERAL_W2 if literal else so.S_FROZEN,
                                 want_trace=True)
            keep = so.unpack_mask(P.mask_np(mask), n)
            diff = keep != sel.keep_bool(n)
            if literal:
                assert not diff.any()
            else:
                assert not (diff & ~P.ewma_allowed_flips(sel)).any() and diff.sum() <= 1
            assert np.array_equal(P.bits(out), np.where(keep, P.bits(W_ref), 0))
            # nothing outside the output slice was touched
            assert (big_out[:, :16] == 7.0).all() and (big_out[:, 16 + n:] == 7.0).all()
    assert np.array_equal(P.bits(W), P.bits(W_ref))   # the input was not modified
