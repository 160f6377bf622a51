"""GPU parity: the CUDA library, called through its C ABI binding, against the CPU oracle on
the same seeded inputs, element by element."""
import numpy as np
import pytest
import torch

from oracle import swiftprune_oracle as so
from tests import parity as P

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sp():
    from paper_2501_16376_b200 import binding
    return binding


def _gen(seed, shape, dtype, std=1.0, device="cuda"):
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return (torch.randn(shape, generator=g, device=device, dtype=torch.float32) * std).to(dtype)


def _activations(seed, T, n, dtype, outliers=4):
    X = _gen(seed, (T, n), torch.float32)
    idx = torch.randperm(n, generator=torch.Generator().manual_seed(seed))[:min(outliers, n)]
    X[:, idx.cuda()] *= 20.0
    return X.to(dtype)


# ------------------------------------------------------------------ statistics

@pytest.mark.parametrize("T,n,dtype,ld_extra", [
    (2048, 512, torch.float16, 0),      # the small single-layer case
    (1000, 520, torch.float16, 0),      # ragged strip (520 = 2*256 + 8), ragged rows
    (77, 1030, torch.float16, 0),       # d_in not a multiple of 8: element-wise path
    (3000, 1024, torch.bfloat16, 0),
    (513, 768, torch.float16, 8),       # strided rows, still 16-byte aligned
    (513, 768, torch.bfloat16, 3),      # strided rows, misaligned: element-wise path
    (5, 8, torch.float16, 0),           # fewer rows than one warp step
    (1, 1, torch.float16, 0),
    (16384, 4096, torch.float16, 0),    # one batch of a LLaMA-7B-width input (134 MB)
])
def test_calib_statistics_match_oracle(sp, T, n, dtype, ld_extra):
    X_full = _activations(T * 31 + n, T, n + ld_extra, dtype)
    X = X_full[:, :n]
    with sp.Context(n) as ctx:
        ctx.sp_calib_accumulate(X)
        colsq, S, factor, ntok = ctx.sp_get_stats()
    st = P.oracle_stats([X], n)
    assert ntok == T
    assert P.rel_err(colsq.numpy(), st.colsq) <= P.SCORE_RTOL
    assert abs(S - st.S) <= P.SCORE_RTOL * st.S
    if n > 1:
        assert P.rel_err(factor.numpy(), st.channel_factor32()) <= P.SCORE_RTOL
    # tighter than the contract: fp32 partial sums of 8 squares, fp64 beyond
    assert P.rel_err(colsq.numpy(), st.colsq) <= 1e-6


def test_calib_accumulates_over_batches_resets_and_is_deterministic(sp):
    n = 1536
    batches = [_activations(100 + i, T, n, torch.float16) for i, T in enumerate([700, 64, 2048, 1])]
    with sp.Context(n) as ctx:
        for X in batches:
            ctx.sp_calib_accumulate(X)
        colsq, S, factor, ntok = ctx.sp_get_stats()
        st = P.oracle_stats(batches, n)
        assert ntok == sum(b.shape[0] for b in batches)
        assert P.rel_err(colsq.numpy(), st.colsq) <= 1e-6
        # same batches again after a reset: bit-identical (no floating-point atomics)
        ctx.sp_calib_reset()
        for X in batches:
            ctx.sp_calib_accumulate(X)
        colsq2, S2, factor2, _ = ctx.sp_get_stats()
        assert torch.equal(colsq, colsq2) and S == S2 and torch.equal(factor, factor2)
        # reset really forgets
        ctx.sp_calib_reset()
        ctx.sp_calib_accumulate(batches[1])
        colsq3, _, _, ntok3 = ctx.sp_get_stats()
        assert ntok3 == 64
        assert P.rel_err(colsq3.numpy(), P.oracle_stats([batches[1]], n).colsq) <= 1e-6
        # an empty batch is a no-op
        ctx.sp_calib_accumulate(batches[1][:0])
        assert ctx.sp_get_stats()[3] == 64


def test_set_stats_round_trip_and_factor_is_bit_exact(sp):
    n = 1000
    rng = np.random.default_rng(3)
    colsq = rng.uniform(0.5, 2.0, n) * 1e4
    colsq[[3, 500]] *= 400.0
    with sp.Context(n) as ctx:
        ctx.sp_set_stats(torch.from_numpy(colsq), 123)
        got, S, factor, ntok = ctx.sp_get_stats()
    st = so.Stats(colsq.copy(), 123)
    assert np.array_equal(got.numpy(), colsq) and ntok == 123
    assert abs(S - st.S) <= 1e-12 * st.S
    assert np.array_equal(factor.numpy(), st.channel_factor32())


# ------------------------------------------------------------------ scores

@pytest.mark.parametrize("R,n,dtype", [(64, 512, torch.float16), (33, 520, torch.bfloat16),
                                       (7, 1030, torch.float16)])
def test_scores_match_oracle(sp, R, n, dtype):
    W = _gen(R + n, (R, n), dtype, 0.02)
    X = _activations(n, 512, n, dtype)
    with sp.Context(n) as ctx:
        ctx.sp_calib_accumulate(X)
        L = ctx.sp_score(W).cpu().numpy()
        colsq, _, _, _ = ctx.sp_get_stats()
    st = P.oracle_stats([X], n)
    want = so.score_f32(P.bits(W), P.odtype(W), st)
    assert P.rel_err(L, want) <= P.SCORE_RTOL
    # with the library's own statistics handed to the oracle the scores are bit-identical
    st_gpu = so.Stats(colsq.numpy().copy(), 512)
    assert np.array_equal(L, so.score_f32(P.bits(W), P.odtype(W), st_gpu))


# ------------------------------------------------------------------ N:M selection

def _ctx_with_stats(sp, X_batches, n):
    ctx = sp.Context(n)
    for X in X_batches:
        ctx.sp_calib_accumulate(X)
    return ctx


@pytest.mark.parametrize("R,n,dtype,N,M", [
    (512, 512, torch.float16, 2, 4),
    (300, 520, torch.float16, 2, 4),      # ragged last tile
    (300, 520, torch.bfloat16, 4, 8),
    (64, 1028, torch.float16, 2, 4),      # d_in % 8 == 4: element-wise path, half-filled chunk
    (129, 2048, torch.bfloat16, 2, 4),    # bf16: many equal scores inside groups
    (40, 1024, torch.float16, 1, 4),
    (40, 1024, torch.float16, 3, 4),
    (40, 1024, torch.float16, 2, 8),
    (40, 1024, torch.float16, 6, 8),
    (1, 8, torch.float16, 4, 8),
    (3, 4, torch.float16, 2, 4),
])
def test_nm_selection_matches_oracle(sp, R, n, dtype, N, M):
    W = _gen(R * 7 + n, (R, n), dtype, 0.02)
    X = _activations(n + 1, 1024, n, dtype)
    with _ctx_with_stats(sp, [X], n) as ctx:
        mask, out = ctx.sp_select_nm(W, N, M)
        colsq = ctx.sp_get_stats()[0]
        # (a) against the oracle fed with the oracle's own statistics: tolerance rule
        st = P.oracle_stats([X], n)
        sel = so.select_nm(P.bits(W), P.odtype(W), st, N, M, want_trace=True)
        P.check_selection(mask, out, W, sel, P.nm_allowed_flips(sel, n, M))
        # (b) against the oracle fed with the library's statistics: bit-exact
        sel2 = so.select_nm(P.bits(W), P.odtype(W), so.Stats(colsq.numpy().copy(), 1), N, M)
        P.check_selection(mask, out, W, sel2, None, strict=True)
    keep = so.unpack_mask(P.mask_np(mask), n)
    assert (keep.reshape(R, n // M, M).sum(-1) == N).all()


def test_nm_ties_follow_the_lower_column_rule(sp):
    # few distinct magnitudes and uniform statistics: ties in almost every group
    R, n = 64, 512
    g = torch.Generator(device="cuda").manual_seed(5)
    vals = torch.tensor([0.01, 0.02, 0.02, 0.03], device="cuda")
    W = vals[torch.randint(0, 4, (R, n), generator=g, device="cuda")]
    W = (W * (torch.randint(0, 2, (R, n), generator=g, device="cuda") * 2 - 1)).to(torch.float16)
    colsq = np.full(n, 1000.0)
    with sp.Context(n) as ctx:
        ctx.sp_set_stats(torch.from_numpy(colsq), 10)
        for N, M in ((2, 4), (4, 8)):
            mask, out = ctx.sp_select_nm(W, N, M)
            sel = so.select_nm(P.bits(W), so.F16, so.Stats(colsq.copy(), 10), N, M)
            P.check_selection(mask, out, W, sel, None, strict=True)


def test_nm_in_place_strided_and_mask_only(sp):
    R, n = 96, 768
    big = _gen(9, (R, n + 16), torch.float16, 0.02)
    big_before = big.clone()
    W = big[:, 8:8 + n]                      # ld = n + 16, 16-byte aligned start
    W_ref = W.clone()
    X = _activations(10, 512, n, torch.float16)
    with _ctx_with_stats(sp, [X], n) as ctx:
        colsq = ctx.sp_get_stats()[0]
        sel = so.select_nm(P.bits(W_ref), so.F16, so.Stats(colsq.numpy().copy(), 1), 2, 4)
        mask, out = ctx.sp_select_nm(W, 2, 4, inplace=True)
        assert out.data_ptr() == W.data_ptr()
        P.check_selection(mask, W, W_ref, sel, None, strict=True)
        # the columns outside the view are untouched
        assert torch.equal(big[:, :8], big_before[:, :8])
        assert torch.equal(big[:, n + 8:], big_before[:, n + 8:])
        # idempotent: selecting again on the pruned matrix reproduces the mask
        mask2, _ = ctx.sp_select_nm(W, 2, 4)
        assert torch.equal(mask, mask2)


# ------------------------------------------------------------------ EWMA selection

def _ewma_params(sp, la, alpha=0.125, beta=0.125, s_update=0):
    return sp.EwmaParams(alpha, beta, la, s_update)


@pytest.mark.parametrize("R,n,dtype,sparsity", [
    (512, 512, torch.float16, 0.5),       # the small single-layer case
    (300, 520, torch.float16, 0.6),       # ragged last tile
    (64, 1030, torch.float16, 0.7),       # element-wise path
    (200, 4096, torch.bfloat16, 0.5),
    (200, 4096, torch.bfloat16, 0.8),
    (50, 11008, torch.float16, 0.5),      # long rows: 43 tiles
    (3, 8, torch.float16, 0.5),
    (2, 1, torch.float16, 0.5),
])
def test_ewma_selection_matches_oracle(sp, R, n, dtype, sparsity):
    W = _gen(R * 3 + n, (R, n), dtype, 0.02)
    X = _activations(n + 2, 2048, n, dtype)
    counters = sp.new_counters()
    with _ctx_with_stats(sp, [X], n) as ctx:
        mask, out = ctx.sp_select_unstructured(W, sparsity, counters=counters)
        colsq = ctx.sp_get_stats()[0]
    st = so.Stats(colsq.numpy().copy(), 1)    # isolate the selection from the statistics
    sel = so.select_unstructured(P.bits(W), P.odtype(W), st, sparsity, want_trace=True,
                                 s_update=so.S_LITERAL_W2)
    # tiny matrices: the 1e-6 fraction allows no flip at all
    P.check_selection(mask, out, W, sel, P.ewma_allowed_flips(sel))
    keep = so.unpack_mask(P.mask_np(mask), n)
    assert keep[:, 0].all()                   # column 0 is never pruned
    assert int(counters[sp.SP_COUNTER_KEPT]) == int(keep.sum())
    # at calibration scale "S - w^2" cannot change S in fp32: no hazard rows
    assert int(counters[sp.SP_COUNTER_S_HAZARD]) == 0
    # also against the oracle's own statistics, under the tolerance rule
    st_o = P.oracle_stats([X], n)
    sel_o = so.select_unstructured(P.bits(W), P.odtype(W), st_o, sparsity, want_trace=True)
    P.check_selection(mask, out, W, sel_o, P.ewma_allowed_flips(sel_o))


@pytest.mark.parametrize("alpha,beta,la", [(0.125, 0.125, 4.0), (0.5, 0.25, 0.5),
                                           (0.03125, 0.0625, -0.2), (1.0, 1.0, 0.5)])
def test_ewma_other_parameters(sp, alpha, beta, la):
    R, n = 128, 2048
    W = _gen(77, (R, n), torch.float16, 0.02)
    X = _activations(78, 1024, n, torch.float16)
    with _ctx_with_stats(sp, [X], n) as ctx:
        mask, out = ctx.sp_select_unstructured(W, params=_ewma_params(sp, la, alpha, beta))
        colsq = ctx.sp_get_stats()[0]
    st = so.Stats(colsq.numpy().copy(), 1)
    sel = so.select_ewma(P.bits(W), so.F16, st, la, alpha, beta, s_update=so.S_FROZEN,
                         want_trace=True)
    P.check_selection(mask, out, W, sel, P.ewma_allowed_flips(sel))


def test_ewma_literal_S_update_is_bit_exact_and_hazard_counter_fires(sp):
    # Tiny statistics: S is comparable to sum w^2, so Algorithm 1's "S = S - w_i^2" matters.
    R, n = 96, 640
    W = _gen(21, (R, n), torch.float16, 0.02)
    colsq = np.random.default_rng(4).uniform(1.0, 2.0, n) * 1e-4
    with sp.Context(n) as ctx:
        ctx.sp_set_stats(torch.from_numpy(colsq), 10)
        st = so.Stats(colsq.copy(), 10)
        lit = so.select_ewma(P.bits(W), so.F16, st, 0.5, s_update=so.S_LITERAL_W2)
        fro = so.select_ewma(P.bits(W), so.F16, st, 0.5, s_update=so.S_FROZEN, want_trace=True)
        assert not np.array_equal(lit.mask, fro.mask)          # the two readings differ here
        counters = sp.new_counters()
        mask, out = ctx.sp_select_unstructured(
            W, params=_ewma_params(sp, 0.5, s_update=sp.SP_S_LITERAL_W2), counters=counters)
        P.check_selection(mask, out, W, lit, None, strict=True)  # sequential kernel: bit-exact
        assert int(counters[sp.SP_COUNTER_KEPT]) == int(lit.keep_bool(n).sum())
        counters.zero_()
        mask_f, out_f = ctx.sp_select_unstructured(
            W, params=_ewma_params(sp, 0.5, s_update=sp.SP_S_FROZEN), counters=counters)
        P.check_selection(mask_f, out_f, W, fro, P.ewma_allowed_flips(fro))
        assert int(counters[sp.SP_COUNTER_S_HAZARD]) == 0      # nothing is gated in this mode
        assert int(counters[sp.SP_COUNTER_KEPT]) == int(so.unpack_mask(P.mask_np(mask_f), n).sum())


@pytest.mark.parametrize("R,n,inplace,misalign", [
    (96, 640, False, False),      # rows of two tiles, several rows per CTA
    (96, 640, True, False),
    (40, 4096, True, False),      # one row per CTA
    (24, 8192 + 512, False, False),  # rows walked in two passes
    (24, 8192 + 512, True, False),   # ... pruned in place: marks come from the pre-pass
    (33, 648, True, True),        # unaligned rows: element-wise kernels
])
def test_default_call_is_algorithm_1_when_S_moves(sp, R, n, inplace, misalign):
    """The drift gate: with statistics so small that "S = S - w_i^2" changes S, the default
    entry point must give the literal result of Algorithm 1 bit for bit, rows of the other
    kind (here: a few rows scaled down until their w^2 cannot move S) stay on the scan path."""
    W = _gen(91 + n, (R, n), torch.float16, 0.02)
    quiet = [1, R // 2, R - 1]
    W[quiet] = W[quiet] * 2.0 ** -13          # w^2 <= 1.2e-10: below the hazard bound of S ~ 0.02
    if misalign:
        buf = torch.zeros(R * n + 1, dtype=W.dtype, device=W.device)
        buf[1:] = W.reshape(-1)
        W = buf[1:].view(R, n)
    colsq = np.random.default_rng(4).uniform(1.0, 2.0, n) * (12.8 / n) * 1e-3   # S ~ sum w^2
    with sp.Context(n) as ctx:
        ctx.sp_set_stats(torch.from_numpy(colsq), 10)
        st = so.Stats(colsq.copy(), 10)
        lit = so.select_unstructured(P.bits(W), so.F16, st, 0.5, s_update=so.S_LITERAL_W2,
                                     want_trace=True)
        fro = so.select_unstructured(P.bits(W), so.F16, st, 0.5, s_update=so.S_FROZEN)
        assert not np.array_equal(lit.mask, fro.mask)
        counters = sp.new_counters()
        W_in = W.clone() if not misalign else W
        src = W_in.clone()
        mask, out = ctx.sp_select_unstructured(W_in, 0.5, counters=counters,
                                               inplace=inplace)
        hazard = int(counters[sp.SP_COUNTER_S_HAZARD])
        assert R - len(quiet) <= hazard <= R
        got = so.unpack_mask(P.mask_np(mask), n)
        rows = np.ones(R, bool)
        rows[quiet] = False
        assert np.array_equal(got[rows], lit.keep_bool(n)[rows])   # gated rows: bit-exact
        P.check_selection(mask, out, src, lit, P.ewma_allowed_flips(lit))
        assert int(counters[sp.SP_COUNTER_KEPT]) == int(got.sum())
        # the row bitmap is clean again: a second call gives the same answer
        if not misalign:
            counters.zero_()
            mask2, out2 = ctx.sp_select_unstructured(src, 0.5, counters=counters)
            assert torch.equal(mask, mask2)
            assert torch.equal(out.view(torch.int16), out2.view(torch.int16))
            assert R - len(quiet) <= int(counters[sp.SP_COUNTER_S_HAZARD]) <= R


def test_ewma_literal_equals_frozen_at_calibration_scale(sp):
    R, n = 64, 1024
    W = _gen(31, (R, n), torch.bfloat16, 0.02)
    X = _activations(32, 4096, n, torch.bfloat16)
    with _ctx_with_stats(sp, [X], n) as ctx:
        a, _ = ctx.sp_select_unstructured(W, params=_ewma_params(sp, 0.5, s_update=1))
        colsq = ctx.sp_get_stats()[0]
    sel = so.select_ewma(P.bits(W), so.BF16, so.Stats(colsq.numpy().copy(), 1), 0.5,
                         s_update=so.S_LITERAL_W2)
    assert np.array_equal(P.mask_np(a), sel.mask)


def test_ewma_in_place_and_determinism(sp):
    R, n = 128, 1536
    W = _gen(41, (R, n), torch.float16, 0.02)
    W_ref = W.clone()
    X = _activations(42, 1024, n, torch.float16)
    with _ctx_with_stats(sp, [X], n) as ctx:
        m1, o1 = ctx.sp_select_unstructured(W, 0.5)
        m2, o2 = ctx.sp_select_unstructured(W, 0.5)
        assert torch.equal(m1, m2) and torch.equal(o1.view(torch.int16), o2.view(torch.int16))
        m3, o3 = ctx.sp_select_unstructured(W, 0.5, inplace=True)
        assert o3.data_ptr() == W.data_ptr()
        assert torch.equal(m1, m3) and torch.equal(W.view(torch.int16), o1.view(torch.int16))
        assert not torch.equal(W, W_ref)


# ------------------------------------------------------------------ write-back

@pytest.mark.parametrize("R,n,dtype", [(100, 520, torch.float16), (17, 1030, torch.bfloat16),
                                       (1, 1, torch.float16), (64, 4096, torch.float16)])
def test_apply_mask_matches_oracle(sp, R, n, dtype):
    W = _gen(R + 3 * n, (R, n), dtype, 0.02)
    g = torch.Generator().manual_seed(R)
    keep = torch.rand(R, n, generator=g) < 0.5
    words = (n + 31) // 32
    packed = np.zeros((R, words * 32), dtype=np.uint8)
    packed[:, :n] = keep.numpy()
    mask = np.packbits(packed, axis=1, bitorder="little").view(np.uint32)
    mask_t = torch.from_numpy(mask.view(np.int32)).cuda()
    out = sp.sp_apply_mask(W, mask_t)
    assert np.array_equal(P.bits(out), so.apply_mask(P.bits(W), mask))
    # in place
    W2 = W.clone()
    sp.sp_apply_mask(W2, mask_t, W2)
    assert torch.equal(W2.view(torch.int16), out.view(torch.int16))


# ------------------------------------------------------------------ edge cases and errors

def test_empty_inputs_are_no_ops(sp):
    n = 256
    X = _activations(1, 64, n, torch.float16)
    with _ctx_with_stats(sp, [X], n) as ctx:
        W0 = torch.empty(0, n, dtype=torch.float16, device="cuda")
        m, o = ctx.sp_select_nm(W0, 2, 4)
        assert m.shape == (0, 8) and o.shape == (0, n)
        m, o = ctx.sp_select_unstructured(W0, 0.5)
        assert m.shape == (0, 8)
        assert ctx.sp_score(W0).shape == (0, n)
    empty_mask = torch.empty(0, 8, dtype=torch.int32, device="cuda")
    assert sp.sp_apply_mask(W0, empty_mask).shape == (0, n)


def test_error_statuses(sp):
    n = 64
    W = _gen(1, (8, n), torch.float16, 0.02)
    with sp.Context(n) as ctx:
        with pytest.raises(sp.SpError) as e:                      # nothing calibrated yet
            ctx.sp_select_nm(W, 2, 4)
        assert e.value.status == sp.SP_ERR_STATE
        with pytest.raises(sp.SpError) as e:
            ctx.sp_get_stats()
        assert e.value.status == sp.SP_ERR_STATE
        ctx.sp_calib_accumulate(_activations(2, 32, n, torch.float16))
        with pytest.raises(sp.SpError) as e:
            ctx.sp_select_nm(W, 4, 4)
        assert e.value.status == sp.SP_ERR_INVALID_ARG
        with pytest.raises(sp.SpError) as e:
            ctx.sp_select_nm(W, 2, 5)
        assert e.value.status == sp.SP_ERR_INVALID_ARG
        with pytest.raises(sp.SpError) as e:
            ctx.sp_select_unstructured(W, 1.5)
        assert e.value.status == sp.SP_ERR_INVALID_ARG
        with pytest.raises(sp.SpError) as e:
            ctx.sp_select_unstructured(W, params=_ewma_params(sp, 0.5, alpha=0.0))
        assert e.value.status == sp.SP_ERR_INVALID_ARG
        with pytest.raises(sp.SpError) as e:
            ctx.sp_calib_accumulate(_activations(2, 32, n + 8, torch.float16))
        assert e.value.status == sp.SP_ERR_SHAPE
        with pytest.raises(sp.SpError) as e:
            ctx.sp_select_nm(W.float(), 2, 4)
        assert e.value.status == sp.SP_ERR_DTYPE
    with sp.Context(60) as ctx:                                    # 60 % 8 != 0
        ctx.sp_calib_accumulate(_activations(3, 32, 60, torch.float16))
        with pytest.raises(sp.SpError) as e:
            ctx.sp_select_nm(_gen(1, (4, 60), torch.float16), 4, 8)
        assert e.value.status == sp.SP_ERR_SHAPE
    with pytest.raises(sp.SpError) as e:
        sp.Context(0)
    assert e.value.status == sp.SP_ERR_SHAPE


def test_degenerate_statistics_are_reported_not_faulted(sp):
    n = 128
    W = _gen(1, (8, n), torch.float16, 0.02)
    with sp.Context(n) as ctx:
        ctx.sp_calib_accumulate(torch.zeros(64, n, dtype=torch.float16, device="cuda"))
        with pytest.raises(sp.SpError) as e:
            ctx.sp_get_stats()
        assert e.value.status == sp.SP_ERR_DEGENERATE
        ctx.sp_select_nm(W, 2, 4)               # still runs; results are unspecified
        torch.cuda.synchronize()
    # a single live channel gives an infinite factor there and ordinary ones elsewhere
    with sp.Context(n) as ctx:
        X = torch.zeros(64, n, dtype=torch.float16, device="cuda")
        X[:, 5] = 1.0
        ctx.sp_calib_accumulate(X)
        factor = ctx.sp_get_stats()[2]
        assert torch.isinf(factor[5]) and (factor[:5] == 0.5).all()


def test_launch_counter_counts_kernels(sp):
    n = 256
    before = sp.sp_launch_count()
    with sp.Context(n) as ctx:
        ctx.sp_calib_accumulate(_activations(1, 64, n, torch.float16))   # 1
        ctx.sp_select_nm(_gen(1, (8, n), torch.float16, 0.02), 2, 4)      # finalise + select
    assert sp.sp_launch_count() - before == 3


# ------------------------------------------------------------------ host-buffer entry points

@pytest.mark.parametrize("pinned", [True, False])
def test_host_buffer_calls_match_device_calls(sp, pinned):
    # wide enough that the 64 MiB staging slots are cycled several times
    R, n, T = 20000, 4096, 40000
    W = _gen(61, (R, n), torch.float16, 0.02)
    X = _activations(62, T, n, torch.float16)

    def host(t):
        h = t.cpu()
        return h.pin_memory() if pinned else h

    Wh, Xh = host(W), host(X)
    words = (n + 31) // 32
    with sp.Context(n) as dev_ctx, sp.Context(n) as host_ctx:
        dev_ctx.sp_calib_accumulate(X)
        host_ctx.sp_calib_accumulate_host(Xh[:15000])
        host_ctx.sp_calib_accumulate_host(Xh[15000:])
        c_dev, S_dev, f_dev, _ = dev_ctx.sp_get_stats()
        c_host, S_host, f_host, ntok = host_ctx.sp_get_stats()
        assert ntok == T
        assert P.rel_err(c_host.numpy(), c_dev.numpy()) <= 1e-6   # chunking changes slab cuts only
        host_ctx.sp_set_stats(c_dev, T)                            # identical statistics from here on
        m_dev, o_dev = dev_ctx.sp_select_nm(W, 2, 4)
        m_host = host(torch.zeros(R, words, dtype=torch.int32))
        o_host = host(torch.zeros(R, n, dtype=torch.float16))
        host_ctx.sp_select_nm_host(Wh, 2, 4, m_host, o_host)
        torch.cuda.synchronize()
        assert torch.equal(m_host, m_dev.cpu())
        assert torch.equal(o_host.view(torch.int16), o_dev.cpu().view(torch.int16))
        m_dev, o_dev = dev_ctx.sp_select_unstructured(W, 0.5)
        host_ctx.sp_select_unstructured_host(Wh, 0.5, m_host, o_host)
        torch.cuda.synchronize()
        assert torch.equal(m_host, m_dev.cpu())
        assert torch.equal(o_host.view(torch.int16), o_dev.cpu().view(torch.int16))
        # in place on the host, mask not wanted
        Wh2 = host(W)
        host_ctx.sp_select_nm_host(Wh2, 2, 4, None, Wh2)
        torch.cuda.synchronize()
        assert torch.equal(Wh2.view(torch.int16), dev_ctx.sp_select_nm(W, 2, 4)[1].cpu().view(torch.int16))


# ------------------------------------------------------------------ la search

@pytest.mark.parametrize("target", [0.5, 0.35, 0.75])
def test_la_search_matches_oracle_bisection(sp, target):
    R, n = 256, 4096
    W = _gen(91, (R, n), torch.bfloat16, 0.02)
    X = _activations(92, 2048, n, torch.bfloat16)
    with _ctx_with_stats(sp, [X], n) as ctx:
        la, achieved = ctx.sp_search_la(W, target)
        colsq = ctx.sp_get_stats()[0]
        st = so.Stats(colsq.numpy().copy(), 1)
        la_o, achieved_o = so.search_la(P.bits(W), so.BF16, st, target, threads=so.max_threads())
        # counts may differ by entries inside the threshold band, which can move the bisection
        # by at most its final resolution
        assert abs(achieved - achieved_o) <= 2e-6 + 1.0 / (R * n)
        assert abs(la - la_o) <= 16.0 / 2 ** 20
        assert abs(achieved - target) < 1e-4
        mask, _ = ctx.sp_select_unstructured(W, params=sp.EwmaParams(0.125, 0.125, la, 0))
        keep = so.unpack_mask(P.mask_np(mask), n)
        assert abs((1.0 - keep.mean()) - achieved) < 1e-12


# ------------------------------------------------------------------ token-sharded calibration

def test_token_shards_merge_into_the_statistics_of_all_tokens(sp):
    # what two ranks that each saw half the tokens would do, in one process: the column sums of
    # squares add up, so the merged context selects exactly like one that saw every token
    from paper_2501_16376_b200 import sharding
    n, T = 1024, 4096
    X = _activations(77, T, n, torch.float16)
    W = _gen(78, (64, n), torch.float16, 0.02)
    with sp.Context(n) as whole, sp.Context(n) as a, sp.Context(n) as b:
        whole.sp_calib_accumulate(X)
        a.sp_calib_accumulate(X[:T // 2])
        b.sp_calib_accumulate(X[T // 2:])
        ca, _, _, ta = a.sp_get_stats()
        cb, _, _, tb = b.sp_get_stats()
        a.sp_set_stats(ca + cb, ta + tb)                    # the all-reduce, written out
        assert sharding.merge_calibration(b, world=1) == T // 2   # one rank: nothing to add
        cw, Sw, fw, tw = whole.sp_get_stats()
        cm, Sm, fm, tm = a.sp_get_stats()
        assert tm == tw == T
        assert torch.allclose(cm, cw, rtol=1e-13, atol=0.0)
        assert abs(Sm - Sw) <= 1e-12 * Sw
        m1, o1 = whole.sp_select_nm(W, 2, 4)
        m2, o2 = a.sp_select_nm(W, 2, 4)
        assert torch.equal(m1, m2) and torch.equal(o1, o2)


# ------------------------------------------------------------------ CUDA graph capture

def test_whole_pass_can_be_captured_and_replayed_as_a_cuda_graph(sp):
    from paper_2501_16376_b200 import pipeline, synth
    w = synth.scaled(synth.WORKLOADS["llama2-7b"], blocks=2, n_seqs=4, seq_len=128, shrink=16)
    mb = pipeline.allocate_model(w, "cuda")
    try:
        batch_tokens = 2 * w.seq_len
        pipeline.prune_model(mb, (2, 4), batch_tokens)
        torch.cuda.synchronize()
        want_masks = [[m.clone() for m in ms] for ms in mb.masks]
        want_out = [[o.clone() for o in os_] for os_ in mb.outputs]
        for ms, os_ in zip(mb.masks, mb.outputs):
            for m, o in zip(ms, os_):
                m.zero_()
                o.zero_()
        graph, counts = pipeline.capture_model_graph(mb, (2, 4), batch_tokens)
        for ms, os_ in zip(mb.masks, mb.outputs):
            for m, o in zip(ms, os_):
                m.zero_()
                o.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert counts["select"] == w.blocks                    # one launch per block
        for b in range(w.blocks):
            for li in range(len(w.layers)):
                assert torch.equal(mb.masks[b][li], want_masks[b][li])
                assert torch.equal(mb.outputs[b][li].view(torch.int16),
                                   want_out[b][li].view(torch.int16))
    finally:
        mb.close()


@pytest.mark.parametrize("name,arg", [("llama3-8b", 0.5), ("llama2-7b", (2, 4)),
                                      ("llama2-13b", (4, 8))])
def test_pass_with_per_block_per_input_and_per_layer_calls_agree(sp, name, arg):
    from paper_2501_16376_b200 import pipeline, synth
    w = synth.scaled(synth.WORKLOADS[name], blocks=2, n_seqs=4, seq_len=128, shrink=16)
    mb = pipeline.allocate_model(w, "cuda")
    try:
        batch_tokens = 2 * w.seq_len
        results = {}
        for how, kw in (("block", {"multi_calib": False}), ("input", {"per_block": False}),
                        ("layer", {"per_block": False, "grouped": False}),
                        ("shared", {"multi_calib": True})):
            for ms, os_ in zip(mb.masks, mb.outputs):
                for m, o in zip(ms, os_):
                    m.zero_()
                    o.zero_()
            counts = pipeline.prune_model(mb, arg, batch_tokens, **kw)
            torch.cuda.synchronize()
            results[how] = ([[m.clone() for m in ms] for ms in mb.masks],
                            [[o.clone() for o in os_] for os_ in mb.outputs], counts)
        assert results["block"][2]["select"] == w.blocks                 # one launch per block
        assert results["input"][2]["select"] == w.blocks * len(w.input_widths())
        assert results["layer"][2]["select"] == w.blocks * len(w.layers)
        batches = w.tokens // batch_tokens
        assert results["block"][2]["calib"] == w.blocks * len(w.input_widths()) * batches
        assert results["shared"][2] == {"calib": w.blocks * batches, "finalize": w.blocks,
                                        "select": w.blocks}
        for how in ("input", "layer", "shared"):
            for b in range(w.blocks):
                for li in range(len(w.layers)):
                    assert torch.equal(results["block"][0][b][li], results[how][0][b][li])
                    assert torch.equal(results["block"][1][b][li].view(torch.int16),
                                       results[how][1][b][li].view(torch.int16))
        # the per-block pass under graph replay, with phase events, gives the same again
        graph, counts = pipeline.capture_model_graph(mb, arg, batch_tokens)
        for ms, os_ in zip(mb.masks, mb.outputs):
            for m, o in zip(ms, os_):
                m.zero_()
                o.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert counts["select"] == w.blocks
        events = []
        pipeline.prune_model(mb, arg, batch_tokens, events)
        torch.cuda.synchronize()
        assert sum(1 for k, *_ in events if k == "select") == w.blocks
        assert sum(u for k, _, _, u in events if k == "select") == w.total_weights()
        for b in range(w.blocks):
            for li in range(len(w.layers)):
                assert torch.equal(mb.masks[b][li], results["block"][0][b][li])
    finally:
        mb.close()


@pytest.mark.parametrize("name,arg", [("llama3-8b", 0.5), ("llama2-7b", (2, 4))])
def test_one_model_split_over_ranks_gives_the_single_rank_result(sp, name, arg):
    # the strong-scaling pass, its ranks played one after the other on this GPU (the block split
    # has no exchange; the token split of a single rank is the plain pass)
    from paper_2501_16376_b200 import pipeline, synth
    w = synth.scaled(synth.WORKLOADS[name], blocks=3, n_seqs=4, seq_len=128, shrink=16)
    mb = pipeline.allocate_model(w, "cuda")
    try:
        batch_tokens = 2 * w.seq_len
        pipeline.prune_model(mb, arg, batch_tokens)
        torch.cuda.synchronize()
        want_masks = [[m.clone() for m in ms] for ms in mb.masks]
        want_out = [[o.clone() for o in os_] for os_ in mb.outputs]

        def clear():
            for ms, os_ in zip(mb.masks, mb.outputs):
                for m, o in zip(ms, os_):
                    m.zero_()
                    o.zero_()

        def check():
            torch.cuda.synchronize()
            for b in range(w.blocks):
                for li in range(len(w.layers)):
                    assert torch.equal(mb.masks[b][li], want_masks[b][li])
                    assert torch.equal(mb.outputs[b][li].view(torch.int16),
                                       want_out[b][li].view(torch.int16))
        clear()
        selects = 0
        for rank in range(2):
            selects += pipeline.prune_model_split(mb, arg, batch_tokens, rank, 2, "blocks")["select"]
        assert selects == w.blocks
        check()
        clear()
        counts = pipeline.prune_model_split(mb, arg, batch_tokens, 0, 1, "tokens")
        assert counts["select"] == w.blocks
        check()
    finally:
        mb.close()


# ------------------------------------------------------------------ compressed 2:4 emission

@pytest.mark.parametrize("R,n,dtype", [(130, 2048, torch.float16), (65, 520, torch.bfloat16),
                                       (33, 1028, torch.float16), (3, 4, torch.float16)])
def test_compressed_24_matches_oracle_and_dense_path(sp, R, n, dtype):
    W = _gen(R * 5 + n, (R, n), dtype, 0.02)
    X = _activations(n + 7, 512, n, dtype)
    with _ctx_with_stats(sp, [X], n) as ctx:
        values, meta = ctx.sp_select_24_compressed(W)
        mask, dense = ctx.sp_select_nm(W, 2, 4)
        colsq = ctx.sp_get_stats()[0]
    sel = so.select_nm(P.bits(W), P.odtype(W), so.Stats(colsq.numpy().copy(), 1), 2, 4)
    v_want, m_want = so.compress_24(P.bits(W), sel.keep_bool(n))
    assert np.array_equal(P.bits(values), v_want)
    assert np.array_equal(P.mask_np(meta), m_want)
    # and it expands to exactly what the dense call wrote
    assert np.array_equal(so.expand_24(P.bits(values), P.mask_np(meta), n), P.bits(dense))


# ------------------------------------------------------------------ EWMA trace diagnostic

@pytest.mark.parametrize("s_update", [0, 1])     # the oracle's S_FROZEN, S_LITERAL_W2
def test_ewma_trace_matches_oracle_state(sp, s_update):
    R, n = 6, 1500
    W = _gen(71, (R, n), torch.float16, 0.02)
    colsq = np.random.default_rng(5).uniform(1.0, 2.0, n) * (1e-4 if s_update else 1e4)
    with sp.Context(n) as ctx:
        ctx.sp_set_stats(torch.from_numpy(colsq), 10)
        est, dev, L = ctx.sp_ewma_trace(W, sp.EwmaParams(
            0.125, 0.125, 0.5, sp.SP_S_LITERAL_W2 if s_update else sp.SP_S_FROZEN))
    st = so.Stats(colsq.copy(), 10)
    # the oracle's recorded threshold est - la*dev gives est (la = 0) and est - dev (la = 1);
    # with the S update on, decisions (hence S) depend on la, so compare at the la used
    ref = so.select_ewma(P.bits(W), so.F16, st, 0.5, s_update=s_update, want_trace=True)
    thr = est.cpu().numpy() - np.float32(0.5) * dev.cpu().numpy()
    assert np.array_equal(L.cpu().numpy(), ref.L)
    assert np.array_equal(thr.astype(np.float32), ref.thr)
    if not s_update:
        e0 = so.select_ewma(P.bits(W), so.F16, st, 0.0, s_update=0, want_trace=True).thr
        e1 = so.select_ewma(P.bits(W), so.F16, st, 1.0, s_update=0, want_trace=True).thr
        assert np.array_equal(est.cpu().numpy(), e0)
        assert np.array_equal((est.cpu().numpy() - dev.cpu().numpy()).astype(np.float32), e1)
    assert (dev[:, 0] == 0).all() and torch.equal(est[:, 0], L[:, 0])


# ------------------------------------------------------------------ grouped selection

def _group_matrices(dtype, n):
    """Four layers on one input: three that allow 16-byte access (one of them with a padded row
    stride) and one that does not (odd offset), so that the call needs more than one launch."""
    shapes = [(96, n), (33, n), (260, n), (17, n)]
    Ws = [_gen(500 + i, s, dtype, 0.02) for i, s in enumerate(shapes)]
    padded = torch.zeros(33, n + 24, dtype=dtype, device="cuda")
    padded[:, :n] = Ws[1]
    Ws[1] = padded[:, :n]                      # ld = n + 24
    buf = torch.zeros(17 * n + 1, dtype=dtype, device="cuda")
    buf[1:] = Ws[3].reshape(-1)
    Ws[3] = buf[1:].view(17, n)                # 2-byte aligned only
    return Ws


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_grouped_ewma_selection_equals_single_calls_and_oracle(sp, dtype):
    n = 1536
    Ws = _group_matrices(dtype, n)
    X = _activations(71, 2048, n, dtype)
    counters = sp.new_counters()
    with _ctx_with_stats(sp, [X], n) as ctx:
        masks, outs = ctx.sp_select_unstructured_group(Ws, 0.6, counters=counters)
        singles = [ctx.sp_select_unstructured(W, 0.6) for W in Ws]
        colsq = ctx.sp_get_stats()[0]
    st = so.Stats(colsq.numpy().copy(), 1)
    kept = 0
    for W, mask, out, (m1, o1) in zip(Ws, masks, outs, singles):
        assert torch.equal(mask, m1)
        assert torch.equal(out.contiguous().view(torch.int16), o1.contiguous().view(torch.int16))
        sel = so.select_unstructured(P.bits(W), P.odtype(W), st, 0.6, want_trace=True)
        P.check_selection(mask, out, W, sel, P.ewma_allowed_flips(sel))
        kept += int(so.unpack_mask(P.mask_np(mask), n).sum())
    assert int(counters[sp.SP_COUNTER_KEPT]) == kept


@pytest.mark.parametrize("N,M", [(2, 4), (4, 8)])
def test_grouped_nm_selection_equals_single_calls_and_oracle(sp, N, M):
    n = 1536
    Ws = _group_matrices(torch.float16, n)
    X = _activations(72, 2048, n, torch.float16)
    with _ctx_with_stats(sp, [X], n) as ctx:
        masks, outs = ctx.sp_select_nm_group(Ws, N, M)
        # a group whose members ask for different outputs (mask only / in place)
        clones = [W.clone() for W in Ws]
        masks2, outs2 = ctx.sp_select_nm_group(clones[:2], N, M, inplace=True)
        colsq = ctx.sp_get_stats()[0]
    st = so.Stats(colsq.numpy().copy(), 1)
    for i, (W, mask, out) in enumerate(zip(Ws, masks, outs)):
        sel = so.select_nm(P.bits(W), so.F16, st, N, M)
        P.check_selection(mask, out, W, sel, None, strict=True)
        if i < 2:
            assert torch.equal(mask, masks2[i]) and outs2[i].data_ptr() == clones[i].data_ptr()
            assert np.array_equal(P.bits(clones[i]), sel.W_out)


@pytest.mark.parametrize("dtype,widths", [
    (torch.float16, [512, 2048, 1024, 2048]),        # whole tiles everywhere, one context twice
    (torch.bfloat16, [1536, 520, 4096, 1001]),       # ragged tiles; 1001: no 16-byte access
])
def test_multi_context_ewma_selection_equals_single_calls_and_oracle(sp, dtype, widths):
    # one call, matrices that read different inputs (different widths and statistics)
    rows = [37, 130, 64, 9, 21]
    ctxs, Ws, owner = {}, [], []
    for k, n in enumerate(widths):
        if n not in ctxs:
            ctxs[n] = _ctx_with_stats(sp, [_activations(90 + k, 1024, n, dtype)], n)
        Ws.append(_gen(700 + k, (rows[k], n), dtype, 0.02))
        owner.append(ctxs[n])
    Ws.append(_gen(777, (rows[4], widths[0]), dtype, 0.02))   # a second matrix on the first input
    owner.append(ctxs[widths[0]])
    counters = sp.new_counters()
    prm = sp.EwmaParams(0.125, 0.125, 0.2, sp.SP_S_GATED)
    try:
        masks, outs = sp.sp_select_unstructured_multi(owner, Ws, params=prm, counters=counters)
        kept = 0
        for ctx, W, mask, out in zip(owner, Ws, masks, outs):
            n = W.shape[1]
            m1, o1 = ctx.sp_select_unstructured(W, params=prm)
            assert torch.equal(mask, m1)
            assert torch.equal(out.contiguous().view(torch.int16), o1.contiguous().view(torch.int16))
            st = so.Stats(ctx.sp_get_stats()[0].numpy().copy(), 1)
            sel = so.select_ewma(P.bits(W), P.odtype(W), st, 0.2, want_trace=True)
            P.check_selection(mask, out, W, sel, P.ewma_allowed_flips(sel))
            kept += int(so.unpack_mask(P.mask_np(mask), n).sum())
        assert int(counters[sp.SP_COUNTER_KEPT]) == kept
        # the sparsity form, and the sequential modes through the same entry point
        m2, o2 = sp.sp_select_unstructured_multi(owner[:2], Ws[:2], 0.6)
        for ctx, W, mask, out in zip(owner[:2], Ws[:2], m2, o2):
            m1, o1 = ctx.sp_select_unstructured(W, 0.6)
            assert torch.equal(mask, m1) and torch.equal(out.view(torch.int16), o1.view(torch.int16))
        lit = sp.EwmaParams(0.125, 0.125, 0.2, sp.SP_S_LITERAL_W2)
        m3, o3 = sp.sp_select_unstructured_multi(owner[:3], Ws[:3], params=lit)
        for ctx, W, mask, out in zip(owner[:3], Ws[:3], m3, o3):
            m1, o1 = ctx.sp_select_unstructured(W, params=lit)
            assert torch.equal(mask, m1) and torch.equal(out.view(torch.int16), o1.view(torch.int16))
    finally:
        for ctx in ctxs.values():
            ctx.close()


@pytest.mark.parametrize("dtype,widths,N,M", [
    (torch.float16, [512, 2048, 1024, 2048], 2, 4),     # whole strips everywhere
    (torch.bfloat16, [1536, 520, 4096, 1004], 2, 4),    # ragged strips; 1004: no 16-byte access
    (torch.float16, [1024, 264, 2048, 512], 4, 8),
])
def test_multi_context_nm_selection_equals_single_calls_and_oracle(sp, dtype, widths, N, M):
    rows = [37, 130, 64, 9, 21]
    ctxs, Ws, owner = {}, [], []
    for k, n in enumerate(widths):
        if n not in ctxs:
            ctxs[n] = _ctx_with_stats(sp, [_activations(190 + k, 1024, n, dtype)], n)
        Ws.append(_gen(800 + k, (rows[k], n), dtype, 0.02))
        owner.append(ctxs[n])
    Ws.append(_gen(877, (rows[4], widths[0]), dtype, 0.02))
    owner.append(ctxs[widths[0]])
    try:
        masks, outs = sp.sp_select_nm_multi(owner, Ws, N, M)
        for ctx, W, mask, out in zip(owner, Ws, masks, outs):
            m1, o1 = ctx.sp_select_nm(W, N, M)
            assert torch.equal(mask, m1)
            assert torch.equal(out.contiguous().view(torch.int16), o1.contiguous().view(torch.int16))
            st = so.Stats(ctx.sp_get_stats()[0].numpy().copy(), 1)
            sel = so.select_nm(P.bits(W), P.odtype(W), st, N, M)
            P.check_selection(mask, out, W, sel, None, strict=True)
        # members that ask for different outputs (in place, no mask): launches of their own
        clones = [W.clone() for W in Ws[:3]]
        m2, o2 = sp.sp_select_nm_multi(owner[:3], clones, N, M, inplace=True, want_mask=False)
        for i in range(3):
            assert m2[i] is None and o2[i].data_ptr() == clones[i].data_ptr()
            assert torch.equal(clones[i].view(torch.int16), outs[i].view(torch.int16))
    finally:
        for ctx in ctxs.values():
            ctx.close()


def test_multi_context_selection_rejects_bad_calls(sp):
    W = _gen(3, (8, 512), torch.float16, 0.02)
    X = _activations(4, 256, 512, torch.float16)
    with _ctx_with_stats(sp, [X], 512) as ctx, sp.Context(512) as empty, sp.Context(1024) as wide:
        with pytest.raises(sp.SpError) as e:
            sp.sp_select_unstructured_multi([ctx] * (sp.SP_MAX_MULTI + 1),
                                            [W] * (sp.SP_MAX_MULTI + 1), 0.5)
        assert e.value.status == sp.SP_ERR_INVALID_ARG
        with pytest.raises(sp.SpError) as e:
            sp.sp_select_unstructured_multi([ctx, empty], [W, W], 0.5)     # no calibration data
        assert e.value.status == sp.SP_ERR_STATE
        with pytest.raises(sp.SpError) as e:
            sp.sp_select_unstructured_multi([ctx, wide], [W, W], 0.5)      # W narrower than d_in
        assert e.value.status == sp.SP_ERR_SHAPE
        with pytest.raises(sp.SpError) as e:
            sp.sp_select_nm_multi([ctx, empty], [W, W], 2, 4)
        assert e.value.status == sp.SP_ERR_STATE
        with pytest.raises(sp.SpError) as e:
            sp.sp_select_nm_multi([ctx], [W], 4, 4)
        assert e.value.status == sp.SP_ERR_INVALID_ARG
    W6 = _gen(5, (8, 516), torch.float16, 0.02)
    with _ctx_with_stats(sp, [_activations(6, 64, 516, torch.float16)], 516) as c6:
        with pytest.raises(sp.SpError) as e:
            sp.sp_select_nm_multi([c6], [W6], 4, 8)                        # 516 % 8 != 0
        assert e.value.status == sp.SP_ERR_SHAPE


def test_grouped_selection_rejects_bad_groups(sp):
    n = 512
    W = _gen(3, (8, n), torch.float16, 0.02)
    X = _activations(4, 256, n, torch.float16)
    with _ctx_with_stats(sp, [X], n) as ctx:
        with pytest.raises(sp.SpError) as e:
            ctx.sp_select_nm_group([W] * (sp.SP_MAX_GROUP + 1), 2, 4)
        assert e.value.status == sp.SP_ERR_INVALID_ARG
        with pytest.raises(sp.SpError) as e:
            ctx.sp_select_unstructured_group([W, W.to(torch.bfloat16)], 0.5)
        assert e.value.status == sp.SP_ERR_DTYPE


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_multi_input_calibration_matches_single_calls_and_the_oracle(sp, dtype):
    # four inputs of different widths (one ragged strip, one without 16-byte access, one with a
    # padded row stride), three batches of different lengths, one launch per batch
    widths = [1024, 520, 1001, 4096]
    lengths = [700, 64, 1300]
    Xs = {n: _activations(300 + n, sum(lengths), n, dtype) for n in widths}
    padded = torch.zeros(sum(lengths), 520 + 24, dtype=dtype, device="cuda")
    padded[:, :520] = Xs[520]
    Xs[520] = padded[:, :520]
    multi = {n: sp.Context(n) for n in widths}
    single = {n: sp.Context(n) for n in widths}
    try:
        t0 = 0
        launches = sp.sp_launch_count()
        for T in lengths:
            sp.sp_calib_accumulate_multi([multi[n] for n in widths],
                                         [Xs[n][t0:t0 + T] for n in widths])
            t0 += T
        assert sp.sp_launch_count() - launches == 2 * len(lengths)   # 3 inputs together + 1001 alone
        t0 = 0
        for T in lengths:
            for n in widths:
                single[n].sp_calib_accumulate(Xs[n][t0:t0 + T])
            t0 += T
        launches = sp.sp_launch_count()
        sp.sp_finalize_multi([multi[n] for n in widths] + [multi[1024]])
        assert sp.sp_launch_count() - launches == 1
        sp.sp_finalize_multi([multi[n] for n in widths])              # nothing pending: no launch
        assert sp.sp_launch_count() - launches == 1
        for n in widths:
            cm, Sm, fm, tm = multi[n].sp_get_stats()
            cs, Ss, fs, ts = single[n].sp_get_stats()
            assert tm == ts == sum(lengths)
            # the same sums up to the grouping of the binary32 partial sums (slabs cut differently)
            assert P.rel_err(cm.numpy(), cs.numpy()) <= 1e-7 and abs(Sm - Ss) <= 1e-7 * Ss
            assert P.rel_err(fm.numpy(), fs.numpy()) <= 1e-6
            st = P.oracle_stats([Xs[n]], n)
            assert P.rel_err(cm.numpy(), st.colsq) <= P.SCORE_RTOL
            assert np.array_equal(fm.numpy(), so.Stats(cm.numpy().copy(), tm).channel_factor32())
        # the EWMA kernel's own copy of the factors comes out of the multi finalisation too
        W = _gen(11, (40, 1024), dtype, 0.02)
        m1, o1 = multi[1024].sp_select_unstructured(W, 0.5)
        own = so.Stats(multi[1024].sp_get_stats()[0].numpy().copy(), 1)
        sel = so.select_unstructured(P.bits(W), P.odtype(W), own, 0.5, want_trace=True)
        P.check_selection(m1, o1, W, sel, P.ewma_allowed_flips(sel))
        # and the sums are reproducible: the same calls again give the same bits
        again = {n: sp.Context(n) for n in widths}
        t0 = 0
        for T in lengths:
            sp.sp_calib_accumulate_multi([again[n] for n in widths],
                                         [Xs[n][t0:t0 + T] for n in widths])
            t0 += T
        for n in widths:
            assert torch.equal(again[n].sp_get_stats()[0], multi[n].sp_get_stats()[0])
            again[n].close()
    finally:
        for c in list(multi.values()) + list(single.values()):
            c.close()


def test_multi_input_calibration_rejects_bad_calls(sp):
    X = _activations(5, 64, 512, torch.float16)
    with sp.Context(512) as a, sp.Context(512) as b, sp.Context(256) as c:
        with pytest.raises(sp.SpError) as e:
            sp.sp_calib_accumulate_multi([a, a], [X, X])                  # the same sums twice
        assert e.value.status == sp.SP_ERR_INVALID_ARG
        with pytest.raises(sp.SpError) as e:
            sp.sp_calib_accumulate_multi([a, c], [X, X])                  # width mismatch
        assert e.value.status == sp.SP_ERR_SHAPE
        with pytest.raises(sp.SpError) as e:
            sp.sp_calib_accumulate_multi([a, b], [X, X.to(torch.bfloat16)])
        assert e.value.status == sp.SP_ERR_DTYPE
        with pytest.raises(sp.SpError) as e:
            sp.sp_finalize_multi([a, b])                                  # no calibration data
        assert e.value.status == sp.SP_ERR_STATE
        sp.sp_calib_accumulate_multi([a, b], [X, X[:0]])                  # an empty batch is skipped
        assert a.sp_get_stats()[3] == 64
        with pytest.raises(sp.SpError):
            b.sp_get_stats()


def test_calls_on_two_user_streams_at_once(sp):
    # two layer inputs, each calibrated and pruned on a stream of its own, the activations written
    # by the kernel that precedes the first library call on that stream (ordinary stream order,
    # no promise about X)
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    shapes = [(2048, 4096, 300), (1536, 1000, 257)]           # (d_in, tokens, rows)
    seeds = [(1.0 + torch.arange(t * n, device="cuda", dtype=torch.float32).reshape(t, n) % 7)
             for n, t, _ in shapes]
    Ws = [_gen(40 + i, (r, n), torch.float16, 0.02) for i, (n, t, r) in enumerate(shapes)]
    torch.cuda.synchronize()
    ctxs = [sp.Context(n) for n, _, _ in shapes]
    got = []
    try:
        Xs = []
        for s, ctx, base, W in zip(streams, ctxs, seeds, Ws):
            with torch.cuda.stream(s):
                X = (base * 0.25 - 0.5).to(torch.float16)     # written on s, right before its use
                Xs.append(X)
                ctx.sp_calib_accumulate(X, stream=s)
                got.append((ctx.sp_select_nm(W, 2, 4, stream=s),
                            ctx.sp_select_unstructured(W, 0.5, stream=s)))
        for s in streams:
            s.synchronize()
        for ctx, X, W, ((m_nm, o_nm), (m_e, o_e)), (n, _, _) in zip(ctxs, Xs, Ws, got, shapes):
            st = P.oracle_stats([X], n)
            colsq = ctx.sp_get_stats()[0]
            assert P.rel_err(colsq.numpy(), st.colsq) <= P.SCORE_RTOL
            own = so.Stats(colsq.numpy().copy(), 1)
            P.check_selection(m_nm, o_nm, W, so.select_nm(P.bits(W), so.F16, own, 2, 4), None,
                              strict=True)
            sel = so.select_unstructured(P.bits(W), so.F16, own, 0.5, want_trace=True)
            P.check_selection(m_e, o_e, W, sel, P.ewma_allowed_flips(sel))
    finally:
        for c in ctxs:
            c.close()


@pytest.mark.parametrize("multi", [False, True])
def test_calibration_waits_for_a_library_kernel_that_writes_its_input(sp, multi):
    # The producer is one of the library's own kernels, which lets its successor start early;
    # without the X_COMPLETE promise the accumulate kernel must still see the finished matrix.
    # Replayed as a CUDA graph, where launches follow each other closely enough for a consumer
    # that did not wait to read the stale fill value (with the promise given wrongly it does).
    n, R = 4096, 8192
    A = _gen(61, (R, n), torch.float16, 0.5)
    stats = _activations(62, 512, n, torch.float16)
    with sp.Context(n) as maker, sp.Context(n) as ctx, sp.Context(n) as other:
        maker.sp_calib_accumulate(stats)
        maker.sp_score(None)
        X = torch.full((R, n), 100.0, dtype=torch.float16, device="cuda")   # stale value: obvious

        def producer_then_consumer():
            ctx.sp_calib_reset()
            other.sp_calib_reset()
            maker.sp_select_nm(A, 2, 4, W_out=X, want_mask=False)
            if multi:
                sp.sp_calib_accumulate_multi([ctx, other], [X, X[:R // 2]])
                sp.sp_finalize_multi([ctx, other])
            else:
                ctx.sp_calib_accumulate(X)
                ctx.sp_score(None)
        producer_then_consumer()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            producer_then_consumer()
        for _ in range(4):
            X.fill_(100.0)
            torch.cuda.synchronize()
            graph.replay()
            torch.cuda.synchronize()
            colsq = ctx.sp_get_stats()[0]
            st = P.oracle_stats([X], n)
            assert float(st.colsq.max()) < 100.0 ** 2 * 16    # nothing of the fill is left in X
            assert P.rel_err(colsq.numpy(), st.colsq) <= P.SCORE_RTOL
            if multi:
                half = other.sp_get_stats()[0]
                assert P.rel_err(half.numpy(), P.oracle_stats([X[:R // 2]], n).colsq) <= P.SCORE_RTOL


def test_calib_accumulate_ex_flag_changes_ordering_only(sp):
    n = 1000
    X = _activations(81, 3000, n, torch.float16)
    torch.cuda.synchronize()                      # X is complete: the promise of the flag holds
    with sp.Context(n) as a, sp.Context(n) as b:
        for t0 in range(0, 3000, 1000):
            a.sp_calib_accumulate(X[t0:t0 + 1000])
            b.sp_calib_accumulate(X[t0:t0 + 1000], x_complete=True)
        ca, Sa, fa, _ = a.sp_get_stats()
        cb, Sb, fb, _ = b.sp_get_stats()
        assert torch.equal(ca, cb) and Sa == Sb and torch.equal(fa, fb)
        st = P.oracle_stats([X], n)
        assert P.rel_err(ca.numpy(), st.colsq) <= P.SCORE_RTOL
        bad = sp.lib.sp_calib_accumulate_ex(a._h, X.data_ptr(), sp.SP_F16, 1000, n, 2, None)
        assert bad == sp.SP_ERR_INVALID_ARG


# ------------------------------------------------------------------ non-finite scores

def _golden_nonfinite():
    import os
    out = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "nonfinite_scores.txt")) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                key, *vals = line.split()
                out[key] = vals
    return out


def _row16(vals, n, dtype=torch.float16):
    row = torch.zeros(n, dtype=torch.float32)
    row[:len(vals)] = torch.tensor([float(v) for v in vals])
    return row.to(dtype)


@pytest.mark.parametrize("n", [8, 512, 520, 12])       # stream kernel (whole / ragged), general
def test_nm_with_nan_and_infinite_scores_hand_cases_and_oracle(sp, n):
    g = _golden_nonfinite()
    # all channels alike: NaN / +inf weights inside the first two groups
    W = torch.stack([_row16(g["nm_a_weights"], n), _row16(g["nm_a_weights"][4:], n)]).cuda()
    with sp.Context(n) as ctx:
        ctx.sp_set_stats(torch.ones(n, dtype=torch.float64), 4)
        mask, out = ctx.sp_select_nm(W, 2, 4)
    sel = so.select_nm(P.bits(W), so.F16, so.Stats(np.ones(n), 4), 2, 4)
    P.check_selection(mask, out, W, sel, None, strict=True)
    keep = so.unpack_mask(P.mask_np(mask), n)
    want = np.array([c == "1" for c in g["nm_a_keep"][0]])
    assert np.array_equal(keep[0, :8], want) and np.array_equal(keep[1, :4], want[4:])
    # one live channel: c_0 = +inf; w_0 = 0 gives a NaN score, w_0 = 0.5 an infinite one
    colsq = np.zeros(n)
    colsq[0] = 1.0
    W = torch.stack([_row16(g["nm_b_row0"], n), _row16(g["nm_b_row1"], n)]).cuda()
    with sp.Context(n) as ctx:
        ctx.sp_set_stats(torch.from_numpy(colsq), 4)
        mask, out = ctx.sp_select_nm(W, 2, 4)
        L = ctx.sp_score(W)
    sel = so.select_nm(P.bits(W), so.F16, so.Stats(colsq.copy(), 4), 2, 4, want_trace=True)
    P.check_selection(mask, out, W, sel, None, strict=True)
    keep = so.unpack_mask(P.mask_np(mask), n)
    assert np.array_equal(keep[0, :4], np.array([c == "1" for c in g["nm_b_keep0"][0]]))
    assert np.array_equal(keep[1, :4], np.array([c == "1" for c in g["nm_b_keep1"][0]]))
    Lc = L.cpu().numpy()
    assert np.isnan(Lc[0, 0]) and np.isinf(Lc[1, 0])
    assert np.array_equal(np.isnan(Lc), np.isnan(sel.L))
    assert np.array_equal(Lc[~np.isnan(Lc)], sel.L[~np.isnan(sel.L)])


@pytest.mark.parametrize("n", [6, 8, 1024, 1030])       # general kernel, pair kernel, several tiles
@pytest.mark.parametrize("mode", ["gated", "frozen", "literal"])
def test_ewma_with_nan_and_infinite_scores_hand_cases_and_oracle(sp, n, mode):
    g = _golden_nonfinite()
    s_lib = {"gated": sp.SP_S_GATED, "frozen": sp.SP_S_FROZEN, "literal": sp.SP_S_LITERAL_W2}[mode]
    s_ora = so.S_FROZEN if mode == "frozen" else so.S_LITERAL_W2
    rows = [_row16(g["ewma_a_weights"], n), _row16(g["ewma_b_weights"], n)]
    if n > 600:        # the same events deep inside a row: after a tile of ordinary weights
        body = _gen(61, (2, n), torch.float16, 0.02).cpu()
        body[0, 600:606] = rows[0][:6]
        body[1, 700:706] = rows[1][:6]
        rows = [body[0], body[1]]
    W = torch.stack(rows).cuda()
    colsq = np.ones(n) * 1e6                              # calibration scale: S cannot move ...
    with sp.Context(n) as ctx:
        ctx.sp_set_stats(torch.from_numpy(colsq), 4)
        counters = sp.new_counters()
        mask, out = ctx.sp_select_unstructured(W, params=_ewma_params(sp, 0.5, s_update=s_lib),
                                               counters=counters)
    sel = so.select_ewma(P.bits(W), so.F16, so.Stats(colsq.copy(), 4), 0.5, s_update=s_ora,
                         want_trace=True)
    keep = so.unpack_mask(P.mask_np(mask), n)
    want = sel.keep_bool(n)
    if n <= 8:
        for r, key in enumerate(("ewma_a_keep", "ewma_b_keep")):
            assert np.array_equal(keep[r, :6], np.array([c == "1" for c in g[key][0]]))
    # before the non-finite weight the usual band rule; from it on everything is kept
    first = 2 if n <= 8 else None
    starts = [first, first] if first is not None else [602, 702]
    for r in range(2):
        assert keep[r, starts[r]:].all() and want[r, starts[r]:].all()
        d = keep[r, :starts[r]] != want[r, :starts[r]]
        assert not (d & ~P.ewma_allowed_flips(sel)[r, :starts[r]]).any() and d.sum() <= 1
    assert np.array_equal(P.bits(out), np.where(keep, P.bits(W), 0))
    assert int(counters[sp.SP_COUNTER_KEPT]) == int(keep.sum())
    if mode == "gated":                                   # ... but NaN / inf rows go the exact way
        assert int(counters[sp.SP_COUNTER_S_HAZARD]) == 2


@pytest.mark.parametrize("target", [0.3, 0.5, 0.55, 0.65, 0.8, 0.9])
def test_search_la_reports_exactly_what_the_selection_then_prunes(sp, target):
    R, n = 256, 2048
    W = _gen(95, (R, n), torch.bfloat16, 0.02)
    X = _activations(96, 2048, n, torch.bfloat16)
    with _ctx_with_stats(sp, [X], n) as ctx:
        la, achieved = ctx.sp_search_la(W, target, iterations=20)
        mask, _ = ctx.sp_select_unstructured(W, params=_ewma_params(sp, la, s_update=sp.SP_S_FROZEN))
        mask_g, _ = ctx.sp_select_unstructured(W, params=_ewma_params(sp, la))
    pruned = 1.0 - so.unpack_mask(P.mask_np(mask), n).mean(dtype=np.float64)
    assert pruned == achieved                 # the same constants in the count and in the selection
    assert torch.equal(mask, mask_g)
    assert abs(achieved - target) < 2e-3


@pytest.mark.parametrize("R,n,misalign", [(96, 640, False), (40, 1032, False), (33, 648, True)])
def test_x2_reading_of_the_S_update_is_bit_exact(sp, R, n, misalign):
    """SP_S_READING_X2 ("S = S - x_i^2"): sequential kernels, bit-exact against the oracle's mode
    of the same name; the reading changes S by tens of percent, so it differs from the others."""
    W = _gen(191 + n, (R, n), torch.float16, 0.02)
    if misalign:
        buf = torch.zeros(R * n + 1, dtype=W.dtype, device=W.device)
        buf[1:] = W.reshape(-1)
        W = buf[1:].view(R, n)
    X = _activations(192, 1024, n, torch.float16)
    counters = sp.new_counters()
    with _ctx_with_stats(sp, [X], n) as ctx:
        mask, out = ctx.sp_select_unstructured(
            W, params=_ewma_params(sp, 0.5, s_update=sp.SP_S_READING_X2), counters=counters)
        est, dev, L = ctx.sp_ewma_trace(W[:4].contiguous(),
                                        sp.EwmaParams(0.125, 0.125, 0.5, sp.SP_S_READING_X2))
        colsq = ctx.sp_get_stats()[0]
    st = so.Stats(colsq.numpy().copy(), 1)
    sel = so.select_ewma(P.bits(W), so.F16, st, 0.5, s_update=so.S_READING_X2, want_trace=True)
    P.check_selection(mask, out, W, sel, None, strict=True)
    assert int(counters[sp.SP_COUNTER_KEPT]) == int(sel.keep_bool(n).sum())
    assert np.array_equal(L.cpu().numpy(), sel.L[:4])
    thr = est.cpu().numpy() - np.float32(0.5) * dev.cpu().numpy()
    assert np.array_equal(thr, sel.thr[:4])
    other = so.select_ewma(P.bits(W), so.F16, st, 0.5, s_update=so.S_LITERAL_W2)
    assert not np.array_equal(other.mask, sel.mask)


def _golden_trace(name):
    import os
    g = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                key, *vals = line.split()
                g[key] = vals
    return g


@pytest.mark.parametrize("name", ["ewma_hand_trace.txt", "ewma_hand_trace_alpha_ne_beta.txt"])
@pytest.mark.parametrize("pad", [0, 2, 10])     # 6 columns: general kernel; 8, 16: paired-chain kernel
def test_fixed_S_hand_traces_through_the_scan_kernels(sp, name, pad):
    # the paper-derived hand evaluations, not the oracle, are the expected values here
    g = _golden_trace(name)
    w = [float(v) for v in g["w"]] + [0.0] * pad          # extra columns: w = 0, after the trace
    colsq = [float(v) for v in g["colsq"]] + [0.0] * pad
    n0, n = len(g["w"]), len(w)
    W = torch.tensor([w, w], dtype=torch.float16, device="cuda")
    prm = sp.EwmaParams(float(g["alpha"][0]), float(g["beta"][0]), float(g["la"][0]), sp.SP_S_FROZEN)
    with sp.Context(n) as ctx:
        ctx.sp_set_stats(torch.tensor(colsq, dtype=torch.float64), 1)
        mask, out = ctx.sp_select_unstructured(W, params=prm)
        est, dev, L = ctx.sp_ewma_trace(W, prm)
    keep = so.unpack_mask(P.mask_np(mask), n)
    want = [int(v) for v in g["keep"]]
    assert keep[0, :n0].astype(int).tolist() == want and keep[1, :n0].astype(int).tolist() == want
    assert out[0, :n0].float().cpu().tolist() == [wi if k else 0.0 for wi, k in zip(w, want)]
    assert L.cpu().numpy()[0, :n0].tolist() == [float(v) for v in g["L"]]
    thr = (est - prm.la * dev).cpu().numpy()[0, :n0].tolist()
    assert thr == [float(v) for v in g["thr"]]


@pytest.mark.parametrize("mode", ["literal", "gated"])
def test_literal_S_hand_trace_through_the_library(sp, mode):
    # S = 16 and w^2 up to 64: every pruned weight moves S, so the default (gated) call must
    # give the printed algorithm's hand-evaluated decisions too
    g = _golden_trace("ewma_hand_trace_literal_s.txt")
    W = torch.tensor([[float(v) for v in g["w"]]], dtype=torch.float16, device="cuda")
    n = W.shape[1]
    prm = sp.EwmaParams(float(g["alpha"][0]), float(g["beta"][0]), float(g["la"][0]),
                        sp.SP_S_LITERAL_W2 if mode == "literal" else sp.SP_S_GATED)
    with sp.Context(n) as ctx:
        ctx.sp_set_stats(torch.tensor([float(v) for v in g["colsq"]], dtype=torch.float64), 1)
        mask, out = ctx.sp_select_unstructured(W, params=prm)
        est, dev, L = ctx.sp_ewma_trace(W, prm)
    keep = so.unpack_mask(P.mask_np(mask), n)[0].astype(int).tolist()
    assert keep == [int(v) for v in g["keep"]]
    thr = (est - prm.la * dev).cpu().numpy()[0].tolist()
    assert thr == [float(v) for v in g["thr"]]
    assert np.allclose(L.cpu().numpy()[0], [float(v) for v in g["L"]], rtol=3e-7)


def test_x2_reading_hand_trace_through_the_library(sp):
    import os
    g = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "ewma_hand_trace_x2_reading.txt")) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                key, *vals = line.split()
                g[key] = vals
    W = torch.tensor([[float(v) for v in g["w"]]], dtype=torch.float16, device="cuda")
    n = W.shape[1]
    prm = sp.EwmaParams(float(g["alpha"][0]), float(g["beta"][0]), float(g["la"][0]),
                        sp.SP_S_READING_X2)
    with sp.Context(n) as ctx:
        ctx.sp_set_stats(torch.tensor([float(v) for v in g["colsq"]], dtype=torch.float64), 1)
        mask, out = ctx.sp_select_unstructured(W, params=prm)
        est, dev, L = ctx.sp_ewma_trace(W, prm)
    keep = so.unpack_mask(P.mask_np(mask), n)[0].astype(int).tolist()
    assert keep == [int(v) for v in g["keep"]]
    assert L.cpu().numpy()[0].tolist() == [float(v) for v in g["L"]]
    thr = (est - prm.la * dev).cpu().numpy()[0].tolist()
    assert thr == [float(v) for v in g["thr"]]


# ------------------------------------------------------------------ fix-point sweeps (SP_S_LITERAL_SCAN)

@pytest.mark.parametrize("R,n,mult,misalign", [
    (64, 2048, 1e9, False),      # calibration scale: S cannot move, one sweep per tile
    (64, 2048, 8.0, False),      # S = 8 x the sum of the pruned w^2 of a row: S moves by 12 %
    (64, 2056, 1.5, False),      # ... S shrinks to a third along the row; ragged last tile
    (33, 1000, 1.5, True),       # element-wise loads
    (48, 640, 1.0, False),       # S comes down to a few percent of its start at the row's end
])
def test_literal_scan_matches_the_oracle_literal_mode(sp, R, n, mult, misalign):
    """SP_S_LITERAL_SCAN against the oracle's literal evaluation of Algorithm 1, under the band
    rule (the sweeps re-associate).  Not covered: statistics so small that S passes through zero
    inside a row - there the factor 1/(1 - x^2/S) has a pole, and two evaluations that round S
    differently (successive subtractions, prefix sum) legitimately decide differently."""
    W = _gen(301 + n, (R, n), torch.float16, 0.02)
    if misalign:
        buf = torch.zeros(R * n + 1, dtype=W.dtype, device=W.device)
        buf[1:] = W.reshape(-1)
        W = buf[1:].view(R, n)
    colsq = np.random.default_rng(7).uniform(1.0, 2.0, n)
    colsq *= mult * n * 3.9e-5 / colsq.sum()      # a row's pruned w^2 add up to about n * 3.9e-5
    counters = sp.new_counters()
    with sp.Context(n) as ctx:
        ctx.sp_set_stats(torch.from_numpy(colsq), 10)
        mask, out = ctx.sp_select_unstructured(
            W, params=_ewma_params(sp, 0.5, s_update=sp.SP_S_LITERAL_SCAN), counters=counters)
    st = so.Stats(colsq.copy(), 10)
    lit = so.select_ewma(P.bits(W), so.F16, st, 0.5, s_update=so.S_LITERAL_W2, want_trace=True)
    fro = so.select_ewma(P.bits(W), so.F16, st, 0.5, s_update=so.S_FROZEN)
    keep = so.unpack_mask(P.mask_np(mask), n)
    want = lit.keep_bool(n)
    diff = keep != want
    assert not (diff & ~P.ewma_allowed_flips(lit)).any()
    assert diff.sum() <= 2, diff.sum()
    assert np.array_equal(P.bits(out), np.where(keep, P.bits(W), 0))
    assert int(counters[sp.SP_COUNTER_KEPT]) == int(keep.sum())
    if mult <= 1.0:
        assert not np.array_equal(lit.mask, fro.mask)      # only here does the update change decisions
    if mult >= 8.0:
        assert int(counters[sp.SP_COUNTER_S_HAZARD]) == 0  # every tile settled
    print("mult", mult, "rows handed to the walk:", int(counters[sp.SP_COUNTER_S_HAZARD]), "of", R)
