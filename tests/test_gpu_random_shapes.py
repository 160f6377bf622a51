"""Randomised small-shape parity: odd widths, padded and misaligned rows, both 16-bit types,
in-place and out-of-place, every selection mode - each case against the oracle fed with the
same statistics (bit-exact for N:M, apply and the sequential EWMA path; band rule for the scan)."""
import numpy as np
import pytest
import torch

from oracle import swiftprune_oracle as so
from tests import parity as P

pytestmark = pytest.mark.gpu

WIDTHS = [1, 3, 4, 8, 12, 24, 31, 32, 40, 100, 248, 256, 264, 300, 511, 512, 520, 777, 1024, 1032]


def _case(rng, need_multiple=1):
    while True:
        n = int(rng.choice(WIDTHS))
        if n % need_multiple == 0:
            break
    R = int(rng.integers(1, 70))
    pad = int(rng.choice([0, 0, 1, 3, 8, 16]))
    off = int(rng.choice([0, 0, 1, 8]))
    dtype = torch.float16 if rng.random() < 0.5 else torch.bfloat16
    g = torch.Generator(device="cuda").manual_seed(int(rng.integers(1 << 30)))
    big = (torch.randn(R, n + pad + off, generator=g, device="cuda") * 0.02).to(dtype)
    W = big[:, off:off + n]
    colsq = rng.uniform(0.5, 2.0, n) * 1e4
    colsq[rng.integers(0, n)] *= 300.0
    return R, n, W, big, colsq


@pytest.fixture(scope="module")
def sp():
    from paper_2501_16376_b200 import binding
    return binding


@pytest.mark.parametrize("seed", range(24))
def test_random_nm_cases(sp, seed):
    rng = np.random.default_rng(1000 + seed)
    N, M = [(2, 4), (4, 8), (1, 4), (3, 4), (2, 8), (7, 8)][seed % 6]
    R, n, W, big, colsq = _case(rng, need_multiple=M)
    W_ref = W.clone()
    inplace = bool(rng.random() < 0.3)
    with sp.Context(n) as ctx:
        ctx.sp_set_stats(torch.from_numpy(colsq), 5)
        mask, out = ctx.sp_select_nm(W, N, M, inplace=inplace)
        sel = so.select_nm(P.bits(W_ref), P.odtype(W_ref), so.Stats(colsq.copy(), 5), N, M)
        P.check_selection(mask, out, W_ref, sel, None, strict=True)
        redo = sp.sp_apply_mask(W_ref, mask)
        assert np.array_equal(P.bits(redo), sel.W_out)
        if (N, M) == (2, 4):
            values, meta = ctx.sp_select_24_compressed(W_ref)
            v, m = so.compress_24(P.bits(W_ref), sel.keep_bool(n))
            assert np.array_equal(P.bits(values), v) and np.array_equal(P.mask_np(meta), m)


@pytest.mark.parametrize("seed", range(24))
def test_random_ewma_cases(sp, seed):
    rng = np.random.default_rng(2000 + seed)
    R, n, W, big, colsq = _case(rng)
    W_ref = W.clone()
    la = float(rng.choice([0.5, 0.2, -0.2, -0.9, 2.0]))
    alpha = float(rng.choice([0.125, 0.25, 0.0625]))
    beta = float(rng.choice([0.125, 0.25]))
    literal = seed % 3 == 0
    inplace = bool(rng.random() < 0.3)
    counters = sp.new_counters() if seed % 2 else None
    with sp.Context(n) as ctx:
        ctx.sp_set_stats(torch.from_numpy(colsq), 5)
        params = sp.EwmaParams(alpha, beta, la, 1 if literal else 0)
        mask, out = ctx.sp_select_unstructured(W, params=params, inplace=inplace, counters=counters)
        sel = so.select_ewma(P.bits(W_ref), P.odtype(W_ref), so.Stats(colsq.copy(), 5), la, alpha,
                             beta, s_update=so.S_LITERAL_W2 if literal else so.S_FROZEN,
                             want_trace=True)
        keep = so.unpack_mask(P.mask_np(mask), n)
        want = sel.keep_bool(n)
        diff = keep != want
        if literal:
            assert not diff.any()
        else:
            assert not (diff & ~P.ewma_allowed_flips(sel)).any()
            assert diff.sum() <= 1           # tiny matrices: at most one in-band entry
        assert np.array_equal(P.bits(out), np.where(keep, P.bits(W_ref), 0))
        if counters is not None:
            assert int(counters[sp.SP_COUNTER_KEPT]) == int(keep.sum())


@pytest.mark.parametrize("seed", range(12))
def test_random_multi_context_calls_equal_single_calls(sp, seed):
    # several random matrices with a context each (widths repeat, so contexts do), one call;
    # every matrix must come out exactly as from its own call (those are checked above)
    rng = np.random.default_rng(3000 + seed)
    nm = seed % 2 == 1
    N, M = [(2, 4), (4, 8), (3, 4)][(seed // 2) % 3]
    k = int(rng.integers(2, 7))
    dtype = torch.float16 if seed % 4 < 2 else torch.bfloat16
    ctxs, owners, Ws = {}, [], []
    try:
        for _ in range(k):
            while True:
                R, n, W, big, colsq = _case(rng, need_multiple=M if nm else 1)
                if W.dtype == dtype:
                    break
            if n not in ctxs:
                ctxs[n] = sp.Context(n)
                ctxs[n].sp_set_stats(torch.from_numpy(colsq), 5)
            owners.append(ctxs[n])
            Ws.append(W)
        if nm:
            masks, outs = sp.sp_select_nm_multi(owners, Ws, N, M)
            singles = [c.sp_select_nm(W, N, M) for c, W in zip(owners, Ws)]
        else:
            counters = sp.new_counters()
            prm = sp.EwmaParams(0.125, 0.25, float(rng.choice([0.5, -0.2, 1.0])), sp.SP_S_GATED)
            masks, outs = sp.sp_select_unstructured_multi(owners, Ws, params=prm, counters=counters)
            singles = [c.sp_select_unstructured(W, params=prm) for c, W in zip(owners, Ws)]
            kept = sum(int(so.unpack_mask(P.mask_np(m), W.shape[1]).sum()) for m, W in zip(masks, Ws))
            assert int(counters[sp.SP_COUNTER_KEPT]) == kept
        for (m1, o1), m, o in zip(singles, masks, outs):
            assert torch.equal(m, m1)
            assert np.array_equal(P.bits(o), P.bits(o1))
    finally:
        for c in ctxs.values():
            c.close()
