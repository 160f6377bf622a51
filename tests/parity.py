"""Helpers shared by the GPU parity tests: moving tensors to the oracle, and the
acceptance rule for masks (bit-exact except inside a relative band around the decision
threshold)."""
from __future__ import annotations

import numpy as np
import torch

from oracle import swiftprune_oracle as so

SCORE_RTOL = 1e-5     # statistics and scores: relative tolerance
BAND_RTOL = 1e-5      # a mask bit may differ only if the oracle score is this close to its threshold
FLIP_FRACTION = 1e-6  # and at most this fraction of the entries may differ

# Flip budget.  Two correct binary32 evaluations of the running threshold (the oracle's
# sequential one, the kernels' scans) differ by a few 1e-7 relative, so an entry that sits
# inside the band flips now and then: about 0.4e-6 of all entries.  A case with fewer than 1e6
# entries cannot hold the fraction 1e-6 other than as "no flip at all", which no re-associated
# evaluation can promise; such a case is allowed one in-band flip, and every flip is added to
# this tally, whose total is held to FLIP_FRACTION by tests/test_gpu_z_flip_budget.py.
FLIP_TALLY = {"flips": 0, "entries": 0, "cases": 0}


def bits(t: torch.Tensor) -> np.ndarray:
    """uint16 bit patterns of a 16-bit float tensor (copied to the host)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def odtype(t: torch.Tensor) -> int:
    return so.F16 if t.dtype == torch.float16 else so.BF16


def mask_np(mask: torch.Tensor) -> np.ndarray:
    return mask.detach().cpu().contiguous().numpy().view(np.uint32)


def oracle_stats(batches, n) -> so.Stats:
    st = so.new_stats(n)
    for X in batches:
        so.colsq_accumulate(st, bits(X), odtype(X), threads=so.max_threads())
    return st


def rel_err(got: np.ndarray, want: np.ndarray) -> float:
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    denom = np.maximum(np.abs(want), np.finfo(np.float64).tiny)
    err = np.abs(got - want) / denom
    err[(got == want)] = 0.0
    return float(err.max()) if err.size else 0.0


def ewma_allowed_flips(sel: so.Selection) -> np.ndarray:
    """Entries whose oracle score lies within the band around the threshold it was tested against."""
    L = sel.L.astype(np.float64)
    thr = sel.thr.astype(np.float64)
    with np.errstate(invalid="ignore"):     # inf - inf (a channel with infinite factor): not in band
        return np.abs(L - thr) <= BAND_RTOL * np.maximum(np.abs(L), np.abs(thr))


def nm_allowed_flips(sel: so.Selection, n: int, M: int) -> np.ndarray:
    """Entries that have, in their group, an entry of the opposite decision whose score is within
    the band (i.e. the two sit on either side of the group's keep/prune boundary)."""
    L = sel.L.astype(np.float64).reshape(-1, n // M, M)
    keep = sel.keep_bool(n).reshape(-1, n // M, M)
    a, b = L[..., :, None], L[..., None, :]
    close = np.abs(a - b) <= BAND_RTOL * np.maximum(np.abs(a), np.abs(b))
    opposite = keep[..., :, None] != keep[..., None, :]
    return (close & opposite).any(-1).reshape(-1, n)


def check_selection(gpu_mask: torch.Tensor, gpu_out: torch.Tensor, W: torch.Tensor,
                    sel: so.Selection, allowed: np.ndarray | None, strict: bool = False):
    """Applies the acceptance rule; returns the number of differing mask bits."""
    R, n = W.shape
    got = so.unpack_mask(mask_np(gpu_mask), n)
    want = sel.keep_bool(n)
    diff = got != want
    flips = int(diff.sum())
    if strict or allowed is None:
        assert flips == 0, "mask differs in %d entries" % flips
    else:
        assert not (diff & ~allowed).any(), "mask differs outside the threshold band"
        limit = max(1.0, FLIP_FRACTION * diff.size)
        assert flips <= limit, "%d flips in %d entries (limit %.3g)" % (flips, diff.size, limit)
        FLIP_TALLY["flips"] += flips
        FLIP_TALLY["entries"] += int(diff.size)
        FLIP_TALLY["cases"] += 1
    # mask words carry no bits past n
    words = mask_np(gpu_mask)
    if n % 32:
        assert (words[:, -1] >> np.uint32(n % 32)).max(initial=0) == 0
    # pruned weights: bit-exact wherever the masks agree; and consistent with the GPU's own mask
    out = bits(gpu_out)
    win = bits(W)
    assert np.array_equal(out[~diff], sel.W_out[~diff])
    assert np.array_equal(out, np.where(got, win, 0))
    return flips
