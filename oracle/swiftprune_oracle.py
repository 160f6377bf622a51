"""ctypes front end of the SwiftPrune CPU oracle (``swiftprune_oracle.c``).

TEST INFRASTRUCTURE, NOT A PRODUCT PATH.  Only the test-suite, the smoke check
and the benchmark's CPU-baseline leg may import this module; the CUDA library
and its Python binding never do, and this module never imports them.

Arrays are numpy arrays.  16-bit float tensors travel as ``uint16`` bit
patterns together with ``dtype`` (``F16`` = IEEE binary16, ``BF16`` =
bfloat16), so that no conversion happens on the way in.

The functions mirror the steps of the paper: calibration statistics
(Algorithm 1, step 1), the contribution metric (Eq. 8), the EWMA selection
(Algorithm 1 with Table 2's state rules, ``la`` from Table 3), the N:M group
selection (Section 3.3) and the write-back (Algorithm 1's ``c_i = w_i``).

"parity unpinned": the mapping nominal sparsity -> achieved sparsity (the
paper prints no worked example), and ``la`` for ratios outside Table 3.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

F16 = 0
BF16 = 1
S_FROZEN = 0
S_LITERAL_W2 = 1
S_READING_X2 = 2     # the other reading of Table 2's row S: S <- S - x_i^2 when pruned

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "swiftprune_oracle.c")
_LIB = os.path.join(_HERE, "libswiftprune_oracle.so")

#: Table 3 of the paper: pruning ratio (%) -> la.
TABLE3_LA = {90: -1.5, 80: -0.9, 70: -0.2, 60: 0.2, 50: 0.5}
#: Smoothing factors the paper states (Section 4.2, with Fig. 2).
ALPHA = 0.125
BETA = 0.125


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-ffp-contract=off keeps one rounding per op)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    cmd = ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared",
           "-fPIC", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        # SWIFTPRUNE_ORACLE_LIBRARY: a library built elsewhere from (a copy of) the C source; the
        # mutation test uses it to check that the pins catch planted mistakes
        lib = ctypes.CDLL(os.environ.get("SWIFTPRUNE_ORACLE_LIBRARY") or build())
        i64, f32, f64, ci, vp = (ctypes.c_int64, ctypes.c_float, ctypes.c_double,
                                 ctypes.c_int, ctypes.c_void_p)
        lib.spo_decode_array.argtypes = [vp, ci, i64, vp]
        lib.spo_colsq_accumulate.argtypes = [vp, ci, i64, i64, i64, vp, ci]
        lib.spo_total.argtypes = [vp, i64]
        lib.spo_total.restype = f64
        lib.spo_channel_factor_f32.argtypes = [vp, f32, i64, vp]
        lib.spo_score_f32.argtypes = [vp, ci, i64, i64, i64, vp, f32, vp]
        lib.spo_score_f64.argtypes = [vp, ci, i64, i64, i64, vp, f64, vp]
        lib.spo_select_ewma_f32.argtypes = [vp, ci, i64, i64, i64, vp, f32, f32, f32, f32, ci,
                                            vp, vp, i64, vp, vp, ci]
        lib.spo_select_ewma_f64.argtypes = [vp, ci, i64, i64, i64, vp, f64, f64, f64, f64, ci,
                                            vp, vp, i64, vp, vp, ci]
        lib.spo_select_nm_f32.argtypes = [vp, ci, i64, i64, i64, vp, f32, ci, ci,
                                          vp, vp, i64, vp, ci]
        lib.spo_select_nm_f32.restype = ci
        lib.spo_apply_mask.argtypes = [vp, i64, i64, i64, vp, vp, i64]
        lib.spo_max_threads.restype = ci
        _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _bits2d(a: np.ndarray) -> np.ndarray:
    a = np.asarray(a)
    if a.dtype != np.uint16 or a.ndim != 2:
        raise TypeError("expected a 2-D uint16 array of 16-bit float bit patterns")
    if a.strides[1] != 2 or a.strides[0] % 2 != 0:
        a = np.ascontiguousarray(a)
    return a


def max_threads() -> int:
    return int(_load().spo_max_threads())


def decode(bits: np.ndarray, dtype: int) -> np.ndarray:
    """Exact 16-bit float -> float32 decode of an array of bit patterns."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(bits.shape, dtype=np.float32)
    _load().spo_decode_array(_ptr(bits), dtype, bits.size, _ptr(out))
    return out


def la_for_sparsity(sparsity: float) -> float:
    """Table 3 lookup.  Ratios the table does not list are interpolated linearly
    between (or extrapolated from) the nearest two entries: parity unpinned."""
    pct = sparsity * 100.0
    key = int(round(pct))
    if abs(pct - key) < 1e-6 and key in TABLE3_LA:
        return TABLE3_LA[key]
    pts = sorted(TABLE3_LA.items())
    xs = [p for p, _ in pts]
    ys = [v for _, v in pts]
    if pct <= xs[0]:
        i = 0
    elif pct >= xs[-1]:
        i = len(xs) - 2
    else:
        i = max(j for j in range(len(xs) - 1) if xs[j] <= pct)
    t = (pct - xs[i]) / (xs[i + 1] - xs[i])
    return ys[i] + t * (ys[i + 1] - ys[i])


@dataclass
class Stats:
    """Calibration statistics of one layer input (Algorithm 1, step 1)."""
    colsq: np.ndarray      # fp64 [n]   sum_t X[t,q]^2
    n_tokens: int = 0

    @property
    def S(self) -> float:
        return float(_load().spo_total(_ptr(self.colsq), self.colsq.size))

    @property
    def colsq32(self) -> np.ndarray:
        return self.colsq.astype(np.float32)

    @property
    def S32(self) -> np.float32:
        return np.float32(self.S)

    def channel_factor32(self) -> np.ndarray:
        """c_q = 1 / (2 (1 - x_q^2/S)) in binary32 (the per-channel part of Eq. 8)."""
        c = np.empty(self.colsq.size, dtype=np.float32)
        c32 = self.colsq32
        _load().spo_channel_factor_f32(_ptr(c32), self.S32, c.size, _ptr(c))
        return c


def new_stats(n: int) -> Stats:
    return Stats(np.zeros(n, dtype=np.float64), 0)


def colsq_accumulate(stats: Stats, X_bits: np.ndarray, dtype: int, threads: int = 1) -> Stats:
    """colsq[q] += sum_t X[t,q]^2 over one batch X [T, n] (fp64)."""
    X = _bits2d(X_bits)
    T, n = X.shape
    if n != stats.colsq.size:
        raise ValueError("channel count mismatch")
    _load().spo_colsq_accumulate(_ptr(X), dtype, T, n, X.strides[0] // 2, _ptr(stats.colsq),
                                 threads)
    stats.n_tokens += T
    return stats


def _check_stats(stats: Stats):
    S = stats.S
    if not np.isfinite(S) or S <= 0.0 or not np.all(np.isfinite(stats.colsq)):
        raise ValueError("degenerate calibration statistics (S == 0 or non-finite)")


def score_f32(W_bits, dtype, stats: Stats) -> np.ndarray:
    W = _bits2d(W_bits)
    _check_stats(stats)
    R, n = W.shape
    L = np.empty((R, n), dtype=np.float32)
    c32 = stats.colsq32
    _load().spo_score_f32(_ptr(W), dtype, R, n, W.strides[0] // 2, _ptr(c32), stats.S32, _ptr(L))
    return L


def score_f64(W_bits, dtype, stats: Stats) -> np.ndarray:
    W = _bits2d(W_bits)
    _check_stats(stats)
    R, n = W.shape
    L = np.empty((R, n), dtype=np.float64)
    _load().spo_score_f64(_ptr(W), dtype, R, n, W.strides[0] // 2, _ptr(stats.colsq), stats.S,
                          _ptr(L))
    return L


@dataclass
class Selection:
    mask: np.ndarray            # uint32 [R, ceil(n/32)]
    W_out: np.ndarray           # uint16 [R, n]
    L: np.ndarray | None = None     # scores the decisions used
    thr: np.ndarray | None = None   # EWMA only: est - la*dev each L_i was tested against

    def keep_bool(self, n: int) -> np.ndarray:
        return unpack_mask(self.mask, n)


def unpack_mask(mask: np.ndarray, n: int) -> np.ndarray:
    """uint32 [R, words] -> bool [R, n] (bit j of word k = column 32k+j)."""
    m = np.ascontiguousarray(mask, dtype=np.uint32)
    bits = np.unpackbits(m.view(np.uint8), axis=1, bitorder="little")
    return bits[:, :n].astype(bool)


def select_ewma(W_bits, dtype, stats: Stats, la: float, alpha: float = ALPHA,
                beta: float = BETA, s_update: int = S_LITERAL_W2, precision: str = "f32",
                want_trace: bool = False, threads: int = 1) -> Selection:
    """Algorithm 1 on every row of W."""
    W = _bits2d(W_bits)
    _check_stats(stats)
    R, n = W.shape
    words = (n + 31) // 32
    mask = np.zeros((R, words), dtype=np.uint32)
    W_out = np.empty((R, n), dtype=np.uint16)
    lib = _load()
    if precision == "f32":
        L = np.empty((R, n), dtype=np.float32) if want_trace else None
        thr = np.empty((R, n), dtype=np.float32) if want_trace else None
        c32 = stats.colsq32
        lib.spo_select_ewma_f32(_ptr(W), dtype, R, n, W.strides[0] // 2, _ptr(c32), stats.S32,
                                alpha, beta, la, s_update, _ptr(mask), _ptr(W_out), n,
                                _ptr(L), _ptr(thr), threads)
    elif precision == "f64":
        L = np.empty((R, n), dtype=np.float64) if want_trace else None
        thr = np.empty((R, n), dtype=np.float64) if want_trace else None
        lib.spo_select_ewma_f64(_ptr(W), dtype, R, n, W.strides[0] // 2, _ptr(stats.colsq),
                                stats.S, alpha, beta, la, s_update, _ptr(mask), _ptr(W_out), n,
                                _ptr(L), _ptr(thr), threads)
    else:
        raise ValueError(precision)
    return Selection(mask, W_out, L, thr)


def select_unstructured(W_bits, dtype, stats: Stats, sparsity: float, **kw) -> Selection:
    """Algorithm 1 with la taken from Table 3 for the requested pruning ratio."""
    return select_ewma(W_bits, dtype, stats, la_for_sparsity(sparsity), **kw)


def search_la(W_bits, dtype, stats: Stats, target_sparsity: float, alpha: float = ALPHA,
              beta: float = BETA, iterations: int = 24, threads: int = 1):
    """Bisection of la on [-8, 8] for a requested pruning ratio (the paper sets la per ratio by
    hand, Table 3): the pruned fraction of Algorithm 1 with S fixed never increases with la.
    Every step evaluates Algorithm 1 at the midpoint (float32 arithmetic for the midpoint);
    returns the visited la whose pruned fraction is closest to the target, and that fraction."""
    lo, hi = np.float32(-8.0), np.float32(8.0)
    best = (2.0, np.float32(0.0), 0.0)
    W = _bits2d(W_bits)
    n = W.shape[1]
    for _ in range(iterations):
        la = np.float32(0.5) * (lo + hi)
        sel = select_ewma(W, dtype, stats, float(la), alpha, beta, s_update=S_FROZEN,
                          threads=threads)
        pruned = 1.0 - float(sel.keep_bool(n).mean(dtype=np.float64))
        gap = abs(pruned - float(np.float32(target_sparsity)))
        if gap < best[0]:
            best = (gap, la, pruned)
        if pruned > float(np.float32(target_sparsity)):
            lo = la
        else:
            hi = la
    return float(best[1]), best[2]


def select_nm(W_bits, dtype, stats: Stats, N: int, M: int, want_trace: bool = False,
              threads: int = 1) -> Selection:
    """Section 3.3: keep N of every M contiguous weights (largest L kept)."""
    W = _bits2d(W_bits)
    _check_stats(stats)
    R, n = W.shape
    words = (n + 31) // 32
    mask = np.zeros((R, words), dtype=np.uint32)
    W_out = np.empty((R, n), dtype=np.uint16)
    L = np.empty((R, n), dtype=np.float32) if want_trace else None
    c32 = stats.colsq32
    rc = _load().spo_select_nm_f32(_ptr(W), dtype, R, n, W.strides[0] // 2, _ptr(c32), stats.S32,
                                   N, M, _ptr(mask), _ptr(W_out), n, _ptr(L), threads)
    if rc != 0:
        raise ValueError("N:M selection needs 0 < N < M <= 32 and n % M == 0")
    return Selection(mask, W_out, L, None)


def compress_24(W_bits, keep: np.ndarray):
    """Compressed form of a 2:4 selection (Section 3.3): for every group of four columns the two
    kept weights in column order, and a 4-bit record idx0 | idx1 << 2 of their positions in the
    group; eight records per uint32 word, group 8k+g at bits 4g..4g+3 of word k.
    Returns (values uint16 [R, n/2], meta uint32 [R, ceil(n/32)])."""
    W = _bits2d(W_bits)
    R, n = W.shape
    keep = np.asarray(keep, dtype=bool)
    if n % 4 or keep.shape != (R, n) or not (keep.reshape(R, n // 4, 4).sum(-1) == 2).all():
        raise ValueError("needs exactly two kept weights in every group of four")
    values = np.zeros((R, n // 2), dtype=np.uint16)
    meta = np.zeros((R, (n + 31) // 32), dtype=np.uint32)
    for r in range(R):
        for g in range(n // 4):
            idx = [j for j in range(4) if keep[r, 4 * g + j]]
            values[r, 2 * g] = W[r, 4 * g + idx[0]]
            values[r, 2 * g + 1] = W[r, 4 * g + idx[1]]
            meta[r, g // 8] |= np.uint32((idx[0] | (idx[1] << 2)) << (4 * (g % 8)))
    return values, meta


def expand_24(values: np.ndarray, meta: np.ndarray, n: int) -> np.ndarray:
    """Inverse of compress_24: the dense pruned matrix (uint16 [R, n])."""
    R = values.shape[0]
    out = np.zeros((R, n), dtype=np.uint16)
    for r in range(R):
        for g in range(n // 4):
            rec = (int(meta[r, g // 8]) >> (4 * (g % 8))) & 0xF
            out[r, 4 * g + (rec & 3)] = values[r, 2 * g]
            out[r, 4 * g + (rec >> 2)] = values[r, 2 * g + 1]
    return out


def apply_mask(W_bits, mask) -> np.ndarray:
    W = _bits2d(W_bits)
    R, n = W.shape
    mask = np.ascontiguousarray(mask, dtype=np.uint32)
    if mask.shape != (R, (n + 31) // 32):
        raise ValueError("mask shape")
    out = np.empty((R, n), dtype=np.uint16)
    _load().spo_apply_mask(_ptr(W), R, n, W.strides[0] // 2, _ptr(mask), _ptr(out), n)
    return out


def topk_keep(L: np.ndarray, n_prune: np.ndarray | int) -> np.ndarray:
    """Sort-based selection the paper describes before introducing EWMA (end of
    Section 3.1): per row, prune the n_prune smallest L (stable, lower column
    first among equals).  Returns bool keep [R, n]."""
    L = np.asarray(L)
    R, n = L.shape
    n_prune = np.broadcast_to(np.asarray(n_prune), (R,))
    order = np.argsort(L, axis=1, kind="stable")
    keep = np.ones((R, n), dtype=bool)
    for r in range(R):
        keep[r, order[r, : int(n_prune[r])]] = False
    return keep
