"""Thin ctypes binding of libswiftprune.so: same names as the C ABI, argument marshalling only.

Every step of the pruning pass runs in the library's CUDA kernels.  PyTorch tensors are used
for device memory and streams; this module reads their ``data_ptr()``, shape and stride and
passes them through.  If the compiled library is missing the import fails: there is no
fallback path.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
#: the compiled library; SWIFTPRUNE_LIBRARY may point at another build of the same ABI
LIB_PATH = os.environ.get("SWIFTPRUNE_LIBRARY") or os.path.join(_HERE, "libswiftprune.so")

SP_OK = 0
SP_ERR_INVALID_ARG, SP_ERR_SHAPE, SP_ERR_DTYPE, SP_ERR_STATE = 1, 2, 3, 4
SP_ERR_DEGENERATE, SP_ERR_CUDA, SP_ERR_NOMEM = 5, 6, 7
SP_F16, SP_BF16 = 0, 1
SP_S_GATED, SP_S_LITERAL_W2, SP_S_FROZEN, SP_S_READING_X2, SP_S_LITERAL_SCAN = 0, 1, 2, 3, 4
SP_COUNTER_KEPT, SP_COUNTER_S_HAZARD, SP_NUM_COUNTERS = 0, 1, 2
SP_CALIB_X_COMPLETE = 1

#: every symbol include/swiftprune.h declares
EXPORTS = (
    "sp_create", "sp_destroy", "sp_calib_reset", "sp_calib_accumulate", "sp_calib_accumulate_ex", "sp_calib_accumulate_multi", "sp_finalize_multi",
    "sp_get_stats",
    "sp_set_stats", "sp_calib_stats_noalloc", "sp_score", "sp_la_for_sparsity", "sp_select_unstructured",
    "sp_select_unstructured_ex", "sp_search_la", "sp_ewma_trace", "sp_select_nm", "sp_select_24_compressed", "sp_apply_mask", "sp_calib_accumulate_host",
    "sp_select_nm_host", "sp_select_unstructured_host", "sp_select_unstructured_group",
    "sp_select_unstructured_group_ex", "sp_select_nm_group", "sp_select_unstructured_multi",
    "sp_select_unstructured_multi_ex", "sp_select_nm_multi", "sp_debug_status", "sp_status_string",
    "sp_last_cuda_error", "sp_launch_count",
)


class SpError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(what)


class EwmaParams(ctypes.Structure):
    _fields_ = [("alpha", ctypes.c_float), ("beta", ctypes.c_float), ("la", ctypes.c_float),
                ("s_update", ctypes.c_int)]


class Matrix(ctypes.Structure):
    """sp_matrix: one weight matrix of a grouped selection call."""
    _fields_ = [("W", ctypes.c_void_p), ("n_rows", ctypes.c_int64), ("ldw", ctypes.c_int64),
                ("mask_out", ctypes.c_void_p), ("W_out", ctypes.c_void_p), ("ldo", ctypes.c_int64)]


class Batch(ctypes.Structure):
    """sp_batch: one batch of calibration activations of a multi-input call."""
    _fields_ = [("X", ctypes.c_void_p), ("n_tokens", ctypes.c_int64), ("ldx", ctypes.c_int64)]


SP_MAX_GROUP = 8
SP_MAX_MULTI = 16


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            "libswiftprune.so is not built (%s); run `python -m paper_2501_16376_b200.build`. "
            "There is no CPU fallback." % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    vp, i64, ci, f32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_float
    lib.sp_create.argtypes = [ctypes.POINTER(vp), i64, ci]
    lib.sp_destroy.argtypes = [vp]
    lib.sp_calib_reset.argtypes = [vp, vp]
    lib.sp_calib_accumulate.argtypes = [vp, vp, ci, i64, i64, vp]
    lib.sp_calib_accumulate_ex.argtypes = [vp, vp, ci, i64, i64, ctypes.c_uint, vp]
    lib.sp_get_stats.argtypes = [vp, vp, vp, vp, ctypes.POINTER(i64), vp]
    lib.sp_set_stats.argtypes = [vp, vp, i64, vp]
    lib.sp_score.argtypes = [vp, vp, ci, i64, i64, vp, vp]
    lib.sp_calib_stats_noalloc.argtypes = [vp, ci, i64, i64, i64, vp, vp, vp, vp]
    lib.sp_la_for_sparsity.argtypes = [f32, ctypes.POINTER(f32)]
    lib.sp_select_unstructured.argtypes = [vp, vp, ci, i64, i64, f32, vp, vp, i64, vp, vp]
    lib.sp_select_unstructured_ex.argtypes = [vp, vp, ci, i64, i64, ctypes.POINTER(EwmaParams),
                                              vp, vp, i64, vp, vp]
    lib.sp_select_nm.argtypes = [vp, vp, ci, i64, i64, ci, ci, vp, vp, i64, vp]
    lib.sp_select_24_compressed.argtypes = [vp, vp, ci, i64, i64, vp, i64, vp, vp]
    lib.sp_ewma_trace.argtypes = [vp, vp, ci, i64, i64, ctypes.POINTER(EwmaParams), vp, vp, vp, vp]
    lib.sp_search_la.argtypes = [vp, vp, ci, i64, i64, f32, f32, f32, ci, ctypes.POINTER(f32),
                                 ctypes.POINTER(ctypes.c_double), vp]
    lib.sp_apply_mask.argtypes = [vp, ci, i64, i64, i64, vp, vp, i64, vp]
    lib.sp_calib_accumulate_host.argtypes = [vp, vp, ci, i64, i64, vp]
    lib.sp_select_nm_host.argtypes = [vp, vp, ci, i64, i64, ci, ci, vp, vp, i64, vp]
    lib.sp_select_unstructured_host.argtypes = [vp, vp, ci, i64, i64, f32, vp, vp, i64, vp]
    lib.sp_select_unstructured_group.argtypes = [vp, ctypes.POINTER(Matrix), ci, ci, f32, vp, vp]
    lib.sp_select_unstructured_group_ex.argtypes = [vp, ctypes.POINTER(Matrix), ci, ci,
                                                    ctypes.POINTER(EwmaParams), vp, vp]
    lib.sp_select_nm_group.argtypes = [vp, ctypes.POINTER(Matrix), ci, ci, ci, ci, vp]
    lib.sp_select_unstructured_multi.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(Matrix), ci,
                                                 ci, f32, vp, vp]
    lib.sp_select_unstructured_multi_ex.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(Matrix), ci,
                                                    ci, ctypes.POINTER(EwmaParams), vp, vp]
    lib.sp_calib_accumulate_multi.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(Batch), ci, ci,
                                              ctypes.c_uint, vp]
    lib.sp_finalize_multi.argtypes = [ctypes.POINTER(vp), ci, vp]
    lib.sp_select_nm_multi.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(Matrix), ci, ci, ci, ci,
                                       vp]
    lib.sp_debug_status.argtypes = [ctypes.POINTER(ci), ctypes.POINTER(ci), ctypes.POINTER(i64),
                                    ctypes.POINTER(i64), ci]
    lib.sp_status_string.argtypes = [ci]
    lib.sp_status_string.restype = ctypes.c_char_p
    lib.sp_last_cuda_error.restype = ctypes.c_char_p
    lib.sp_launch_count.restype = ctypes.c_uint64
    for name in EXPORTS:
        fn = getattr(lib, name)
        if fn.restype is ctypes.c_int and name not in ("sp_status_string",):
            fn.restype = ci
    return lib


lib = _load()


def _check(status: int):
    if status != SP_OK:
        msg = lib.sp_status_string(status).decode()
        if status in (SP_ERR_CUDA, SP_ERR_NOMEM):
            msg += " [" + lib.sp_last_cuda_error().decode() + "]"
        raise SpError(status, msg)


def _dtype_of(t: torch.Tensor) -> int:
    if t.dtype == torch.float16:
        return SP_F16
    if t.dtype == torch.bfloat16:
        return SP_BF16
    raise SpError(SP_ERR_DTYPE, "expected a float16 or bfloat16 tensor, got %s" % t.dtype)


def _matrix(t: torch.Tensor, what: str, host: bool = False):
    if t.dim() != 2 or (t.shape[1] > 1 and t.stride(1) != 1):
        raise SpError(SP_ERR_SHAPE, "%s must be 2-D with unit stride along its rows" % what)
    if t.is_cuda == host:
        raise SpError(SP_ERR_INVALID_ARG,
                      "%s must be a %s tensor" % (what, "CPU" if host else "CUDA"))
    ld = t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1])
    return t.data_ptr(), t.shape[0], t.shape[1], ld


def _stream(stream) -> int:
    if stream is None:
        return torch._C._cuda_getCurrentRawStream(torch.cuda.current_device())
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _ptr(t):
    return None if t is None else t.data_ptr()


def sp_launch_count() -> int:
    return int(lib.sp_launch_count())


def sp_debug_status(clear: bool = False):
    """(violations, first_code, first_index, first_limit) of the debug build's index checks;
    violations is -1 for the release build."""
    v, c = ctypes.c_int(), ctypes.c_int()
    i, lim = ctypes.c_int64(), ctypes.c_int64()
    _check(lib.sp_debug_status(ctypes.byref(v), ctypes.byref(c), ctypes.byref(i), ctypes.byref(lim),
                               1 if clear else 0))
    return v.value, c.value, i.value, lim.value


def sp_la_for_sparsity(sparsity: float) -> float:
    out = ctypes.c_float()
    _check(lib.sp_la_for_sparsity(sparsity, ctypes.byref(out)))
    return out.value


class Context:
    """Owns one ``sp_ctx`` (one layer input of ``d_in`` channels)."""

    def __init__(self, d_in: int, device: int | None = None):
        if device is None:
            device = torch.cuda.current_device()
        self.d_in = int(d_in)
        self.device = int(device)
        h = ctypes.c_void_p()
        _check(lib.sp_create(ctypes.byref(h), self.d_in, self.device))
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            lib.sp_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # -- calibration ---------------------------------------------------------
    def sp_calib_reset(self, stream=None):
        _check(lib.sp_calib_reset(self._h, _stream(stream)))

    def sp_calib_accumulate(self, X: torch.Tensor, stream=None, x_complete: bool = False):
        """x_complete: X was complete before the preceding operation on the stream began
        (SP_CALIB_X_COMPLETE, see the C header)."""
        ptr, T, n, ld = _matrix(X, "X")
        if n != self.d_in:
            raise SpError(SP_ERR_SHAPE, "X has %d channels, context has %d" % (n, self.d_in))
        if x_complete:
            _check(lib.sp_calib_accumulate_ex(self._h, ptr, _dtype_of(X), T, ld,
                                              SP_CALIB_X_COMPLETE, _stream(stream)))
        else:
            _check(lib.sp_calib_accumulate(self._h, ptr, _dtype_of(X), T, ld, _stream(stream)))

    def sp_get_stats(self, stream=None):
        """Returns (colsq fp64 [d_in], S, factor fp32 [d_in], n_tokens) as CPU tensors/numbers."""
        colsq = torch.empty(self.d_in, dtype=torch.float64)
        factor = torch.empty(self.d_in, dtype=torch.float32)
        S = ctypes.c_double()
        ntok = ctypes.c_int64()
        _check(lib.sp_get_stats(self._h, colsq.data_ptr(), ctypes.addressof(S), factor.data_ptr(),
                                ctypes.byref(ntok), _stream(stream)))
        return colsq, S.value, factor, ntok.value

    def sp_set_stats(self, colsq: torch.Tensor, n_tokens: int, stream=None):
        colsq = colsq.detach().to("cpu", torch.float64).contiguous()
        if colsq.numel() != self.d_in:
            raise SpError(SP_ERR_SHAPE, "colsq must have d_in entries")
        _check(lib.sp_set_stats(self._h, colsq.data_ptr(), int(n_tokens), _stream(stream)))

    # -- metric --------------------------------------------------------------
    def sp_score(self, W: torch.Tensor | None = None, want_scores: bool = True, stream=None):
        """Finalises the statistics; with W, returns the fp32 score matrix L (Eq. 8)."""
        if W is None or not want_scores:
            _check(lib.sp_score(self._h, None, SP_F16, 0, self.d_in, None, _stream(stream)))
            return None
        ptr, R, n, ld = _matrix(W, "W")
        self._check_width(n)
        scores = torch.empty(R, n, dtype=torch.float32, device=W.device)
        _check(lib.sp_score(self._h, ptr, _dtype_of(W), R, ld, scores.data_ptr(), _stream(stream)))
        return scores

    def sp_select_24_compressed(self, W, values=None, meta=None, stream=None):
        """2:4 selection emitted as kept values [R, d_in/2] + 4-bit-per-group indices
        [R, ceil(d_in/32)] int32 (layout in the C header).  Returns (values, meta)."""
        ptr, R, n, ld = _matrix(W, "W")
        self._check_width(n)
        if values is None:
            values = torch.empty(R, n // 2, dtype=W.dtype, device=W.device)
        if meta is None:
            meta = torch.zeros(R, (n + 31) // 32, dtype=torch.int32, device=W.device)
        vptr, _, _, ldv = _matrix(values, "values")
        _check(lib.sp_select_24_compressed(self._h, ptr, _dtype_of(W), R, ld, vptr, ldv,
                                           meta.data_ptr(), _stream(stream)))
        return values, meta

    def _check_width(self, n):
        if n != self.d_in:
            raise SpError(SP_ERR_SHAPE, "W has %d columns, context has %d" % (n, self.d_in))

    def _outputs(self, W, mask, W_out, want_mask, inplace):
        R, n = W.shape
        if mask is None and want_mask:
            mask = torch.empty(R, (n + 31) // 32, dtype=torch.int32, device=W.device)
        if inplace:
            W_out = W
        elif W_out is None:
            W_out = torch.empty_like(W)
        return mask, W_out

    # -- selection -----------------------------------------------------------
    def sp_select_unstructured(self, W, sparsity=None, *, params: EwmaParams | None = None,
                               mask=None, W_out=None, inplace=False, want_mask=True,
                               counters=None, stream=None):
        """Algorithm 1 on every row of W.  Returns (mask int32 [R, ceil(n/32)], W_out)."""
        ptr, R, n, ld = _matrix(W, "W")
        self._check_width(n)
        mask, W_out = self._outputs(W, mask, W_out, want_mask, inplace)
        optr, _, _, ldo = _matrix(W_out, "W_out")
        if params is not None:
            _check(lib.sp_select_unstructured_ex(self._h, ptr, _dtype_of(W), R, ld,
                                                 ctypes.byref(params), _ptr(mask), optr, ldo,
                                                 _ptr(counters), _stream(stream)))
        else:
            _check(lib.sp_select_unstructured(self._h, ptr, _dtype_of(W), R, ld, float(sparsity),
                                              _ptr(mask), optr, ldo, _ptr(counters),
                                              _stream(stream)))
        return mask, W_out

    def sp_ewma_trace(self, W, params: EwmaParams, stream=None):
        """est, dev (state before each element's update) and L along every row: three fp32
        tensors [R, d_in].  Sequential diagnostic, meant for a few rows."""
        ptr, R, n, ld = _matrix(W, "W")
        self._check_width(n)
        est, dev, L = (torch.empty(R, n, dtype=torch.float32, device=W.device) for _ in range(3))
        _check(lib.sp_ewma_trace(self._h, ptr, _dtype_of(W), R, ld, ctypes.byref(params),
                                 est.data_ptr(), dev.data_ptr(), L.data_ptr(), _stream(stream)))
        return est, dev, L

    def sp_search_la(self, W, target_sparsity: float, alpha: float = 0.125, beta: float = 0.125,
                     iterations: int = 24, stream=None):
        """Bisects la so that Algorithm 1 prunes target_sparsity of W.  Returns (la, achieved)."""
        ptr, R, n, ld = _matrix(W, "W")
        self._check_width(n)
        la = ctypes.c_float()
        got = ctypes.c_double()
        _check(lib.sp_search_la(self._h, ptr, _dtype_of(W), R, ld, float(target_sparsity),
                                float(alpha), float(beta), int(iterations), ctypes.byref(la),
                                ctypes.byref(got), _stream(stream)))
        return la.value, got.value

    def sp_select_nm(self, W, N: int, M: int, *, mask=None, W_out=None, inplace=False,
                     want_mask=True, stream=None):
        """N:M selection (keep N of every M).  Returns (mask, W_out)."""
        ptr, R, n, ld = _matrix(W, "W")
        self._check_width(n)
        mask, W_out = self._outputs(W, mask, W_out, want_mask, inplace)
        optr, _, _, ldo = _matrix(W_out, "W_out")
        _check(lib.sp_select_nm(self._h, ptr, _dtype_of(W), R, ld, int(N), int(M), _ptr(mask),
                                optr, ldo, _stream(stream)))
        return mask, W_out

    # -- grouped selection (layers that read this context's input) ----------------------
    def sp_select_unstructured_group(self, Ws, sparsity=None, *, params: EwmaParams | None = None,
                                     masks=None, W_outs=None, inplace=False, want_mask=True,
                                     counters=None, stream=None):
        """Algorithm 1 on several matrices that read this context's input, in one call.
        Returns (masks, W_outs)."""
        arr, k, dtype, masks, W_outs = _group(self, Ws, masks, W_outs, want_mask, inplace)
        if params is not None:
            _check(lib.sp_select_unstructured_group_ex(self._h, arr, k, dtype, ctypes.byref(params),
                                                       _ptr(counters), _stream(stream)))
        else:
            _check(lib.sp_select_unstructured_group(self._h, arr, k, dtype, float(sparsity),
                                                    _ptr(counters), _stream(stream)))
        return masks, W_outs

    def sp_select_nm_group(self, Ws, N: int, M: int, *, masks=None, W_outs=None, inplace=False,
                           want_mask=True, stream=None):
        """N:M selection of several matrices that read this context's input, in one call.
        Returns (masks, W_outs)."""
        arr, k, dtype, masks, W_outs = _group(self, Ws, masks, W_outs, want_mask, inplace)
        _check(lib.sp_select_nm_group(self._h, arr, k, dtype, int(N), int(M), _stream(stream)))
        return masks, W_outs

    # -- host-buffer variants: tensors are CPU tensors (pinned for overlap); see the C header

    def sp_calib_accumulate_host(self, X: torch.Tensor, stream=None):
        ptr, T, n, ld = _matrix(X, "X", host=True)
        if n != self.d_in:
            raise SpError(SP_ERR_SHAPE, "X has %d channels, context has %d" % (n, self.d_in))
        _check(lib.sp_calib_accumulate_host(self._h, ptr, _dtype_of(X), T, ld, _stream(stream)))

    def sp_select_nm_host(self, W, N, M, mask, W_out, stream=None):
        ptr, R, n, ld = _matrix(W, "W", host=True)
        self._check_width(n)
        optr, ldo = (None, ld) if W_out is None else (_matrix(W_out, "W_out", host=True)[0],
                                                      _matrix(W_out, "W_out", host=True)[3])
        _check(lib.sp_select_nm_host(self._h, ptr, _dtype_of(W), R, ld, int(N), int(M),
                                     _ptr(mask), optr, ldo, _stream(stream)))

    def sp_select_unstructured_host(self, W, sparsity, mask, W_out, stream=None):
        ptr, R, n, ld = _matrix(W, "W", host=True)
        self._check_width(n)
        optr, ldo = (None, ld) if W_out is None else (_matrix(W_out, "W_out", host=True)[0],
                                                      _matrix(W_out, "W_out", host=True)[3])
        _check(lib.sp_select_unstructured_host(self._h, ptr, _dtype_of(W), R, ld, float(sparsity),
                                               _ptr(mask), optr, ldo, _stream(stream)))


def _group(ctx, Ws, masks, W_outs, want_mask, inplace):
    """Marshals a list of weight tensors (and optional outputs) into an sp_matrix array."""
    k = len(Ws)
    masks = list(masks) if masks is not None else [None] * k
    W_outs = list(W_outs) if W_outs is not None else [None] * k
    arr = (Matrix * k)()
    dtype = _dtype_of(Ws[0])
    for i, W in enumerate(Ws):
        ptr, R, n, ld = _matrix(W, "W")
        ctx._check_width(n)
        if _dtype_of(W) != dtype:
            raise SpError(SP_ERR_DTYPE, "all matrices of a group must have the same dtype")
        masks[i], W_outs[i] = ctx._outputs(W, masks[i], W_outs[i], want_mask, inplace)
        optr, _, _, ldo = _matrix(W_outs[i], "W_out")
        arr[i] = Matrix(ptr, R, ld, _ptr(masks[i]), optr, ldo)
    return arr, k, dtype, masks, W_outs


def sp_calib_accumulate_multi(ctxs, Xs, stream=None, x_complete: bool = False):
    """One batch for each of several layer inputs in one call: Xs[i] ([tokens, d_in of ctxs[i]],
    all of one dtype) is added to the statistics of ctxs[i]; the contexts must all differ."""
    k = len(Xs)
    if k != len(ctxs) or k < 1:
        raise SpError(SP_ERR_INVALID_ARG, "one context per batch")
    arr = (Batch * k)()
    handles = (ctypes.c_void_p * k)()
    dtype = _dtype_of(Xs[0])
    for i, (ctx, X) in enumerate(zip(ctxs, Xs)):
        ptr, T, n, ld = _matrix(X, "X")
        if n != ctx.d_in:
            raise SpError(SP_ERR_SHAPE, "X has %d channels, context has %d" % (n, ctx.d_in))
        if _dtype_of(X) != dtype:
            raise SpError(SP_ERR_DTYPE, "all batches of a call must have the same dtype")
        arr[i] = Batch(ptr, T, ld)
        handles[i] = ctx._h
    _check(lib.sp_calib_accumulate_multi(handles, arr, k, dtype,
                                         SP_CALIB_X_COMPLETE if x_complete else 0,
                                         _stream(stream)))


def sp_finalize_multi(ctxs, stream=None):
    """S and the per-channel factors of every listed context with batches pending, one launch."""
    handles = (ctypes.c_void_p * len(ctxs))(*[c._h for c in ctxs])
    _check(lib.sp_finalize_multi(handles, len(ctxs), _stream(stream)))


def _multi(ctxs, Ws, masks, W_outs, want_mask, inplace):
    """Marshals matrices with a context each into an sp_matrix array and a handle array."""
    k = len(Ws)
    if k != len(ctxs) or k < 1:
        raise SpError(SP_ERR_INVALID_ARG, "one context per matrix")
    masks = list(masks) if masks is not None else [None] * k
    W_outs = list(W_outs) if W_outs is not None else [None] * k
    arr = (Matrix * k)()
    handles = (ctypes.c_void_p * k)()
    dtype = _dtype_of(Ws[0])
    for i, (ctx, W) in enumerate(zip(ctxs, Ws)):
        ptr, R, n, ld = _matrix(W, "W")
        ctx._check_width(n)
        if _dtype_of(W) != dtype:
            raise SpError(SP_ERR_DTYPE, "all matrices of a call must have the same dtype")
        masks[i], W_outs[i] = ctx._outputs(W, masks[i], W_outs[i], want_mask, inplace)
        optr, _, _, ldo = _matrix(W_outs[i], "W_out")
        arr[i] = Matrix(ptr, R, ld, _ptr(masks[i]), optr, ldo)
        handles[i] = ctx._h
    return handles, arr, k, dtype, masks, W_outs


def sp_select_unstructured_multi(ctxs, Ws, sparsity=None, *, params: EwmaParams | None = None,
                                 masks=None, W_outs=None, inplace=False, want_mask=True,
                                 counters=None, stream=None):
    """Algorithm 1 on matrices that read different layer inputs, in one call: Ws[i] is pruned
    with the statistics of ctxs[i] (contexts may repeat).  Returns (masks, W_outs)."""
    handles, arr, k, dtype, masks, W_outs = _multi(ctxs, Ws, masks, W_outs, want_mask, inplace)
    if params is not None:
        _check(lib.sp_select_unstructured_multi_ex(handles, arr, k, dtype, ctypes.byref(params),
                                                   _ptr(counters), _stream(stream)))
    else:
        _check(lib.sp_select_unstructured_multi(handles, arr, k, dtype, float(sparsity),
                                                _ptr(counters), _stream(stream)))
    return masks, W_outs


def sp_select_nm_multi(ctxs, Ws, N: int, M: int, *, masks=None, W_outs=None, inplace=False,
                       want_mask=True, stream=None):
    """N:M selection of matrices that read different layer inputs, in one call: Ws[i] is pruned
    with the statistics of ctxs[i].  Returns (masks, W_outs)."""
    handles, arr, k, dtype, masks, W_outs = _multi(ctxs, Ws, masks, W_outs, want_mask, inplace)
    _check(lib.sp_select_nm_multi(handles, arr, k, dtype, int(N), int(M), _stream(stream)))
    return masks, W_outs


def sp_apply_mask(W: torch.Tensor, mask: torch.Tensor, W_out: torch.Tensor | None = None,
                  stream=None) -> torch.Tensor:
    ptr, R, n, ld = _matrix(W, "W")
    if W_out is None:
        W_out = torch.empty_like(W)
    optr, _, _, ldo = _matrix(W_out, "W_out")
    if mask.dim() != 2 or tuple(mask.shape) != (R, (n + 31) // 32) or not mask.is_contiguous():
        raise SpError(SP_ERR_SHAPE, "mask must be contiguous [rows, ceil(cols/32)]")
    _check(lib.sp_apply_mask(ptr, _dtype_of(W), R, n, ld, mask.data_ptr(), optr, ldo,
                             _stream(stream)))
    return W_out


def sp_calib_stats_noalloc(X: torch.Tensor, colsq_out: torch.Tensor | None = None,
                           factor_out: torch.Tensor | None = None,
                           S_out: torch.Tensor | None = None, stream=None):
    """One-shot statistics of a single batch for callers that cannot allocate device memory:
    the library uses a fixed internal array instead of a context (d_in <= 16384).  The outputs
    are device tensors the caller already owns (fp64 [d_in], fp32 [d_in], fp64 [1]); this
    wrapper allocates nothing either.  Calls on one device must not overlap on the GPU."""
    ptr, T, n, ld = _matrix(X, "X")
    for t, dt, numel in ((colsq_out, torch.float64, n), (factor_out, torch.float32, n),
                         (S_out, torch.float64, 1)):
        if t is not None and (t.dtype != dt or t.numel() < numel or not t.is_cuda
                              or not t.is_contiguous()):
            raise SpError(SP_ERR_INVALID_ARG, "output buffers must be contiguous CUDA tensors "
                                              "of the documented type and size")
    with torch.cuda.device(X.device):
        _check(lib.sp_calib_stats_noalloc(ptr, _dtype_of(X), T, n, ld, _ptr(colsq_out),
                                          _ptr(factor_out), _ptr(S_out), _stream(stream)))


def new_counters(device=None) -> torch.Tensor:
    """Zeroed device counter block for the selection calls (int64 view of the uint64 pair)."""
    return torch.zeros(SP_NUM_COUNTERS, dtype=torch.int64, device=device or "cuda")
