"""ctypes binding of libobc.so: one Python function per C entry point, same names, argument marshalling only.

torch is used for device memory (tensors, workspaces) and for the current CUDA stream; every step of the
method runs inside the library's kernels.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIBPATH = os.path.join(_HERE, "libobc.so")

OP_HESSIAN, OP_INVERSE, OP_PRUNE_TRACE, OP_SELECT, OP_PRUNE_APPLY, OP_QUANTIZE, OP_PRUNE_BLOCKS, OP_CROSS_GRAM, OP_REFIT = range(9)
PREC_FP32, PREC_TF32, PREC_BF16X3 = 0, 1, 2
FLAG_OUTLIERS = 1
ENGINE_AUTO, ENGINE_STREAMING, ENGINE_BLOCKED = 0, 1, 2
ENGINE_WHOLE_WAVES = 1

EXPORTED_SYMBOLS = (
    "obc_status_string", "obc_kernel_launches", "obc_engine_plan", "obc_workspace_bytes", "obc_hessian", "obc_cross_gram", "obc_refit", "obc_hessian_inverse", "obc_prune_trace", "obc_prune_nm", "obc_prune_blocks",
    "obc_select_global_mask", "obc_select_global_mask_static", "obc_prune_apply", "obc_minmax_grid", "obc_quantize",
)


class OBCError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__(f"{where}: status {status} ({obc_status_string(status)})")


_lib = None


def library_path() -> str:
    return _LIBPATH


def load_library():
    """dlopen libobc.so; raises if it has not been built (there is no fallback path)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIBPATH):
        raise RuntimeError(f"{_LIBPATH} is missing: build it with `python -m paper_2208_11580_b200.build` "
                           "(the CUDA library is the only implementation)")
    lib = ctypes.CDLL(_LIBPATH)
    c_int, c_i64, c_sz, c_f, vp = ctypes.c_int, ctypes.c_int64, ctypes.c_size_t, ctypes.c_float, ctypes.c_void_p
    lib.obc_status_string.restype = ctypes.c_char_p
    lib.obc_status_string.argtypes = [c_int]
    lib.obc_kernel_launches.restype = ctypes.c_ulonglong
    lib.obc_kernel_launches.argtypes = []
    lib.obc_engine_plan.restype = c_int
    lib.obc_engine_plan.argtypes = [c_int, c_int, c_int, vp, ctypes.POINTER(ctypes.c_int32)]
    lib.obc_workspace_bytes.restype = c_sz
    lib.obc_workspace_bytes.argtypes = [c_int, c_int, c_int, c_i64]
    lib.obc_hessian.restype = c_int
    lib.obc_hessian.argtypes = [vp, c_int, c_i64, c_i64, vp, c_int, c_int, c_int, vp, c_int, vp, c_sz, vp]
    lib.obc_cross_gram.restype = c_int
    lib.obc_cross_gram.argtypes = [vp, c_i64, vp, c_i64, c_int, c_int, c_i64, vp, c_int, c_int, c_int, vp, c_int, vp, c_sz, vp]
    lib.obc_refit.restype = c_int
    lib.obc_refit.argtypes = [vp, c_int, vp, c_int, c_int, c_int, vp, c_int, c_int, vp, c_sz, vp]
    lib.obc_hessian_inverse.restype = c_int
    lib.obc_hessian_inverse.argtypes = [vp, c_int, c_int, c_f, vp, c_int, vp, vp, c_sz, vp]
    lib.obc_prune_trace.restype = c_int
    lib.obc_prune_trace.argtypes = [vp, c_int, c_int, c_int, c_int, c_int, vp, c_int, c_int, vp, vp, vp, vp, vp, c_sz, vp, vp]
    lib.obc_prune_nm.restype = c_int
    lib.obc_prune_nm.argtypes = [vp, c_int, c_int, c_int, c_int, c_int, vp, c_int, c_int, c_int, vp, vp, vp, c_int, vp, vp,
                                 vp, c_sz, vp, vp]
    lib.obc_prune_blocks.restype = c_int
    lib.obc_prune_blocks.argtypes = [vp, c_int, c_int, c_int, c_int, c_int, vp, c_int, c_int, vp, vp, vp, vp, vp, c_sz, vp, vp]
    lib.obc_select_global_mask.restype = c_int
    lib.obc_select_global_mask.argtypes = [vp, vp, c_int, c_int, c_i64, vp, vp, vp, c_sz, vp]
    lib.obc_select_global_mask_static.restype = c_int
    lib.obc_select_global_mask_static.argtypes = [vp, vp, c_int, c_int, c_i64, vp, vp, vp]
    lib.obc_prune_apply.restype = c_int
    lib.obc_prune_apply.argtypes = [vp, c_int, c_int, c_int, c_int, c_int, vp, c_int, vp, vp, vp, c_int, vp, c_int, vp,
                                    vp, c_sz, vp, vp]
    lib.obc_minmax_grid.restype = c_int
    lib.obc_minmax_grid.argtypes = [vp, c_int, c_int, c_int, vp, c_int, c_int, vp, vp, ctypes.POINTER(c_int), vp]
    lib.obc_quantize.restype = c_int
    lib.obc_quantize.argtypes = [vp, c_int, c_int, c_int, c_int, c_int, vp, c_int, vp, vp, c_int, c_int, vp, vp, c_int,
                                 vp, c_int, vp, vp, vp, vp, vp, c_sz, vp, vp]
    _lib = lib
    return lib


def obc_status_string(status: int) -> str:
    return load_library().obc_status_string(int(status)).decode()


def obc_kernel_launches() -> int:
    return int(load_library().obc_kernel_launches())


class EngineOpts(ctypes.Structure):
    """obc_engine_opts: per-call choice of the row elimination engine (engine, threads per row, limit on deferred
    updates); all zero = the library's defaults."""
    _fields_ = [("engine", ctypes.c_int32), ("threads", ctypes.c_int32), ("max_pending", ctypes.c_int32),
                ("flags", ctypes.c_int32)]


def engine_opts(engine: int = ENGINE_AUTO, threads: int = 0, max_pending: int = 0, flags: int = 0) -> EngineOpts:
    return EngineOpts(int(engine), int(threads), int(max_pending), int(flags))


def _opts(opts):
    """None, an EngineOpts, or a (engine, threads, max_pending) tuple -> pointer argument (kept alive by the caller)."""
    if opts is None:
        return None
    if not isinstance(opts, EngineOpts):
        opts = engine_opts(*opts)
    return ctypes.cast(ctypes.pointer(opts), ctypes.c_void_p)


def obc_engine_plan(d_col: int, with_trace: bool = False, row_count: int = 0, opts=None) -> dict:
    """How row_count rows (0 = many) of length d_col would run on the current device with the engine options `opts`."""
    plan = (ctypes.c_int32 * 8)()
    _raise(load_library().obc_engine_plan(int(d_col), int(bool(with_trace)), int(row_count), _opts(opts), plan), "obc_engine_plan")
    return {"engine": int(plan[0]), "threads": int(plan[1]), "rows_per_sm": int(plan[2]), "on_chip_below": int(plan[3]),
            "panel_floats": int(plan[4]), "max_pending": int(plan[5]), "sm_count": int(plan[6]),
            "l2_vectors": int(plan[7])}


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check(t, dtype, name, cuda=True):
    if t is None:
        return
    if t.dtype != dtype:
        raise TypeError(f"{name}: expected {dtype}, got {t.dtype}")
    if cuda and not t.is_cuda:
        raise ValueError(f"{name}: must be a CUDA tensor")
    if t.dim() >= 1 and t.stride(-1) != 1:
        raise ValueError(f"{name}: innermost dimension must be contiguous")


def _ld(t):
    return int(t.stride(0)) if t.dim() == 2 and t.shape[0] > 1 else int(t.shape[-1])


def obc_workspace_bytes(op: int, row_count: int, d_col: int, n: int = 0) -> int:
    return int(load_library().obc_workspace_bytes(int(op), int(row_count), int(d_col), int(n)))


def _workspace(ws, op, row_count, d_col, n, device, where):
    need = obc_workspace_bytes(op, row_count, d_col, n)
    if need == 0:
        raise OBCError(8, where + " (workspace query)")
    if ws is None:
        ws = torch.empty(need, dtype=torch.uint8, device=device)
    return ws, ws.numel()


def _raise(status, where):
    if status != 0:
        raise OBCError(status, where)


def obc_hessian(X, H, accumulate=False, prec=PREC_FP32, ws=None, stream=None, info=None, wait_limit=0):
    """H (+)= 2 X X^T for one chunk X (d_col x n) of the calibration data.  info: optional device int32[1] that
    receives 0 or the time-out status of the tensor-core kernels' bounded waits (wait_limit: see obc.h)."""
    _check(X, torch.float32, "X"); _check(H, torch.float32, "H"); _check(info, torch.int32, "info")
    d, n = X.shape
    ws, nb = _workspace(ws, OP_HESSIAN, 0, d, n, X.device, "obc_hessian")
    _raise(load_library().obc_hessian(_ptr(X), d, n, _ld(X), _ptr(H), _ld(H), int(bool(accumulate)), int(prec),
                                      _ptr(info), int(wait_limit), _ptr(ws), nb, _stream(stream)), "obc_hessian")
    return H


def obc_cross_gram(Y, X, G, accumulate=False, prec=PREC_FP32, ws=None, stream=None, info=None, wait_limit=0):
    """G (+)= Y X^T for one chunk of the calibration axis (Y: d_row x n dense outputs, X: d_col x n inputs)."""
    _check(Y, torch.float32, "Y"); _check(X, torch.float32, "X"); _check(G, torch.float32, "G")
    R, n = Y.shape
    d = X.shape[0]
    nb = 0
    if prec != PREC_FP32:
        ws, nb = _workspace(ws, OP_CROSS_GRAM, R, d, n, X.device, "obc_cross_gram")
    _raise(load_library().obc_cross_gram(_ptr(Y), _ld(Y), _ptr(X), _ld(X), R, d, n, _ptr(G), _ld(G), int(bool(accumulate)),
                                         int(prec), _ptr(info), int(wait_limit), _ptr(ws), nb, _stream(stream)), "obc_cross_gram")
    return G


def obc_refit(G, Hinv, W_out, prec=PREC_FP32, ws=None, stream=None):
    """W_out = 2 G Hinv: the dense least-squares weights for the inputs behind G and Hinv (prec: CUDA cores or the
    tensor-core kernel of obc_cross_gram)."""
    _check(G, torch.float32, "G"); _check(Hinv, torch.float32, "Hinv"); _check(W_out, torch.float32, "W_out")
    R, d = G.shape
    nb = 0
    if prec != PREC_FP32:
        ws, nb = _workspace(ws, OP_REFIT, R, d, 0, G.device, "obc_refit")
    _raise(load_library().obc_refit(_ptr(G), _ld(G), _ptr(Hinv), _ld(Hinv), R, d, _ptr(W_out), _ld(W_out), int(prec),
                                    _ptr(ws), nb, _stream(stream)), "obc_refit")
    return W_out


def obc_hessian_inverse(H, damp_rel, Hinv=None, info=None, ws=None, stream=None):
    """Hinv = inv(H + damp_rel*mean(diag H)*I); returns (Hinv, info) with info a device int32[1]."""
    _check(H, torch.float32, "H")
    d = H.shape[0]
    if Hinv is None:   # leading dimension padded to a multiple of 4 floats
        Hinv = torch.empty(d, (d + 3) // 4 * 4, dtype=torch.float32, device=H.device)[:, :d]
    info = torch.zeros(1, dtype=torch.int32, device=H.device) if info is None else info
    _check(Hinv, torch.float32, "Hinv"); _check(info, torch.int32, "info")
    ws, nb = _workspace(ws, OP_INVERSE, 0, d, 0, H.device, "obc_hessian_inverse")
    _raise(load_library().obc_hessian_inverse(_ptr(H), d, _ld(H), float(damp_rel), _ptr(Hinv), _ld(Hinv), _ptr(info),
                                              _ptr(ws), nb, _stream(stream)), "obc_hessian_inverse")
    return Hinv, info


def obc_prune_trace(W, Hinv, order, loss, row_status, steps=None, w_trace=None, row_begin=0, row_count=None,
                    ws=None, opts=None, stream=None):
    """Algorithm 1 on rows [row_begin, row_begin+row_count): fills order, loss (and w_trace)."""
    _check(W, torch.float32, "W"); _check(Hinv, torch.float32, "Hinv"); _check(order, torch.int32, "order")
    _check(loss, torch.float32, "loss"); _check(row_status, torch.int32, "row_status"); _check(w_trace, torch.float32, "w_trace")
    R, d = W.shape
    row_count = R - row_begin if row_count is None else row_count
    steps = d if steps is None else steps
    ws, nb = _workspace(ws, OP_PRUNE_TRACE, row_count, d, 0, W.device, "obc_prune_trace")
    _raise(load_library().obc_prune_trace(_ptr(W), _ld(W), R, d, row_begin, row_count, _ptr(Hinv), _ld(Hinv), steps,
                                          _ptr(order), _ptr(loss), _ptr(w_trace), _ptr(row_status), _ptr(ws), nb,
                                          _opts(opts), _stream(stream)), "obc_prune_trace")


def obc_prune_nm(W, Hinv, n_keep, m_block, W_out, row_status, order=None, loss=None, mask=None, row_begin=0,
                 row_count=None, ws=None, opts=None, stream=None):
    """N:M pruning of rows [row_begin, row_begin+row_count): every block of m_block columns keeps n_keep weights."""
    _check(W, torch.float32, "W"); _check(Hinv, torch.float32, "Hinv"); _check(W_out, torch.float32, "W_out")
    _check(row_status, torch.int32, "row_status"); _check(order, torch.int32, "order"); _check(loss, torch.float32, "loss")
    _check(mask, torch.uint8, "mask")
    R, d = W.shape
    row_count = R - row_begin if row_count is None else row_count
    ws, nb = _workspace(ws, OP_PRUNE_TRACE, row_count, d, 0, W.device, "obc_prune_nm")
    _raise(load_library().obc_prune_nm(_ptr(W), _ld(W), R, d, row_begin, row_count, _ptr(Hinv), _ld(Hinv), int(n_keep),
                                       int(m_block), _ptr(order), _ptr(loss), _ptr(W_out), _ld(W_out), _ptr(mask),
                                       _ptr(row_status), _ptr(ws), nb, _opts(opts), _stream(stream)), "obc_prune_nm")


def obc_prune_blocks(W, Hinv, order, loss, row_status, block=4, w_trace=None, row_begin=0, row_count=None, ws=None,
                     opts=None, stream=None):
    """Block pruning (blocks of `block` consecutive columns, Eq. 5) of rows [row_begin, row_begin+row_count): full trace."""
    _check(W, torch.float32, "W"); _check(Hinv, torch.float32, "Hinv"); _check(order, torch.int32, "order")
    _check(loss, torch.float32, "loss"); _check(row_status, torch.int32, "row_status"); _check(w_trace, torch.float32, "w_trace")
    R, d = W.shape
    row_count = R - row_begin if row_count is None else row_count
    ws, nb = _workspace(ws, OP_PRUNE_BLOCKS, row_count, d, 0, W.device, "obc_prune_blocks")
    _raise(load_library().obc_prune_blocks(_ptr(W), _ld(W), R, d, row_begin, row_count, _ptr(Hinv), _ld(Hinv), int(block),
                                           _ptr(order), _ptr(loss), _ptr(w_trace), _ptr(row_status), _ptr(ws), nb,
                                           _opts(opts), _stream(stream)), "obc_prune_blocks")


def obc_select_global_mask(loss, order, k, counts, mask, ws=None, stream=None):
    """Algorithm 2: per-row counts and the mask (1 = kept) with k pruned weights."""
    _check(loss, torch.float32, "loss"); _check(order, torch.int32, "order"); _check(counts, torch.int32, "counts")
    _check(mask, torch.uint8, "mask")
    R, d = loss.shape
    ws, nb = _workspace(ws, OP_SELECT, R, d, 0, loss.device, "obc_select_global_mask")
    _raise(load_library().obc_select_global_mask(_ptr(loss), _ptr(order), R, d, int(k), _ptr(counts), _ptr(mask),
                                                 _ptr(ws), nb, _stream(stream)), "obc_select_global_mask")


def obc_select_global_mask_static(loss, order, k, counts, mask, stream=None):
    """Algorithm 2 without a workspace: for callers that must not allocate device memory.  Uses the scratch array
    built into the library (limits: OBC_SELECT_STATIC_MAX_ROWS rows, OBC_SELECT_STATIC_MAX_KEYS entries); calls that
    may overlap on the GPU must not share a device.  Same results as obc_select_global_mask."""
    _check(loss, torch.float32, "loss"); _check(order, torch.int32, "order"); _check(counts, torch.int32, "counts")
    _check(mask, torch.uint8, "mask")
    R, d = loss.shape
    _raise(load_library().obc_select_global_mask_static(_ptr(loss), _ptr(order), R, d, int(k), _ptr(counts), _ptr(mask),
                                                        _stream(stream)), "obc_select_global_mask_static")


def obc_prune_apply(W, Hinv, order, counts, W_out, row_status, w_trace=None, trace_steps=0, row_begin=0,
                    row_count=None, ws=None, opts=None, stream=None):
    """Weights after the first counts[r] eliminations (trace gather if w_trace is given, else replay)."""
    _check(W, torch.float32, "W"); _check(W_out, torch.float32, "W_out"); _check(counts, torch.int32, "counts")
    R, d = W.shape
    row_count = R - row_begin if row_count is None else row_count
    if w_trace is None:
        ws, nb = _workspace(ws, OP_PRUNE_APPLY, row_count, d, 0, W.device, "obc_prune_apply")
    else:
        nb = 0 if ws is None else ws.numel()
    _raise(load_library().obc_prune_apply(_ptr(W), _ld(W), R, d, row_begin, row_count, _ptr(Hinv),
                                          0 if Hinv is None else _ld(Hinv), _ptr(order), _ptr(counts), _ptr(w_trace),
                                          int(trace_steps), _ptr(W_out), _ld(W_out), _ptr(row_status), _ptr(ws), nb,
                                          _opts(opts), _stream(stream)), "obc_prune_apply")


def obc_minmax_grid(W, bits, symmetric, scale, zero, mask=None, stream=None) -> int:
    """Per-row min-max grid over kept entries; returns maxq."""
    _check(W, torch.float32, "W"); _check(scale, torch.float32, "scale"); _check(zero, torch.float32, "zero")
    _check(mask, torch.uint8, "mask")
    R, d = W.shape
    maxq = ctypes.c_int(0)
    _raise(load_library().obc_minmax_grid(_ptr(W), _ld(W), R, d, _ptr(mask), int(bits), int(bool(symmetric)),
                                          _ptr(scale), _ptr(zero), ctypes.byref(maxq), _stream(stream)), "obc_minmax_grid")
    return int(maxq.value)


def obc_quantize(W, Hinv, scale, zero, bits, symmetric, W_out, codes, row_status, prune_order=None,
                 prune_counts=None, flags=0, loss=None, qorder=None, row_begin=0, row_count=None, ws=None, opts=None, stream=None):
    """Algorithm 3 (OBQ); with prune_order/prune_counts: replay the pruning first, then quantise survivors."""
    _check(W, torch.float32, "W"); _check(Hinv, torch.float32, "Hinv"); _check(scale, torch.float32, "scale")
    _check(zero, torch.float32, "zero"); _check(W_out, torch.float32, "W_out"); _check(codes, torch.int32, "codes")
    _check(row_status, torch.int32, "row_status"); _check(prune_order, torch.int32, "prune_order")
    _check(prune_counts, torch.int32, "prune_counts"); _check(loss, torch.float32, "loss"); _check(qorder, torch.int32, "qorder")
    R, d = W.shape
    row_count = R - row_begin if row_count is None else row_count
    ws, nb = _workspace(ws, OP_QUANTIZE, row_count, d, 0, W.device, "obc_quantize")
    _raise(load_library().obc_quantize(_ptr(W), _ld(W), R, d, row_begin, row_count, _ptr(Hinv), _ld(Hinv), _ptr(scale),
                                       _ptr(zero), int(bits), int(bool(symmetric)), _ptr(prune_order), _ptr(prune_counts),
                                       int(flags), _ptr(W_out), _ld(W_out), _ptr(codes), _ptr(loss), _ptr(qorder),
                                       _ptr(row_status), _ptr(ws), nb, _opts(opts), _stream(stream)), "obc_quantize")
