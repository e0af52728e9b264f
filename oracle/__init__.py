"""TEST INFRASTRUCTURE ONLY: FP64 CPU oracle of the ExactOBS / OBQ layer solver (Optimal Brain Compression).

Thin ctypes wrapper over obc_oracle.c plus the few steps that are plain library primitives in FP64
(the Hessian matmul for large layers, the block formulas used for the compound case).  Only tests, the
smoke check and the benchmark's CPU-baseline leg may import this package; the CUDA path never does, and
this package never imports the CUDA path.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "obc_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
FLAG_OUTLIERS = 1


def build(force: bool = False) -> str:
    """Compile obc_oracle.c with gcc (OpenMP over rows) next to its source; returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _L():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_inverse.restype = ctypes.c_int
        _lib.oracle_global_mask.restype = ctypes.c_int
    return _lib


def _p(a, ct):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ct))


def threads() -> int:
    """Number of host threads the row loop will use (OpenMP default = cores available to the process)."""
    return int(os.environ.get("OMP_NUM_THREADS", len(os.sched_getaffinity(0))))


# ---------------------------------------------------------------------------------------------------------
def hessian(X: np.ndarray, plain_loops: bool = False) -> np.ndarray:
    """H = 2 X X^T in FP64 (Section 3: Hessian of the per-row least-squares objective).

    plain_loops=True runs the C triple loop (small cases); otherwise the FP64 matmul primitive is used,
    accumulated over chunks of the calibration axis.
    """
    X = np.ascontiguousarray(X, dtype=np.float32)
    d, n = X.shape
    if plain_loops:
        H = np.empty((d, d), dtype=np.float64)
        _L().oracle_hessian(_p(X, ctypes.c_float), ctypes.c_int(d), ctypes.c_int64(n), _p(H, ctypes.c_double))
        return H
    H = np.zeros((d, d), dtype=np.float64)
    for c0 in range(0, n, 8192):
        xb = X[:, c0:c0 + 8192].astype(np.float64)
        H += xb @ xb.T
    return 2.0 * H


def inverse(H: np.ndarray, damp_rel: float):
    """(Hinv, info): inverse of H + damp_rel*mean(diag H)*I by the oracle's own Cholesky."""
    H = np.ascontiguousarray(H, dtype=np.float64)
    d = H.shape[0]
    Hinv = np.zeros((d, d), dtype=np.float64)
    info = _L().oracle_inverse(_p(H, ctypes.c_double), ctypes.c_int(d), ctypes.c_double(damp_rel),
                               _p(Hinv, ctypes.c_double))
    return Hinv, int(info)


def run_rows(Hinv, W, steps=None, mode="prune", scale=None, zero=None, maxq=0, flags=0,
             forced=None, active0=None, want_trace=False, nm=None):
    """Algorithm 1 (mode='prune') / Algorithm 3 (mode='quant') on every row of W with the shared Hinv.

    nm=(N, M): the N:M pattern of Section 3 ("N:M Sparsity", pruning only): a weight is a candidate only while its
    block of M consecutive columns has lost fewer than M - N weights; steps defaults to d (M - N) / M.

    Returns a dict: order, loss, margin, best, forced_gap, round_dist, pivot_diag (rows x steps), w (rows x d final
    weights), codes (rows x d, quant only), w_trace (rows x (steps+1) x d if want_trace), status (rows).
    """
    Hinv = np.ascontiguousarray(Hinv, dtype=np.float64)
    Wd = np.array(W, dtype=np.float64, order="C", copy=True)
    if Wd.ndim == 1:
        Wd = Wd[None, :]
    rows, d = Wd.shape
    assert Hinv.shape == (d, d)
    nm_prune, nm_block = 0, 0
    if nm is not None:
        n_keep, nm_block = int(nm[0]), int(nm[1])
        assert mode == "prune" and 0 < n_keep < nm_block and d % nm_block == 0
        nm_prune = nm_block - n_keep
        if steps is None:
            steps = d // nm_block * nm_prune
    steps = d if steps is None else int(steps)
    m = 1 if mode == "quant" else 0
    sc = None if scale is None else np.ascontiguousarray(np.broadcast_to(np.asarray(scale, np.float64), (rows,)))
    ze = None if zero is None else np.ascontiguousarray(np.broadcast_to(np.asarray(zero, np.float64), (rows,)))
    if m:
        assert sc is not None and ze is not None
    fo = None if forced is None else np.ascontiguousarray(np.asarray(forced, np.int32).reshape(rows, steps))
    a0 = None if active0 is None else np.ascontiguousarray(np.asarray(active0, np.uint8).reshape(rows, d))
    out = dict(
        order=np.full((rows, steps), -1, np.int32), loss=np.zeros((rows, steps)),
        margin=np.ones((rows, steps)), best=np.full((rows, steps), -1, np.int32),
        forced_gap=np.zeros((rows, steps)), round_dist=np.full((rows, steps), 0.5),
        pivot_diag=np.zeros((rows, steps)),
        codes=np.full((rows, d), -1, np.int32), status=np.zeros(rows, np.int32),
        w_trace=np.zeros((rows, steps + 1, d)) if want_trace else None)
    I32, F64, U8 = ctypes.c_int32, ctypes.c_double, ctypes.c_uint8
    _L().oracle_rows(_p(Hinv, F64), ctypes.c_int(d), ctypes.c_int(rows), _p(Wd, F64), ctypes.c_int(steps),
                     ctypes.c_int(m), _p(sc, F64), _p(ze, F64), ctypes.c_int(int(maxq)), ctypes.c_int(int(flags)),
                     _p(fo, I32), _p(a0, U8), _p(out["order"], I32), _p(out["loss"], F64),
                     _p(out["margin"], F64), _p(out["best"], I32), _p(out["forced_gap"], F64),
                     _p(out["round_dist"], F64), _p(out["pivot_diag"], F64), _p(out["w_trace"], F64), _p(out["codes"], I32),
                     _p(out["status"], I32), ctypes.c_int(nm_prune), ctypes.c_int(nm_block))
    out["w"] = Wd
    return out


def run_rows_blocks(Hinv, W, c: int, steps=None, forced_blocks=None, return_hi=False):
    """Block pruning (Section 3, "Block-Sparsity", Eq. 5) of every row of W: blocks of c consecutive weights are
    removed together, chosen by w_P^T ((Hinv)_P)^-1 w_P.  steps = number of blocks to remove (default all).
    Returns a dict: order, loss (rows x steps*c; a block's loss sits at its first member, zeros after it), margin,
    best_block, forced_gap (rows x steps), w (rows x d), status (rows), and Hi (list of matrices) if return_hi."""
    Hinv = np.ascontiguousarray(Hinv, dtype=np.float64)
    Wd = np.array(W, dtype=np.float64, order="C", copy=True)
    if Wd.ndim == 1:
        Wd = Wd[None, :]
    rows, d = Wd.shape
    assert 1 <= c <= 8 and d % c == 0
    steps = d // c if steps is None else int(steps)
    fo = None if forced_blocks is None else np.ascontiguousarray(np.asarray(forced_blocks, np.int32).reshape(rows, steps))
    out = dict(order=np.full((rows, steps * c), -1, np.int32), loss=np.zeros((rows, steps * c)),
               margin=np.ones((rows, steps)), best_block=np.full((rows, steps), -1, np.int32),
               forced_gap=np.zeros((rows, steps)), status=np.zeros(rows, np.int32))
    lib = _L()
    lib.oracle_row_blocks.restype = ctypes.c_int
    I32, F64 = ctypes.c_int32, ctypes.c_double
    his = []
    for r in range(rows):
        Hi = Hinv.copy()
        out["status"][r] = lib.oracle_row_blocks(_p(Hi, F64), ctypes.c_int(d), _p(Wd[r], F64), ctypes.c_int(c),
                                                 ctypes.c_int(steps), None if fo is None else _p(fo[r], I32),
                                                 _p(out["order"][r], I32), _p(out["loss"][r], F64),
                                                 _p(out["margin"][r], F64), _p(out["best_block"][r], I32),
                                                 _p(out["forced_gap"][r], F64))
        if return_hi:
            his.append(Hi)
    out["w"] = Wd
    if return_hi:
        out["Hi"] = his
    return out


def refit(X, Y, damp_rel: float):
    """Dense refit before sequential compression (appendix "Sequential Quantization with OBQ"): the closed-form
    least-squares weights W^T = (X X^T)^-1 X Y^T, with the solver's dampening: W = Y X^T (X X^T + (lambda/2) I)^-1,
    lambda = damp_rel * mean(diag(2 X X^T)), solved in FP64 with the library's linear solver."""
    X = np.asarray(X, dtype=np.float64)
    Y = np.asarray(Y, dtype=np.float64)
    d = X.shape[0]
    A = X @ X.T
    lam = damp_rel * np.trace(2.0 * A) / d
    return np.linalg.solve(A + 0.5 * lam * np.eye(d), X @ Y.T).T


def eliminate_one_row(Hinv, w, **kw):
    """Single-row variant that also returns the row's private Hinv copy after the steps ('Hi')."""
    Hi = np.array(Hinv, dtype=np.float64, order="C", copy=True)
    wd = np.array(w, dtype=np.float64, copy=True)
    d = wd.shape[0]
    steps = int(kw.get("steps", d))
    m = 1 if kw.get("mode", "prune") == "quant" else 0
    forced = kw.get("forced")
    fo = None if forced is None else np.ascontiguousarray(forced, dtype=np.int32)
    a0 = kw.get("active0")
    a0 = None if a0 is None else np.ascontiguousarray(a0, dtype=np.uint8)
    order = np.full(steps, -1, np.int32); loss = np.zeros(steps); margin = np.ones(steps)
    best = np.full(steps, -1, np.int32); gap = np.zeros(steps); rd = np.full(steps, 0.5)
    codes = np.full(d, -1, np.int32); trace = np.zeros((steps + 1, d)); pdg = np.zeros(steps)
    I32, F64, U8 = ctypes.c_int32, ctypes.c_double, ctypes.c_uint8
    lib = _L()
    lib.oracle_row.restype = ctypes.c_int
    st = lib.oracle_row(_p(Hi, F64), ctypes.c_int(d), _p(wd, F64), ctypes.c_int(steps), ctypes.c_int(m),
                        ctypes.c_double(float(kw.get("scale", 1.0))), ctypes.c_double(float(kw.get("zero", 0.0))),
                        ctypes.c_int(int(kw.get("maxq", 0))), ctypes.c_int(int(kw.get("flags", 0))),
                        _p(fo, I32), _p(a0, U8), _p(order, I32), _p(loss, F64), _p(margin, F64), _p(best, I32),
                        _p(gap, F64), _p(rd, F64), _p(pdg, F64), _p(trace, F64), _p(codes, I32),
                        ctypes.c_int(int(kw.get("nm_prune", 0))), ctypes.c_int(int(kw.get("nm_block", 0))))
    return dict(Hi=Hi, w=wd, order=order, loss=loss, margin=margin, best=best, forced_gap=gap,
                round_dist=rd, pivot_diag=pdg, codes=codes, w_trace=trace, status=int(st))


def global_mask(loss, order, k: int):
    """Algorithm 2 with a literal min-heap: (counts, mask) for k pruned weights; mask 1 = kept."""
    L = np.ascontiguousarray(loss, dtype=np.float64)
    P = np.ascontiguousarray(order, dtype=np.int32)
    rows, d = L.shape
    counts = np.zeros(rows, np.int32)
    mask = np.ones((rows, d), np.uint8)
    rc = _L().oracle_global_mask(_p(L, ctypes.c_double), _p(P, ctypes.c_int32), ctypes.c_int(rows),
                                 ctypes.c_int(d), ctypes.c_int64(int(k)), _p(counts, ctypes.c_int32),
                                 _p(mask, ctypes.c_uint8))
    if rc:
        raise ValueError("k out of range")
    return counts, mask


def minmax_grid(W, bits: int, symmetric: bool, mask=None):
    """Per-row min-max grid (scale, zero, maxq) over the kept entries; the range always contains 0."""
    Wd = np.ascontiguousarray(W, dtype=np.float64)
    rows, d = Wd.shape
    mk = None if mask is None else np.ascontiguousarray(mask, dtype=np.uint8)
    scale = np.zeros(rows); zero = np.zeros(rows); maxq = ctypes.c_int32(0)
    _L().oracle_minmax_grid(_p(Wd, ctypes.c_double), ctypes.c_int(rows), ctypes.c_int(d), _p(mk, ctypes.c_uint8),
                            ctypes.c_int(bits), ctypes.c_int(1 if symmetric else 0), _p(scale, ctypes.c_double),
                            _p(zero, ctypes.c_double), ctypes.byref(maxq))
    return scale, zero, int(maxq.value)


def weights_from_trace(w_trace, counts):
    """Figure 1, 'more memory' option: the row's weight vector after its first counts[r] eliminations."""
    return np.stack([w_trace[r, int(c)] for r, c in enumerate(counts)])


def group_obs_state(Hinv, w0, pruned_idx):
    """Block (group-OBS) formulas, Eq. 5 with the minus sign, evaluated directly with FP64 solves:
    removing the index set P at once gives  w_F = w0_F - Hinv[F,P] inv(Hinv[P,P]) w0_P  and the reduced
    inverse  inv(H[F,F]) = Hinv[F,F] - Hinv[F,P] inv(Hinv[P,P]) Hinv[P,F].  Returns (F, w_F, HiF)."""
    Hinv = np.asarray(Hinv, dtype=np.float64)
    d = Hinv.shape[0]
    P = np.asarray(sorted(int(i) for i in pruned_idx), dtype=np.int64)
    keep = np.ones(d, bool)
    keep[P] = False
    F = np.nonzero(keep)[0]
    w0 = np.asarray(w0, dtype=np.float64)
    if P.size == 0:
        return F, w0.copy(), Hinv.copy()
    App = Hinv[np.ix_(P, P)]
    Afp = Hinv[np.ix_(F, P)]
    sol = np.linalg.solve(App, np.concatenate([w0[P][:, None], Afp.T], axis=1))
    wF = w0[F] - Afp @ sol[:, 0]
    HiF = Hinv[np.ix_(F, F)] - Afp @ sol[:, 1:]
    return F, wF, 0.5 * (HiF + HiF.T)


def compound_row(Hinv, w0, pruned_idx, bits, symmetric, grid=None, flags=0):
    """Sparsify first, then quantise the remaining weights (Section 6 'Experimental Setup'; Section 3 on
    already-sparse rows): the survivors' sub-problem is formed directly by group_obs_state, the grid is
    the min-max grid of the compensated survivors unless `grid`=(scale, zero, maxq) is given, then
    Algorithm 3 runs on the |F|-dimensional problem and the result is scattered back (pruned entries 0).
    """
    F, wF, HiF = group_obs_state(Hinv, w0, pruned_idx)
    d = len(w0)
    if grid is None:
        sc, ze, mq = minmax_grid(wF[None, :], bits, symmetric)
        sc, ze = float(sc[0]), float(ze[0])
    else:
        sc, ze, mq = float(grid[0]), float(grid[1]), int(grid[2])
    res = dict(F=F, wF=wF, scale=sc, zero=ze, maxq=mq, w=np.zeros(d), codes=np.full(d, -1, np.int32))
    if len(F):
        r = run_rows(HiF, wF[None, :], mode="quant", scale=[sc], zero=[ze], maxq=mq, flags=flags)
        res["w"][F] = r["w"][0]
        res["codes"][F] = r["codes"][0]
        res["order"] = F[r["order"][0]]
        res["loss"] = r["loss"][0]
        res["margin"] = r["margin"][0]
        res["round_dist"] = r["round_dist"][0]
    return res
