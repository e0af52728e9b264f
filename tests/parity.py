"""Shared machinery of the GPU-vs-oracle parity tests (margin-gated, teacher-forced comparison).

The greedy order is chaotic: one flipped pick changes everything after it in that row.  So the oracle is
run along the order the GPU chose (teacher forcing) and reports, for every step, its own best pick at that
state and the relative score gap between the forced pick and its best.  A GPU pick passes if it IS the
oracle's pick, or if that gap is within MARGIN_TOL (a tie within the selection margin).  Loss traces and
weights are then compared along the common trajectory.
"""
import json
import os

import numpy as np

import oracle

MARGIN_TOL = 1e-6      # picks must agree wherever best and forced scores differ by more than this (relative)
OBQ_GATE_CAP = 4e-5    # upper limit of the OBQ pick gate (see check_rows)
REL_TOL = 1e-4         # loss traces and weights: relative error bound in FP32.  Weights are compared relative to
                       # max(|reference entry|, largest initial weight of the row): late in a row the few remaining
                       # weights carry the compensation of all the others and grow to several times the initial scale
ROUND_TOL = 1e-4       # integer codes may differ only if x/Delta is this close to a rounding boundary


def check_rows(Hinv32, W32, gpu_order, gpu_loss, gpu_w=None, *, mode="prune", scale=None, zero=None, maxq=0,
               flags=0, gpu_codes=None, gpu_trace=None, steps=None, active0=None, nm=None):
    """Compare GPU results for a set of rows with the oracle fed the same FP32 Hinv / W.
    Returns a dict of statistics; raises AssertionError on a parity violation."""
    Hinv = np.asarray(Hinv32, dtype=np.float64)
    W = np.asarray(W32, dtype=np.float64)
    rows, d = W.shape
    steps = d if steps is None else steps
    gpu_order = np.asarray(gpu_order)[:, :steps]
    res = oracle.run_rows(Hinv, W, steps=steps, mode=mode, scale=scale, zero=zero, maxq=maxq, flags=flags,
                          forced=gpu_order, active0=active0, want_trace=gpu_trace is not None, nm=nm)
    assert np.all(res["status"] == 0), f"oracle rejected the GPU order: {res['status']}"
    differ = res["best"] != gpu_order
    gap = res["forced_gap"]
    if mode == "quant":
        # OBQ scores are squared DIFFERENCES w - q(w) over the pivot diagonal, so their natural scale is the score
        # of a half-step error at that pivot, (Delta/2)^2/[Hinv]_pp; the margin is taken relative to
        # max(score, that scale): a tiny score is only known to the absolute accuracy of w.
        half = 0.5 * np.broadcast_to(np.asarray(scale, dtype=np.float64), (rows,))[:, None]
        s_f = res["loss"]
        s_ref = np.maximum(s_f, half * half / np.maximum(res["pivot_diag"], 1e-300))
        gap = gap * s_f / np.maximum(s_ref, 1e-300)
        # The FP32 pipeline resolves a row's weights to a few roundings of its largest weight,
        # |dw| <= 2.5e-7 max|w| (4 * 2^-24), and a half-step score moves by the relative amount 4 |dw| / Delta
        # under such a perturbation.  The 1e-6 margin is therefore taken on the weight scale: picks whose
        # scores differ by less than 1e-6 * max|w| / Delta of the half-step score are ties.
        # That bound is 1.3e-4 on an 8-bit grid; the largest gap seen at a differing pick is 1.9e-5 (the 8-bit compound
        # configuration, streaming engine), so the gate is capped at about twice that.
        wmax = np.abs(W).max(axis=1, keepdims=True)
        tol = np.minimum(MARGIN_TOL * np.maximum(1.0, wmax / (2.0 * half)), OBQ_GATE_CAP)
    else:
        tol = MARGIN_TOL
    bad = differ & (gap > tol)
    stats = dict(steps=int(rows * steps), picks_differ=int(differ.sum()), max_gap_at_differ=float(gap[differ].max()) if differ.any() else 0.0,
                 max_gap_over_tol=float((gap / tol)[differ].max()) if differ.any() else 0.0,
                 # differing picks whose gap lies above the plain 1e-6 margin (all of them inside the gate, or the
                 # assertion below fails): the ones the weight-scale reading of the margin lets through
                 picks_differ_gap_over_1e6=int((differ & (gap > MARGIN_TOL)).sum()),
                 gate=float(np.max(tol)),
                 sub_1e5_margin=int((res["margin"] < 1e-5).sum()))
    assert not bad.any(), (f"{int(bad.sum())} picks differ beyond the margin; first at row/step "
                           f"{np.argwhere(bad)[0].tolist()}, gap {gap[bad][0]:.3e}")
    L = res["loss"]
    gl = np.asarray(gpu_loss, dtype=np.float64)[:, :steps]
    floor = 1e-7 * np.abs(L).max(axis=1, keepdims=True)
    if mode == "quant":
        # the quantisation loss is a squared DIFFERENCE w - q(w): an absolute weight error within the weight
        # tolerance moves it by up to ~REL_TOL of the loss of a half-step error at that pivot
        half = 0.5 * np.broadcast_to(np.asarray(scale, dtype=np.float64), (rows,))[:, None]
        floor = np.maximum(floor, half * half / res["pivot_diag"])
    err = np.abs(gl - L) / (np.abs(L) + floor + 1e-300)
    stats["loss_max_rel"] = float(err.max())
    big = np.abs(L) >= 1e-3 * np.abs(L).max(axis=1, keepdims=True)      # against |L| alone, where L is not tiny
    stats["loss_max_rel_unfloored"] = float((np.abs(gl - L) / np.maximum(np.abs(L), 1e-300))[big].max()) if big.any() else 0.0
    assert err.max() <= REL_TOL, f"loss trace off by {err.max():.3e} at {np.unravel_index(err.argmax(), err.shape)}"
    if gpu_w is not None:
        gw = np.asarray(gpu_w, dtype=np.float64)
        wscale = np.abs(W).max(axis=1, keepdims=True)
        if mode == "quant" and gpu_codes is not None:
            gc = np.asarray(gpu_codes)
            cd = gc != res["codes"]
            if active0 is not None:
                cd &= np.asarray(active0, bool)
            # a differing code is only tolerated where the quotient sat on a rounding boundary
            rd_by_col = np.full((rows, d), 1.0)
            np.put_along_axis(rd_by_col, gpu_order.astype(np.int64), res["round_dist"], axis=1)
            stats["codes_differ"] = int(cd.sum())
            assert not (cd & (rd_by_col > ROUND_TOL)).any(), "integer codes differ away from rounding boundaries"
            same = ~cd
            werr = np.abs(gw - res["w"]) / np.maximum(np.abs(res["w"]), wscale)
            stats["w_max_rel"] = float(werr[same].max()) if same.any() else 0.0
            assert werr[same].max() <= REL_TOL
        else:
            werr = np.abs(gw - res["w"]) / np.maximum(np.abs(res["w"]), wscale)
            stats["w_max_rel"] = float(werr.max())
            assert werr.max() <= REL_TOL, f"weights off by {werr.max():.3e}"
    if gpu_trace is not None:
        gt = np.asarray(gpu_trace, dtype=np.float64)
        wscale = np.abs(W).max(axis=1)[:, None, None]
        terr = np.abs(gt - res["w_trace"]) / np.maximum(np.abs(res["w_trace"]), wscale)
        stats["trace_max_rel"] = float(terr.max())
        stats["trace_max_over_initial_scale"] = float((np.abs(gt - res["w_trace"]) / wscale).max())
        stats["trace_rows_max_rel"] = [float(x) for x in terr.reshape(rows, -1).max(axis=1)]
        assert terr.max() <= REL_TOL, (f"weight trace off by {terr.max():.3e} at (row, step, column) "
                                       f"{np.unravel_index(terr.argmax(), terr.shape)}; per row {stats['trace_rows_max_rel']}")
    stats["oracle"] = res
    return stats



def record_stats(label, stats):
    """Prints one line of parity statistics (picks that differ, gaps, errors) and, when the environment variable
    OBC_PARITY_STATS names a file, appends it there as JSON."""
    rec = {"case": label, **{k: v for k, v in stats.items() if k != "oracle"}}
    print(label, rec)
    path = os.environ.get("OBC_PARITY_STATS")
    if not path:
        return
    try:
        os.makedirs(os.path.dirname(os.path.abspath(path)), exist_ok=True)
        with open(path, "a") as f:
            f.write(json.dumps(rec) + "\n")
    except OSError:
        pass


class WithEngineOpts:
    """The binding module with per-call engine options (engine, threads, max_pending) added to every row-engine
    call that does not name its own: lets one test body run under several engine choices without any library state."""
    _ENGINE_CALLS = ("obc_prune_trace", "obc_prune_apply", "obc_quantize", "obc_prune_nm", "obc_prune_blocks",
                     "obc_engine_plan")

    def __init__(self, module, engine=0, threads=0, max_pending=0, flags=0):
        self._m = module
        self.engine_name = {0: "auto", 1: "streaming", 2: "blocked"}.get(int(engine), str(engine))
        self.opts = module.engine_opts(engine, threads, max_pending, flags)

    def __getattr__(self, name):
        f = getattr(self._m, name)
        if name in self._ENGINE_CALLS:
            def call(*a, **k):
                k.setdefault("opts", self.opts)
                return f(*a, **k)
            return call
        return f
