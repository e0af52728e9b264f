"""Blocked engine with more rows than resident blocks that do not divide evenly: every block gets the same amount of
work, so some rows are started by one block and finished by the next (state handed over at a flush boundary).  All
modes that support it, every thread count, against the oracle on every row; results must also be bit-identical to
the same rows run in calls small enough to need no hand-over (the arithmetic of a row does not depend on which block
runs which part of it -- only a pass over its matrix is forced at the hand-over)."""
import numpy as np
import pytest
import torch

import obc_synth
import oracle
from parity import check_rows, REL_TOL, WithEngineOpts

pytestmark = pytest.mark.gpu
DAMP = obc_synth.DAMP_REL


def _padded(a, ld):
    r, c = a.shape
    buf = torch.zeros(r, ld, dtype=torch.float32, device="cuda")
    buf[:, :c] = torch.from_numpy(a)
    return buf[:, :c]


def _sm_count():
    return torch.cuda.get_device_properties(0).multi_processor_count


@pytest.mark.parametrize("threads,d,extra,waves", [(128, 300, 37, 1), (256, 520, 11, 1), (512, 520, 29, 1), (0, 640, 5, 1),
                                                   (512, 1100, 3, 1), (512, 520, 61, 4), (256, 400, 100, 2)])
def test_row_shares_prune_trace_quant_replay(threads, d, extra, waves):
    import paper_2208_11580_b200 as m
    m.load_library()
    m = WithEngineOpts(m, m.ENGINE_BLOCKED, threads, 0)
    plan = m.obc_engine_plan(d, True, 0)
    grid = plan["rows_per_sm"] * plan["sm_count"]
    assert d > plan["on_chip_below"]
    # whole waves and a little: almost every block shares a row (with one row per SM shares are taken at any number of
    # waves, otherwise up to three)
    rows = waves * grid + extra
    W, X = obc_synth.make_small(rows, d, 3 * d + 64, 5100 + d, "relu")
    H = oracle.hessian(X).astype(np.float32)
    ld = (d + 3) // 4 * 4
    Hinv, info = m.obc_hessian_inverse(_padded(H, ld), DAMP)
    assert int(info.item()) == 0
    Hh = Hinv.cpu().numpy()
    Wd = _padded(W, ld)
    i32 = lambda *s, fill=0: torch.full(s, fill, dtype=torch.int32, device="cuda")
    f32 = lambda *s: torch.zeros(*s, dtype=torch.float32, device="cuda")
    # ---- prune trace with the full weight trace --------------------------------------------------------------
    order, loss, rs, trace = i32(rows, d, fill=-7), f32(rows, d), i32(rows, fill=-7), f32(rows, d + 1, d)
    m.obc_prune_trace(Wd, Hinv, order, loss, rs, w_trace=trace)
    torch.cuda.synchronize()
    assert int(rs.abs().sum()) == 0
    sample = np.unique(np.concatenate([np.arange(0, rows, max(1, rows // 24)), [rows - 1]]))
    P, L = order.cpu().numpy(), loss.cpu().numpy()
    assert np.array_equal(np.sort(P, axis=1), np.broadcast_to(np.arange(d), (rows, d)))
    st = check_rows(Hh, W[sample], P[sample], L[sample], gpu_trace=trace[torch.from_numpy(sample).cuda()].cpu().numpy())
    # the same rows in calls of at most `grid` rows (no hand-over): identical picks, losses within rounding of the
    # one extra pass over the matrix at a hand-over
    o2, l2, r2 = i32(rows, d), f32(rows, d), i32(rows)
    for b in range(0, rows, grid):
        m.obc_prune_trace(Wd, Hinv, o2, l2, r2, row_begin=b, row_count=min(grid, rows - b))
    torch.cuda.synchronize()
    same = (o2 == order).all(dim=1).cpu().numpy()
    assert same.mean() > 0.9, "orders of handed-over rows should match the plain run except at sub-margin ties"
    rel = (l2 - loss).abs() / (loss.abs() + 1e-7 * loss.abs().max(dim=1, keepdim=True).values)
    assert float(rel[torch.from_numpy(same).cuda()].max()) <= REL_TOL
    # ---- OBQ -------------------------------------------------------------------------------------------------------
    scale, zero = f32(rows), f32(rows)
    maxq = m.obc_minmax_grid(Wd, 4, False, scale, zero)
    Wq, codes, ql, qo = f32(rows, d), i32(rows, d), f32(rows, d), i32(rows, d)
    m.obc_quantize(Wd, Hinv, scale, zero, 4, False, Wq, codes, rs, loss=ql, qorder=qo)
    torch.cuda.synchronize()
    assert int(rs.abs().sum()) == 0
    check_rows(Hh, W[sample], qo.cpu().numpy()[sample], ql.cpu().numpy()[sample], gpu_w=Wq.cpu().numpy()[sample], mode="quant",
               scale=scale.cpu().numpy().astype(np.float64)[sample], zero=zero.cpu().numpy().astype(np.float64)[sample],
               maxq=maxq, gpu_codes=codes.cpu().numpy()[sample])
    # ---- forced replay, and replay followed by OBQ of the survivors -------------------------------------------------
    rng = np.random.default_rng(d)
    cnt = rng.integers(0, d + 1, size=rows).astype(np.int32)
    counts = torch.from_numpy(cnt).cuda()
    got = f32(rows, d)
    m.obc_prune_apply(Wd, Hinv, order, counts, got, rs)
    ref = f32(rows, d)
    m.obc_prune_apply(Wd, Hinv, order, counts, ref, rs, w_trace=trace, trace_steps=d)
    torch.cuda.synchronize()
    assert int(rs.abs().sum()) == 0
    wscale = np.abs(W).max(axis=1, keepdims=True)
    gr = ref.cpu().numpy()
    assert (np.abs(got.cpu().numpy() - gr) / np.maximum(np.abs(gr), wscale)).max() <= 2 * REL_TOL
    cnt2 = np.minimum(cnt, d - 8).astype(np.int32)
    counts2 = torch.from_numpy(cnt2).cuda()
    m.obc_quantize(Wd, Hinv, scale, zero, 4, True, Wq, codes, rs, prune_order=order, prune_counts=counts2, loss=ql, qorder=qo)
    torch.cuda.synchronize()
    assert int(rs.abs().sum()) == 0
    gq, gc = Wq.cpu().numpy(), codes.cpu().numpy()
    H64 = Hh.astype(np.float64)
    for r in sample[:6]:
        pruned = P[r, :cnt2[r]]
        F, wF, HiF = oracle.group_obs_state(H64, W[r], pruned)
        assert np.all(gq[r, pruned] == 0.0) and np.all(gc[r, pruned] == -1)
        pos = {int(j): i for i, j in enumerate(F)}
        nF = len(F)
        forced = np.array([pos[int(j)] for j in qo.cpu().numpy()[r, :nF]], dtype=np.int32)
        check_rows(HiF, wF[None, :], forced[None, :], ql.cpu().numpy()[r:r + 1, :nF], gpu_w=gq[r, F][None, :], mode="quant",
                   scale=np.array([float(scale[r].item())]), zero=np.array([float(zero[r].item())]), maxq=14,
                   gpu_codes=gc[r, F][None, :])
    print("row shares", threads, d, rows, {k: v for k, v in st.items() if k not in ("oracle", "trace_rows_max_rel")})


@pytest.mark.parametrize("d", [120, 160, 200, 236, 300])
def test_workspace_query_is_valid_for_every_engine_option(d):
    """obc_workspace_bytes does not know the options a call will carry: the size it reports must do for every thread
    count and both engines (row lengths around the on-chip thresholds, which differ by thread count)"""
    import paper_2208_11580_b200 as m
    m.load_library()
    rows = 5
    W, X = obc_synth.make_small(rows, d, 3 * d + 64, 6100 + d, "relu")
    H = oracle.hessian(X).astype(np.float32)
    ld = (d + 3) // 4 * 4
    Hinv, info = m.obc_hessian_inverse(_padded(H, ld), DAMP)
    Wd = _padded(W, ld)
    ws = torch.empty(m.obc_workspace_bytes(m.OP_PRUNE_TRACE, rows, d), dtype=torch.uint8, device="cuda")
    ref = None
    for opts in [(m.ENGINE_BLOCKED, 128, 0), (m.ENGINE_BLOCKED, 256, 0), (m.ENGINE_BLOCKED, 512, 0), (m.ENGINE_BLOCKED, 0, 3),
                 (m.ENGINE_STREAMING, 0, 0), (m.ENGINE_BLOCKED, 256, 0, m.ENGINE_WHOLE_WAVES)]:
        order = torch.full((rows, d), -7, dtype=torch.int32, device="cuda")
        loss = torch.zeros(rows, d, dtype=torch.float32, device="cuda")
        rs = torch.full((rows,), -7, dtype=torch.int32, device="cuda")
        m.obc_prune_trace(Wd, Hinv, order, loss, rs, ws=ws, opts=opts)        # raises on OBC_ERR_WORKSPACE
        torch.cuda.synchronize()
        assert int(rs.abs().sum()) == 0
        if ref is None:
            ref = order.clone()
            check_rows(Hinv.cpu().numpy(), W, order.cpu().numpy(), loss.cpu().numpy())
        else:
            assert (order == ref).float().mean() > 0.99


def test_row_shares_partial_trace_and_failing_rows():
    """rows handed over between blocks with a partial trace (steps < d_col); rows that fail late (a non-finite weight is
    met when nothing else is left: in the part the second block runs) and early (a replayed order that names a column
    twice: in the part the first block runs): their status is reported, every other row is unaffected"""
    import paper_2208_11580_b200 as m
    m.load_library()
    raw = m
    m = WithEngineOpts(raw, raw.ENGINE_BLOCKED, 512, 0)
    whole = WithEngineOpts(raw, raw.ENGINE_BLOCKED, 512, 0, raw.ENGINE_WHOLE_WAVES)
    d = 520
    plan = m.obc_engine_plan(d, False, 0)
    grid = plan["rows_per_sm"] * plan["sm_count"]
    rows = grid + grid // 2 + 3
    W, X = obc_synth.make_small(rows, d, 3 * d + 64, 7100, "relu")
    H = oracle.hessian(X).astype(np.float32)
    ld = (d + 3) // 4 * 4
    Hinv, info = m.obc_hessian_inverse(_padded(H, ld), DAMP)
    Hh = Hinv.cpu().numpy()
    i32 = lambda *s, fill=-7: torch.full(s, fill, dtype=torch.int32, device="cuda")
    f32 = lambda *s: torch.full(s, -7.0, dtype=torch.float32, device="cuda")
    sample = np.arange(0, rows, max(1, rows // 20))
    # ---- partial trace ---------------------------------------------------------------------------------------------
    steps = d // 3
    Wd = _padded(W, ld)
    order, loss, rs = i32(rows, d), f32(rows, d), i32(rows)
    m.obc_prune_trace(Wd, Hinv, order, loss, rs, steps=steps)
    o2, l2, r2 = i32(rows, d), f32(rows, d), i32(rows)
    whole.obc_prune_trace(Wd, Hinv, o2, l2, r2, steps=steps)
    torch.cuda.synchronize()
    assert int(rs.abs().sum()) == 0 and int(r2.abs().sum()) == 0
    o, l = order.cpu().numpy(), loss.cpu().numpy()
    assert np.all(o[:, steps:] == -7) and np.all(l[:, steps:] == -7.0)
    check_rows(Hh, W[sample], o[sample], l[sample], steps=steps)
    assert (o2 == order).float().mean() > 0.995
    # ---- rows that fail in their last steps ------------------------------------------------------------------------
    bad = np.array([1, grid // 3, grid, rows - 2])
    Wb = W.copy()
    Wb[bad, 7] = np.nan
    order, loss, rs = i32(rows, d), f32(rows, d), i32(rows)
    m.obc_prune_trace(_padded(Wb, ld), Hinv, order, loss, rs)
    torch.cuda.synchronize()
    st = rs.cpu().numpy()
    good = np.setdiff1d(np.arange(rows), bad)
    assert np.all(st[good] == 0) and np.all(st[bad] >= 1)
    o, l = order.cpu().numpy(), loss.cpu().numpy()
    for b in bad:
        assert np.all(o[b, st[b] - 1:] == -1) and np.all(np.isinf(l[b, st[b] - 1:]))
    gs = good[:: max(1, len(good) // 12)]
    check_rows(Hh, W[gs], o[gs], l[gs])
    # ---- rows that fail early in a forced replay (the order names its first column again at step 2) ------------------
    full_o = torch.from_numpy(o).cuda()
    full_o[torch.from_numpy(bad).cuda()] = full_o[torch.from_numpy(good[:len(bad)]).cuda()]      # valid orders for those rows
    bad_o = full_o.clone()
    bad_o[torch.from_numpy(bad).cuda(), 2] = bad_o[torch.from_numpy(bad).cuda(), 0]
    counts = torch.full((rows,), d - 40, dtype=torch.int32, device="cuda")
    out, rsa = f32(rows, d), i32(rows)
    m.obc_prune_apply(Wd, Hinv, bad_o, counts, out, rsa)
    ref, rsb = f32(rows, d), i32(rows)
    whole.obc_prune_apply(Wd, Hinv, full_o, counts, ref, rsb)
    torch.cuda.synchronize()
    sa = rsa.cpu().numpy()
    assert np.all(sa[bad] == 1 + 2) and np.all(sa[good] == 0) and int(rsb.abs().sum()) == 0
    g, r = out.cpu().numpy()[good], ref.cpu().numpy()[good]
    wscale = np.abs(W[good]).max(axis=1, keepdims=True)
    assert (np.abs(g - r) / np.maximum(np.abs(r), wscale)).max() <= 2 * REL_TOL
