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


@pytest.mark.parametrize("threads,d,extra", [(128, 300, 37), (256, 520, 11), (512, 520, 29), (0, 640, 5), (512, 1100, 3)])
def test_row_shares_prune_trace_quant_replay(threads, d, extra):
    import paper_2208_11580_b200 as m
    m.load_library()
    m = WithEngineOpts(m, m.ENGINE_BLOCKED, threads, 0)
    plan = m.obc_engine_plan(d, True, 0)
    grid = plan["rows_per_sm"] * plan["sm_count"]
    assert d > plan["on_chip_below"]
    rows = grid + extra                                   # one whole wave and a little: almost every block shares a row
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
