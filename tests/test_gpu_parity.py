"""GPU parity tests: every stage of the CUDA path, called through the C ABI, against the FP64 oracle."""
import numpy as np
import pytest
import torch

import obc_synth
import oracle
from parity import check_rows, REL_TOL, WithEngineOpts

pytestmark = pytest.mark.gpu
DAMP = obc_synth.DAMP_REL


@pytest.fixture(scope="module", params=["blocked", "streaming"])
def obc(request):
    """the library with one of its two row elimination engines selected; every test runs with both"""
    import paper_2208_11580_b200 as m
    m.load_library()
    return WithEngineOpts(m, m.ENGINE_BLOCKED if request.param == "blocked" else m.ENGINE_STREAMING)


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t if dtype is None else t.to(dtype)


def padded(a, ld):
    """device copy of a 2-D float32 array with leading dimension ld (a view of a wider buffer)"""
    r, c = a.shape
    buf = torch.zeros(r, ld, dtype=torch.float32, device="cuda")
    buf[:, :c] = torch.from_numpy(a)
    return buf[:, :c]


def gpu_hinv(obc, X, prec=0):
    d = X.shape[0]
    Xd = dev(X)
    H = torch.empty(d, d, dtype=torch.float32, device="cuda")
    obc.obc_hessian(Xd, H, prec=prec)
    Hinv, info = obc.obc_hessian_inverse(H, DAMP)
    assert int(info.item()) == 0
    return H, Hinv


def run_trace(obc, Wd, Hinv, steps=None, want_trace=False, row_begin=0, row_count=None):
    R, d = Wd.shape
    steps = d if steps is None else steps
    order = torch.full((R, d), -7, dtype=torch.int32, device="cuda")
    loss = torch.full((R, d), -7.0, dtype=torch.float32, device="cuda")
    status = torch.full((R,), -7, dtype=torch.int32, device="cuda")
    trace = torch.zeros(R, steps + 1, d, dtype=torch.float32, device="cuda") if want_trace else None
    obc.obc_prune_trace(Wd, Hinv, order, loss, status, steps=steps, w_trace=trace, row_begin=row_begin, row_count=row_count)
    torch.cuda.synchronize()
    return order, loss, status, trace


# ---------------------------------------------------------------------------------------------------------------
HESSIAN_TOL = {0: 2e-5, 1: 2e-3, 2: 3e-5}     # FP32 CUDA cores, TF32 and BF16x3 tensor cores; relative to max|H|


@pytest.mark.parametrize("prec", [0, 1, 2])
@pytest.mark.parametrize("d,n", [(64, 1024), (5, 37), (130, 4100), (576, 2048), (300, 20000)])
def test_hessian_matches_fp64(obc, d, n, prec):
    _, X = obc_synth.make_small(1, d, n, 100 + d)
    ldx = (n + 3) // 4 * 4
    Xd = padded(X, ldx)
    ldh = (d + 3) // 4 * 4
    H = torch.zeros(d, ldh, dtype=torch.float32, device="cuda")[:, :d]
    obc.obc_hessian(Xd, H, prec=prec)
    ref = oracle.hessian(X)
    got = H.cpu().numpy().astype(np.float64)
    assert np.array_equal(got, got.T)
    tol = HESSIAN_TOL[prec]
    print("hessian", d, n, prec, np.abs(got - ref).max() / np.abs(ref).max())
    assert np.abs(got - ref).max() <= tol * np.abs(ref).max()
    # accumulation over chunks of the calibration axis
    H2 = torch.zeros(d, ldh, dtype=torch.float32, device="cuda")[:, :d]
    h = (n // 2 + 3) // 4 * 4
    obc.obc_hessian(Xd[:, :h], H2, accumulate=False, prec=prec)
    obc.obc_hessian(Xd[:, h:], H2, accumulate=True, prec=prec)
    assert np.abs(H2.cpu().numpy() - ref).max() <= tol * np.abs(ref).max()


@pytest.mark.parametrize("d", [5, 48, 64, 100, 576, 1000])
def test_inverse_matches_oracle(obc, d):
    _, X = obc_synth.make_small(1, d, 2 * d + 50, 200 + d, "relu")
    H64 = oracle.hessian(X)
    H32 = H64.astype(np.float32)
    ld = (d + 3) // 4 * 4
    Hinv, info = obc.obc_hessian_inverse(padded(H32, ld), DAMP)
    ref, oinfo = oracle.inverse(H32.astype(np.float64), DAMP)
    assert int(info.item()) == 0 and oinfo == 0
    got = Hinv.cpu().numpy()
    assert np.array_equal(got, got.T)
    # FP64 inside, one FP32 rounding at the end
    assert np.abs(got - ref).max() <= 2e-7 * np.abs(ref).max() + 1e-30
    lam = DAMP * np.trace(H32.astype(np.float64)) / d
    resid = got.astype(np.float64) @ (H32.astype(np.float64) + lam * np.eye(d)) - np.eye(d)
    assert np.abs(resid).max() < 1e-3


def test_inverse_reports_non_positive_definite(obc):
    X = np.random.default_rng(0).normal(size=(8, 40)).astype(np.float32)
    X[5] = X[2]
    H = oracle.hessian(X).astype(np.float32)
    # indefinite (smallest eigenvalue -1): some pivot is negative whatever the rounding, and it cannot come before
    # the first leading minor that is not positive definite
    Hneg = (H - np.eye(8, dtype=np.float32)).astype(np.float32)
    _, info = obc.obc_hessian_inverse(dev(Hneg), 0.0)
    _, oinfo = oracle.inverse(Hneg.astype(np.float64), 0.0)
    assert oinfo > 0 and int(info.item()) == oinfo
    # exactly singular: the pivot of the duplicated row is zero up to rounding, so it is either reported or the
    # result blows up
    Hi, info = obc.obc_hessian_inverse(dev(H), 0.0)
    _, oinfo = oracle.inverse(H.astype(np.float64), 0.0)
    assert oinfo > 0
    assert int(info.item()) > 0 or not np.isfinite(Hi.cpu().numpy()).all() or np.abs(Hi.cpu().numpy()).max() > 1e3


# ---------------------------------------------------------------------------------------------------------------
def test_config1_full_pipeline(obc):
    """benchmark configuration C1: 32x64 layer; full prune trace -> 50% global mask -> weights; 4-bit symmetric OBQ."""
    W, X, spec = obc_synth.make_layer("C1")
    R, d = W.shape
    H, Hinv = gpu_hinv(obc, X)
    Href = oracle.hessian(X)
    assert np.abs(H.cpu().numpy() - Href).max() <= 2e-5 * np.abs(Href).max()
    Wd = dev(W)
    order, loss, status, trace = run_trace(obc, Wd, Hinv, want_trace=True)
    assert int(status.abs().sum()) == 0
    Hinv_h = Hinv.cpu().numpy()
    st = check_rows(Hinv_h, W, order.cpu().numpy(), loss.cpu().numpy(), gpu_w=trace[:, -1].cpu().numpy(),
                    gpu_trace=trace.cpu().numpy())
    assert np.all(trace[:, -1].cpu().numpy() == 0.0)
    # global step on the GPU's own L, P: bit-exact against the heap
    k = obc_synth.pruned_count(R, d, 0.5)
    counts = torch.zeros(R, dtype=torch.int32, device="cuda")
    mask = torch.zeros(R, d, dtype=torch.uint8, device="cuda")
    obc.obc_select_global_mask(loss, order, k, counts, mask)
    oc, om = oracle.global_mask(loss.cpu().numpy(), order.cpu().numpy(), k)
    assert np.array_equal(counts.cpu().numpy(), oc) and np.array_equal(mask.cpu().numpy(), om)
    # final weights: trace gather and forced-order replay agree with the oracle's trace reload
    want = oracle.weights_from_trace(st["oracle"]["w_trace"], oc)
    wscale = np.abs(W).max(axis=1, keepdims=True)
    out1 = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    rs = torch.zeros(R, dtype=torch.int32, device="cuda")
    obc.obc_prune_apply(Wd, Hinv, order, counts, out1, rs, w_trace=trace, trace_steps=d)
    out2 = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    obc.obc_prune_apply(Wd, Hinv, order, counts, out2, rs)
    for out in (out1, out2):
        o = out.cpu().numpy()
        assert np.all(o[om == 0] == 0.0)
        assert (np.abs(o - want) / wscale).max() <= REL_TOL
    # OBQ, 4-bit symmetric min-max grid
    scale = torch.zeros(R, dtype=torch.float32, device="cuda")
    zero = torch.zeros(R, dtype=torch.float32, device="cuda")
    maxq = obc.obc_minmax_grid(Wd, 4, True, scale, zero)
    osc, oze, omq = oracle.minmax_grid(W, 4, True)
    assert maxq == omq == 14 and np.array_equal(zero.cpu().numpy(), oze)
    assert np.allclose(scale.cpu().numpy(), osc, rtol=2e-7)
    Wq = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    codes = torch.zeros(R, d, dtype=torch.int32, device="cuda")
    ql = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    qo = torch.zeros(R, d, dtype=torch.int32, device="cuda")
    obc.obc_quantize(Wd, Hinv, scale, zero, 4, True, Wq, codes, rs, loss=ql, qorder=qo)
    torch.cuda.synchronize()
    assert int(rs.abs().sum()) == 0
    sc64 = scale.cpu().numpy().astype(np.float64)
    check_rows(Hinv_h, W, qo.cpu().numpy(), ql.cpu().numpy(), gpu_w=Wq.cpu().numpy(), mode="quant", scale=sc64,
               zero=zero.cpu().numpy().astype(np.float64), maxq=maxq, gpu_codes=codes.cpu().numpy())
    c = codes.cpu().numpy()
    assert c.min() >= 0 and c.max() <= maxq
    assert np.allclose(Wq.cpu().numpy(), (sc64[:, None] * (c - 7.0)).astype(np.float32), rtol=1e-6, atol=0)


@pytest.mark.parametrize("d,rows,kind", [(4, 3, "correlated"), (5, 4, "correlated"), (7, 2, "relu"), (33, 5, "correlated"),
                                         (230, 3, "relu"), (300, 5, "correlated"), (301, 2, "relu")])
def test_prune_trace_small_and_ragged(obc, d, rows, kind):
    """sizes below, at and above the on-chip threshold, d not a multiple of 4, padded leading dimensions"""
    W, X = obc_synth.make_small(rows, d, 3 * d + 64, 300 + d, kind)
    ld = (d + 3) // 4 * 4 + 4
    H = oracle.hessian(X).astype(np.float32)
    Hinv, info = obc.obc_hessian_inverse(padded(H, ld), DAMP)
    Wd = padded(W, ld)
    order, loss, status, trace = run_trace(obc, Wd, Hinv, want_trace=True)
    assert int(status.abs().sum()) == 0
    o = order.cpu().numpy()
    assert all(sorted(o[r].tolist()) == list(range(d)) for r in range(rows))
    check_rows(Hinv.cpu().numpy(), W, o, loss.cpu().numpy(), gpu_trace=trace.cpu().numpy())
    # determinism: a second run is bit-identical
    order2, loss2, _, trace2 = run_trace(obc, Wd, Hinv, want_trace=True)
    assert torch.equal(order, order2) and torch.equal(loss, loss2) and torch.equal(trace, trace2)


def test_prune_trace_partial_steps_and_row_range(obc):
    d, rows = 260, 6
    W, X = obc_synth.make_small(rows, d, 900, 77)
    H = oracle.hessian(X).astype(np.float32)
    Hinv, _ = obc.obc_hessian_inverse(dev(H), DAMP)
    Wd = dev(W)
    order, loss, status, _ = run_trace(obc, Wd, Hinv, steps=100, row_begin=2, row_count=3)
    o, l, s = order.cpu().numpy(), loss.cpu().numpy(), status.cpu().numpy()
    assert np.all(o[[0, 1, 5]] == -7) and np.all(l[[0, 1, 5]] == -7.0) and np.all(s[[0, 1, 5]] == -7)
    assert np.all(o[2:5, 100:] == -7) and np.all(s[2:5] == 0)
    check_rows(Hinv.cpu().numpy(), W[2:5], o[2:5], l[2:5], steps=100)


@pytest.mark.parametrize("name,rows,n", [("C2", 6, 4096), ("C4", 4, 4096)])
def test_prune_trace_config_shapes(obc, name, rows, n):
    W, X, spec = obc_synth.make_layer(name, n_override=n)
    W = W[:rows]
    H, Hinv = gpu_hinv(obc, X)
    order, loss, status, _ = run_trace(obc, dev(W), Hinv)
    assert int(status.abs().sum()) == 0
    st = check_rows(Hinv.cpu().numpy(), W, order.cpu().numpy(), loss.cpu().numpy())
    print(name, {k: v for k, v in st.items() if k != "oracle"})


@pytest.mark.parametrize("bits,symmetric,flags", [(4, False, 0), (3, True, 0), (2, False, 1), (8, True, 0)])
def test_quantize_against_oracle(obc, bits, symmetric, flags):
    d, rows = 280, 5
    W, X = obc_synth.make_small(rows, d, 1000, 500 + bits, "relu")
    H = oracle.hessian(X).astype(np.float32)
    Hinv, _ = obc.obc_hessian_inverse(dev(H), DAMP)
    Wd = dev(W)
    scale = torch.zeros(rows, dtype=torch.float32, device="cuda")
    zero = torch.zeros(rows, dtype=torch.float32, device="cuda")
    maxq = obc.obc_minmax_grid(Wd, bits, symmetric, scale, zero)
    if flags:   # shrink the grid so that some weights start outside it and the outlier rule has work to do
        scale *= 0.6
    Wq = torch.zeros(rows, d, dtype=torch.float32, device="cuda")
    codes = torch.zeros(rows, d, dtype=torch.int32, device="cuda")
    ql = torch.zeros(rows, d, dtype=torch.float32, device="cuda")
    qo = torch.zeros(rows, d, dtype=torch.int32, device="cuda")
    rs = torch.zeros(rows, dtype=torch.int32, device="cuda")
    obc.obc_quantize(Wd, Hinv, scale, zero, bits, symmetric, Wq, codes, rs, flags=flags, loss=ql, qorder=qo)
    torch.cuda.synchronize()
    assert int(rs.abs().sum()) == 0
    st = check_rows(Hinv.cpu().numpy(), W, qo.cpu().numpy(), ql.cpu().numpy(), gpu_w=Wq.cpu().numpy(), mode="quant",
                    scale=scale.cpu().numpy().astype(np.float64), zero=zero.cpu().numpy().astype(np.float64), maxq=maxq,
                    flags=flags, gpu_codes=codes.cpu().numpy())
    assert st["codes_differ"] == 0


def test_minmax_grid_against_oracle(obc):
    rng = np.random.default_rng(5)
    W = rng.normal(size=(9, 50)).astype(np.float32)
    W[3] = 0.0
    W[4] = np.abs(W[4])
    W[5] = -np.abs(W[5])
    mask = (rng.uniform(size=W.shape) < 0.6).astype(np.uint8)
    for bits, sym in [(4, False), (4, True), (8, True), (2, False)]:
        for mk in (None, mask):
            scale = torch.zeros(9, dtype=torch.float32, device="cuda")
            zero = torch.zeros(9, dtype=torch.float32, device="cuda")
            maxq = obc.obc_minmax_grid(padded(W, 52), bits, sym, scale, zero, mask=None if mk is None else dev(mk))
            osc, oze, omq = oracle.minmax_grid(W, bits, sym, mk)
            assert maxq == omq
            assert np.allclose(scale.cpu().numpy(), osc, rtol=3e-7)
            near = np.abs(np.abs((-np.minimum((W * (1 if mk is None else mk)).min(axis=1), 0) / osc) % 1.0 - 0.5)) < 1e-4
            assert np.array_equal(zero.cpu().numpy()[~near], oze[~near])


def test_compound_prune_then_quantize(obc):
    """benchmark configuration C4 in small: global 50% mask from the trace, then 8-bit OBQ on the survivors."""
    W, X, spec = obc_synth.make_layer("C4", n_override=4096)
    rows = 5
    W = W[:rows]
    R, d = W.shape
    H, Hinv = gpu_hinv(obc, X)
    Wd = dev(W)
    order, loss, status, _ = run_trace(obc, Wd, Hinv)
    k = obc_synth.pruned_count(R, d, 0.5)
    counts = torch.zeros(R, dtype=torch.int32, device="cuda")
    mask = torch.zeros(R, d, dtype=torch.uint8, device="cuda")
    obc.obc_select_global_mask(loss, order, k, counts, mask)
    scale = torch.zeros(R, dtype=torch.float32, device="cuda")
    zero = torch.zeros(R, dtype=torch.float32, device="cuda")
    Wq = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    codes = torch.zeros(R, d, dtype=torch.int32, device="cuda")
    ql = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    qo = torch.full((R, d), -1, dtype=torch.int32, device="cuda")
    rs = torch.zeros(R, dtype=torch.int32, device="cuda")
    obc.obc_quantize(Wd, Hinv, scale, zero, 8, True, Wq, codes, rs, prune_order=order, prune_counts=counts, loss=ql, qorder=qo)
    torch.cuda.synchronize()
    assert int(rs.abs().sum()) == 0
    Hh = Hinv.cpu().numpy().astype(np.float64)
    o, c = order.cpu().numpy(), counts.cpu().numpy()
    m = mask.cpu().numpy()
    gq, gc, gsc, gze = Wq.cpu().numpy(), codes.cpu().numpy(), scale.cpu().numpy(), zero.cpu().numpy()
    assert np.all(gq[m == 0] == 0.0) and np.all(gc[m == 0] == -1) and np.all(gc[m == 1] >= 0)
    for r in range(R):
        pruned = o[r, :c[r]]
        own = oracle.compound_row(Hh, W[r], pruned, 8, True)                # oracle's own grid from its survivors
        assert np.isclose(gsc[r], own["scale"], rtol=1e-4) and gze[r] == own["zero"]
        ref = oracle.compound_row(Hh, W[r], pruned, 8, True, grid=(float(gsc[r]), float(gze[r]), 254))
        nF = d - c[r]
        # same protocol as check_rows, on the directly formed sub-problem
        F, wF, HiF = oracle.group_obs_state(Hh, W[r], pruned)
        pos = {int(j): i for i, j in enumerate(F)}
        forced = np.array([pos[int(j)] for j in qo.cpu().numpy()[r, :nF]], dtype=np.int32)
        sub_codes = gc[r, F][None, :]
        check_rows(HiF, wF[None, :], forced[None, :], ql.cpu().numpy()[r:r + 1, :nF], gpu_w=gq[r, F][None, :], mode="quant",
                   scale=np.array([float(gsc[r])]), zero=np.array([float(gze[r])]), maxq=254, gpu_codes=sub_codes)
        assert (ref["codes"][F] != gc[r, F]).mean() < 0.02


def test_select_global_mask_bit_exact(obc):
    rng = np.random.default_rng(9)
    for R, d in [(7, 9), (64, 576), (300, 257)]:
        L = rng.exponential(size=(R, d)).astype(np.float32)
        L[rng.uniform(size=L.shape) < 0.2] = np.float32(0.5)        # many exact ties
        L[:, 0] = 0.0
        P = np.stack([rng.permutation(d) for _ in range(R)]).astype(np.int32)
        Ld, Pd = dev(L), dev(P)
        for k in (0, 1, R * d // 3, R * d // 2, R * d - 1, R * d):
            counts = torch.full((R,), -1, dtype=torch.int32, device="cuda")
            mask = torch.full((R, d), 9, dtype=torch.uint8, device="cuda")
            obc.obc_select_global_mask(Ld, Pd, k, counts, mask)
            oc, om = oracle.global_mask(L, P, k)
            assert np.array_equal(counts.cpu().numpy(), oc), (R, d, k)
            assert np.array_equal(mask.cpu().numpy(), om)


def test_nonfinite_rows_are_reported_not_trapped(obc):
    d, rows = 40, 3
    W, X = obc_synth.make_small(rows, d, 200, 31)
    H = oracle.hessian(X).astype(np.float32)
    Hinv, _ = obc.obc_hessian_inverse(dev(H), DAMP)
    W[1, 7] = np.nan
    order, loss, status, _ = run_trace(obc, dev(W), Hinv)
    s = status.cpu().numpy()
    assert s[0] == 0 and s[2] == 0 and s[1] > 0
    o = order.cpu().numpy()
    assert np.all(o[1, s[1] - 1:] == -1) and np.all(np.isinf(loss.cpu().numpy()[1, s[1] - 1:]))
    check_rows(Hinv.cpu().numpy(), W[[0, 2]], o[[0, 2]], loss.cpu().numpy()[[0, 2]])


@pytest.mark.parametrize("threads,max_pending", [(128, 1), (128, 3), (256, 7), (512, 2), (512, 64), (0, 0)])
@pytest.mark.parametrize("d,rows", [(9, 3), (301, 4), (640, 3)])
def test_blocked_engine_block_sizes(threads, max_pending, d, rows):
    """deferred-update engine: every thread count, block lengths from 1 (a flush per step) to the maximum, sizes
    around the on-chip threshold; prune trace with the full weight trace, and OBQ"""
    import paper_2208_11580_b200 as m
    m.load_library()
    m = WithEngineOpts(m, m.ENGINE_BLOCKED, threads, max_pending)
    W, X = obc_synth.make_small(rows, d, 3 * d + 64, 900 + d, "relu")
    H = oracle.hessian(X).astype(np.float32)
    ld = (d + 3) // 4 * 4
    Hinv, info = m.obc_hessian_inverse(padded(H, ld), DAMP)
    Wd = padded(W, ld)
    order, loss, status, trace = run_trace(m, Wd, Hinv, want_trace=True)
    assert int(status.abs().sum()) == 0
    check_rows(Hinv.cpu().numpy(), W, order.cpu().numpy(), loss.cpu().numpy(), gpu_trace=trace.cpu().numpy())
    scale = torch.zeros(rows, dtype=torch.float32, device="cuda")
    zero = torch.zeros(rows, dtype=torch.float32, device="cuda")
    maxq = m.obc_minmax_grid(Wd, 4, False, scale, zero)
    Wq = torch.zeros(rows, d, dtype=torch.float32, device="cuda")
    codes = torch.zeros(rows, d, dtype=torch.int32, device="cuda")
    ql = torch.zeros(rows, d, dtype=torch.float32, device="cuda")
    qo = torch.zeros(rows, d, dtype=torch.int32, device="cuda")
    rs = torch.zeros(rows, dtype=torch.int32, device="cuda")
    m.obc_quantize(Wd, Hinv, scale, zero, 4, False, Wq, codes, rs, loss=ql, qorder=qo)
    torch.cuda.synchronize()
    assert int(rs.abs().sum()) == 0
    check_rows(Hinv.cpu().numpy(), W, qo.cpu().numpy(), ql.cpu().numpy(), gpu_w=Wq.cpu().numpy(), mode="quant",
               scale=scale.cpu().numpy().astype(np.float64), zero=zero.cpu().numpy().astype(np.float64), maxq=maxq,
               gpu_codes=codes.cpu().numpy())


@pytest.mark.parametrize("threads,max_pending,d,rows", [(0, 0, 300, 9), (128, 0, 520, 9), (256, 7, 520, 9), (256, 64, 1100, 6),
                                                        (512, 0, 1100, 6), (512, 5, 300, 9), (0, 0, 301, 9), (256, 0, 519, 7)])
def test_forced_replay_against_trace_and_oracle(threads, max_pending, d, rows):
    """forced-order replay (obc_prune_apply without a trace) on rows long enough to run off chip, where the blocked
    engine takes the forced eliminations four at a time: per-row counts from 0 to d_col, against the GPU's own trace,
    the oracle's trace, and -- for an order that names a column twice -- the reported status"""
    import paper_2208_11580_b200 as m
    m.load_library()
    m = WithEngineOpts(m, m.ENGINE_BLOCKED, threads, max_pending)
    W, X = obc_synth.make_small(rows, d, 3 * d + 64, 4100 + d, "relu")
    H = oracle.hessian(X).astype(np.float32)
    ld = (d + 3) // 4 * 4
    Hinv, info = m.obc_hessian_inverse(padded(H, ld), DAMP)
    Wd = padded(W, ld)
    order, loss, status, trace = run_trace(m, Wd, Hinv, want_trace=True)
    assert int(status.abs().sum()) == 0
    st = check_rows(Hinv.cpu().numpy(), W, order.cpu().numpy(), loss.cpu().numpy(), gpu_trace=trace.cpu().numpy())
    cnt = np.array([0, 1, 3, 4, 5, d // 2 + 1, d - 1, d, 37][:rows], dtype=np.int32)
    counts = torch.from_numpy(cnt).cuda()
    rs = torch.zeros(rows, dtype=torch.int32, device="cuda")
    got = torch.zeros(rows, d, dtype=torch.float32, device="cuda")
    m.obc_prune_apply(Wd, Hinv, order, counts, got, rs)
    ref = torch.zeros(rows, d, dtype=torch.float32, device="cuda")
    m.obc_prune_apply(Wd, Hinv, order, counts, ref, rs, w_trace=trace, trace_steps=d)
    torch.cuda.synchronize()
    assert int(rs.abs().sum()) == 0
    g, r = got.cpu().numpy(), ref.cpu().numpy()
    wscale = np.abs(W).max(axis=1, keepdims=True)
    assert (np.abs(g - r) / wscale).max() <= REL_TOL
    want = oracle.weights_from_trace(st["oracle"]["w_trace"], cnt)
    assert (np.abs(g - want) / wscale).max() <= REL_TOL
    o = order.cpu().numpy()
    for i in range(rows):
        assert np.all(g[i, o[i, :cnt[i]]] == 0.0)
    # an order that is not a permutation: row 5 names its first column again at step 6
    bad = order.clone()
    bad[5, 6] = bad[5, 0]
    rs2 = torch.zeros(rows, dtype=torch.int32, device="cuda")
    out2 = torch.zeros(rows, d, dtype=torch.float32, device="cuda")
    m.obc_prune_apply(Wd, Hinv, bad, counts, out2, rs2)
    torch.cuda.synchronize()
    r2 = rs2.cpu().numpy()
    assert r2[5] == 1 + 6 and np.all(np.delete(r2, 5) == 0)
    assert np.array_equal(np.delete(out2.cpu().numpy(), 5, axis=0), np.delete(g, 5, axis=0))



def test_sharded_layer_driver_single_rank(obc):
    """the row-sharded layer driver with one rank (no process group): same masks and weights as the oracle"""
    from paper_2208_11580_b200.sharding import prune_layer_sharded
    W, X, spec = obc_synth.make_layer("C1")
    R, d = W.shape
    out = prune_layer_sharded(dev(W), dev(X), (0.5, 0.75), DAMP, prec=obc.PREC_FP32)
    torch.cuda.synchronize()
    assert (out["row_begin"], out["row_count"]) == (0, R) and int(out["info"].item()) == 0
    H = torch.empty(d, d, dtype=torch.float32, device="cuda")
    obc.obc_hessian(dev(X), H, prec=obc.PREC_FP32)
    Hinv, _ = obc.obc_hessian_inverse(H, DAMP)
    order, loss, status, trace = run_trace(obc, dev(W), Hinv, want_trace=True)
    res = oracle.run_rows(Hinv.cpu().numpy().astype(np.float64), W, forced=order.cpu().numpy(), want_trace=True)
    for i, sp in enumerate((0.5, 0.75)):
        k = obc_synth.pruned_count(R, d, sp)
        oc, om = oracle.global_mask(loss.cpu().numpy(), order.cpu().numpy(), k)
        assert np.array_equal(out["counts"][i].cpu().numpy(), oc) and np.array_equal(out["masks"][i].cpu().numpy(), om)
        want = oracle.weights_from_trace(res["w_trace"], oc)
        got = out["weights"][i].cpu().numpy()
        assert (np.abs(got - want) / np.abs(W).max(axis=1, keepdims=True)).max() <= REL_TOL


@pytest.mark.parametrize("threads,max_pending", [(0, 0), (128, 3), (512, 5)])
@pytest.mark.parametrize("nm", [(2, 4), (4, 8), (1, 4), (1, 2)])
@pytest.mark.parametrize("d,rows", [(16, 3), (304, 4), (640, 3)])
def test_prune_nm_against_oracle(nm, d, rows, threads, max_pending):
    """N:M pruning (Section 3, "N:M Sparsity"): picks, losses and compensated weights against the oracle, the mask
    keeps exactly N weights in every block of M"""
    import paper_2208_11580_b200 as m
    m.load_library()
    n_keep, mb = nm
    m = WithEngineOpts(m, m.ENGINE_BLOCKED, threads, max_pending)
    W, X = obc_synth.make_small(rows, d, 3 * d + 64, 1200 + d + mb, "relu")
    H = oracle.hessian(X).astype(np.float32)
    Hinv, info = m.obc_hessian_inverse(dev(H), DAMP)
    Wd = dev(W)
    steps = d // mb * (mb - n_keep)
    order = torch.full((rows, d), -7, dtype=torch.int32, device="cuda")
    loss = torch.full((rows, d), -7.0, dtype=torch.float32, device="cuda")
    Wout = torch.full((rows, d), 9.0, dtype=torch.float32, device="cuda")
    mask = torch.full((rows, d), 9, dtype=torch.uint8, device="cuda")
    rs = torch.full((rows,), -7, dtype=torch.int32, device="cuda")
    m.obc_prune_nm(Wd, Hinv, n_keep, mb, Wout, rs, order=order, loss=loss, mask=mask)
    torch.cuda.synchronize()
    assert int(rs.abs().sum()) == 0
    o, mk, wo = order.cpu().numpy(), mask.cpu().numpy(), Wout.cpu().numpy()
    assert np.all(o[:, steps:] == -7) and np.all(mk.reshape(rows, d // mb, mb).sum(axis=2) == n_keep)
    assert np.all(wo[mk == 0] == 0.0)
    for r in range(rows):
        assert set(np.nonzero(mk[r] == 0)[0].tolist()) == set(o[r, :steps].tolist())
    check_rows(Hinv.cpu().numpy(), W, o, loss.cpu().numpy(), gpu_w=wo, steps=steps, nm=nm)


@pytest.mark.parametrize("c", [4, 8])
@pytest.mark.parametrize("threads,max_pending", [(0, 0), (128, 4), (256, 9), (512, 64)])
@pytest.mark.parametrize("d,rows,kind", [(8, 3, "correlated"), (64, 4, "relu"), (300, 4, "correlated"), (640, 3, "relu")])
def test_prune_blocks_against_oracle(d, rows, kind, threads, max_pending, c):
    """block pruning in blocks of c = 4 or 8 (Section 3, "Block-Sparsity", Eq. 5): block picks (margin-gated), block
    losses, weights after a given number of blocks, and whole-block global masks"""
    import paper_2208_11580_b200 as m
    m.load_library()
    m = WithEngineOpts(m, m.ENGINE_BLOCKED, threads, max_pending)
    d += -d % c
    W, X = obc_synth.make_small(rows, d, 3 * d + 64, 1500 + d + c, kind)
    H = oracle.hessian(X).astype(np.float32)
    Hinv, info = m.obc_hessian_inverse(dev(H), DAMP)
    Wd = dev(W)
    order = torch.full((rows, d), -7, dtype=torch.int32, device="cuda")
    loss = torch.full((rows, d), -7.0, dtype=torch.float32, device="cuda")
    rs = torch.full((rows,), -7, dtype=torch.int32, device="cuda")
    trace = torch.zeros(rows, d + 1, d, dtype=torch.float32, device="cuda")
    m.obc_prune_blocks(Wd, Hinv, order, loss, rs, block=c, w_trace=trace)
    torch.cuda.synchronize()
    assert int(rs.abs().sum()) == 0
    o, l = order.cpu().numpy(), loss.cpu().numpy().astype(np.float64)
    blocks = o[:, ::c] // c
    assert np.array_equal(o, (blocks[:, :, None] * c + np.arange(c)).reshape(rows, d))        # members ascending
    assert all(sorted(blocks[r].tolist()) == list(range(d // c)) for r in range(rows))
    assert np.all(l.reshape(rows, d // c, c)[:, :, 1:] == 0.0)
    Hh = Hinv.cpu().numpy().astype(np.float64)
    res = oracle.run_rows_blocks(Hh, W, c, forced_blocks=blocks)
    assert np.all(res["status"] == 0)
    differ = res["best_block"] != blocks
    assert not (differ & (res["forced_gap"] > 1e-6)).any()
    L = res["loss"][:, ::c]
    floor = 1e-7 * np.abs(L).max(axis=1, keepdims=True)
    assert (np.abs(l[:, ::c] - L) / (np.abs(L) + floor)).max() <= REL_TOL
    assert np.all(trace[:, -1].cpu().numpy() == 0.0)
    # weights after nb blocks (trace row c*nb) against the oracle stopped there
    wscale = np.abs(W).max(axis=1, keepdims=True)
    for nb in sorted({1, max(1, d // (2 * c)), max(1, d // c - 1)}):
        part = oracle.run_rows_blocks(Hh, W, c, steps=nb, forced_blocks=blocks[:, :nb])
        assert (np.abs(trace[:, c * nb].cpu().numpy() - part["w"]) / wscale).max() <= REL_TOL
    # global step on whole blocks: k a multiple of c
    k = (rows * d // (2 * c)) * c
    counts = torch.zeros(rows, dtype=torch.int32, device="cuda")
    mask = torch.zeros(rows, d, dtype=torch.uint8, device="cuda")
    m.obc_select_global_mask(loss, order, k, counts, mask)
    cn, mk = counts.cpu().numpy(), mask.cpu().numpy()
    assert np.all(cn % c == 0) and int((mk == 0).sum()) == k
    per_block = mk.reshape(rows, d // c, c).sum(axis=2)
    assert np.all((per_block == 0) | (per_block == c))
    oc, om = oracle.global_mask(l, o, k)
    assert np.array_equal(cn, oc) and np.array_equal(mk, om)


def test_prune_trace_at_maximum_row_length(obc):
    """d_col = OBC_MAX_DCOL (5120): the first 160 steps of two rows against the oracle (shared memory holds only a
    few pending vectors at this length, the rest overflow to the L2-resident buffer of the blocked engine)"""
    d, rows, steps = 5120, 2, 160
    W, X = obc_synth.make_small(rows, d, d + 512, 5120, "relu")
    H, Hinv = gpu_hinv(obc, X, prec=obc.PREC_BF16X3)
    order, loss, status, _ = run_trace(obc, dev(W), Hinv, steps=steps)
    assert int(status.abs().sum()) == 0
    o = order.cpu().numpy()
    assert np.all(o[:, steps:] == -7) and all(len(set(o[r, :steps].tolist())) == steps for r in range(rows))
    check_rows(Hinv.cpu().numpy(), W, o, loss.cpu().numpy(), steps=steps)
    order2, loss2, _, _ = run_trace(obc, dev(W), Hinv, steps=steps)          # a second run is bit-identical
    assert torch.equal(order, order2) and torch.equal(loss, loss2)


@pytest.mark.parametrize("prec", [0, 1, 2])
@pytest.mark.parametrize("R,d,n", [(5, 12, 100), (64, 576, 4096), (130, 300, 5000)])
def test_dense_refit_against_oracle(obc, R, d, n, prec):
    """dense refit before sequential compression: G = Y X^T (accumulated over two chunks) against FP64, and
    W = 2 G Hinv against the oracle's regularised least-squares solve"""
    W0, X = obc_synth.make_small(R, d, n, 2100 + d, "relu")
    rng = np.random.default_rng(d)
    Y = (W0.astype(np.float64) @ X.astype(np.float64) + 0.05 * rng.normal(size=(R, n))).astype(np.float32)
    ldn = (n + 3) // 4 * 4
    Xd, Yd = padded(X, ldn), padded(Y, ldn)
    G = torch.zeros(R, (d + 3) // 4 * 4, dtype=torch.float32, device="cuda")[:, :d]
    h = (n // 2 + 3) // 4 * 4
    obc.obc_cross_gram(Yd[:, :h], Xd[:, :h], G, accumulate=False, prec=prec)
    obc.obc_cross_gram(Yd[:, h:], Xd[:, h:], G, accumulate=True, prec=prec)
    ref = Y.astype(np.float64) @ X.astype(np.float64).T
    scale = np.sqrt((Y.astype(np.float64) ** 2).sum(axis=1).max() * (X.astype(np.float64) ** 2).sum(axis=1).max())
    tol = {0: 2e-6, 1: 1e-3, 2: 2e-5}[prec]
    assert np.abs(G.cpu().numpy() - ref).max() <= tol * scale
    H, Hinv = gpu_hinv(obc, X, prec=prec)
    Wn = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    obc.obc_refit(G, Hinv, Wn, prec=prec)                  # the product G Hinv in the same precision as the Gram matrices
    torch.cuda.synchronize()
    want = oracle.refit(X, Y, DAMP)
    wtol = {0: 2e-4, 1: 2e-2, 2: 5e-4}[prec]
    assert np.abs(Wn.cpu().numpy() - want).max() <= wtol * np.abs(want).max()
    # the product alone, against FP64 on the same FP32 operands
    Wf = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    obc.obc_refit(G, Hinv, Wf, prec=prec)
    prod = 2.0 * G.cpu().numpy().astype(np.float64) @ Hinv.cpu().numpy().astype(np.float64)
    ptol = {0: 2e-6, 1: 1e-3, 2: 2e-5}[prec]
    pscale = 2.0 * np.sqrt((G.cpu().numpy().astype(np.float64) ** 2).sum(axis=1).max() *
                           (Hinv.cpu().numpy().astype(np.float64) ** 2).sum(axis=1).max())
    assert np.abs(Wf.cpu().numpy() - prod).max() <= ptol * pscale
