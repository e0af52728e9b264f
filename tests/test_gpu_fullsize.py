"""Parity at the benchmark configurations' full sizes, in the launch configuration bench.py times (all rows of the
layer in one call), checked on sampled rows the oracle can compute one by one, plus properties that hold at any
size (every order is a permutation, masks match counts, codes lie on the grid)."""
import numpy as np
import pytest
import torch

import obc_synth
import oracle
from parity import check_rows, record_stats, REL_TOL, WithEngineOpts

pytestmark = pytest.mark.gpu
DAMP = obc_synth.DAMP_REL


@pytest.fixture(scope="module", params=["blocked", "streaming"])
def obc(request):
    """the library with one of its two row elimination engines selected; every test runs with both"""
    import paper_2208_11580_b200 as m
    m.load_library()
    return WithEngineOpts(m, m.ENGINE_BLOCKED if request.param == "blocked" else m.ENGINE_STREAMING)


def _sample(R, k, seed):
    """the first row, the last row (it runs in the partial tail wave of the launch) and k further seeded rows"""
    rng = np.random.default_rng(seed)
    inner = rng.choice(np.arange(1, R - 1), size=min(R - 2, k), replace=False).tolist()
    return np.array(sorted({0, R - 1} | set(inner)))


def _front(obc, name, prec):
    W, X, spec = obc_synth.make_layer(name)
    Xd, Wd = torch.from_numpy(X).cuda(), torch.from_numpy(W).cuda()
    d = W.shape[1]
    H = torch.empty(d, d, dtype=torch.float32, device="cuda")
    obc.obc_hessian(Xd, H, prec=prec)
    Hinv, info = obc.obc_hessian_inverse(H, DAMP)
    assert int(info.item()) == 0
    # Hessian: sampled entries against the FP64 definition 2 * <x_i, x_j>
    rng = np.random.default_rng(1)
    ii, jj = rng.integers(0, d, 64), rng.integers(0, d, 64)
    ref = 2.0 * np.einsum("kn,kn->k", X[ii].astype(np.float64), X[jj].astype(np.float64))
    got = H[torch.from_numpy(ii).cuda(), torch.from_numpy(jj).cuda()].cpu().numpy()
    scale = 2.0 * float((X.astype(np.float64) ** 2).sum(axis=1).max())
    assert np.abs(got - ref).max() <= 3e-5 * scale
    # inverse: residual of sampled columns of (H + lambda I) Hinv = I, in FP64
    Hh = H.cpu().numpy().astype(np.float64)
    lam = DAMP * np.trace(Hh) / d
    cols = rng.integers(0, d, 8)
    resid = (Hh + lam * np.eye(d)) @ Hinv[:, torch.from_numpy(cols).cuda()].cpu().numpy().astype(np.float64)
    resid[cols, np.arange(8)] -= 1.0
    assert np.abs(resid).max() < 2e-3
    del Xd
    return W, spec, Wd, Hinv


def test_config2_full_all_rows(obc):
    W, spec, Wd, Hinv = _front(obc, "C2", obc.PREC_BF16X3)
    R, d = W.shape
    order = torch.zeros(R, d, dtype=torch.int32, device="cuda")
    loss = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    status = torch.zeros(R, dtype=torch.int32, device="cuda")
    trace = torch.zeros(R, d + 1, d, dtype=torch.float32, device="cuda")
    obc.obc_prune_trace(Wd, Hinv, order, loss, status, w_trace=trace)
    torch.cuda.synchronize()
    assert int(status.abs().sum()) == 0
    st = check_rows(Hinv.cpu().numpy(), W, order.cpu().numpy(), loss.cpu().numpy(), gpu_w=trace[:, -1].cpu().numpy())
    k = obc_synth.pruned_count(R, d, 0.6)
    counts = torch.zeros(R, dtype=torch.int32, device="cuda")
    mask = torch.zeros(R, d, dtype=torch.uint8, device="cuda")
    obc.obc_select_global_mask(loss, order, k, counts, mask)
    oc, om = oracle.global_mask(loss.cpu().numpy(), order.cpu().numpy(), k)
    assert np.array_equal(counts.cpu().numpy(), oc) and np.array_equal(mask.cpu().numpy(), om) and k == 22118
    What = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    obc.obc_prune_apply(Wd, Hinv, order, counts, What, status, w_trace=trace, trace_steps=d)
    res = oracle.run_rows(Hinv.cpu().numpy().astype(np.float64), W, forced=order.cpu().numpy(), want_trace=True)
    want = oracle.weights_from_trace(res["w_trace"], oc)
    assert (np.abs(What.cpu().numpy() - want) / np.abs(W).max(axis=1, keepdims=True)).max() <= REL_TOL
    record_stats(f"C2 prune trace, all rows, {obc.engine_name}", st)


def test_config3_full_quantize_sampled_rows(obc):
    W, spec, Wd, Hinv = _front(obc, "C3", obc.PREC_BF16X3)
    R, d = W.shape
    scale = torch.zeros(R, dtype=torch.float32, device="cuda")
    zero = torch.zeros(R, dtype=torch.float32, device="cuda")
    maxq = obc.obc_minmax_grid(Wd, 4, False, scale, zero)
    Wq = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    codes = torch.zeros(R, d, dtype=torch.int32, device="cuda")
    ql = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    qo = torch.zeros(R, d, dtype=torch.int32, device="cuda")
    rs = torch.zeros(R, dtype=torch.int32, device="cuda")
    obc.obc_quantize(Wd, Hinv, scale, zero, 4, False, Wq, codes, rs, loss=ql, qorder=qo)
    torch.cuda.synchronize()
    assert int(rs.abs().sum()) == 0 and maxq == 15
    o, c = qo.cpu().numpy(), codes.cpu().numpy()
    assert np.array_equal(np.sort(o, axis=1), np.broadcast_to(np.arange(d), (R, d)))
    assert c.min() >= 0 and c.max() <= 15
    sc, ze = scale.cpu().numpy().astype(np.float64), zero.cpu().numpy().astype(np.float64)
    assert np.allclose(Wq.cpu().numpy(), (sc[:, None] * (c - ze[:, None])).astype(np.float32), rtol=1e-6, atol=0)
    rows = _sample(R, 8, 3)
    st = check_rows(Hinv.cpu().numpy(), W[rows], o[rows], ql.cpu().numpy()[rows], gpu_w=Wq.cpu().numpy()[rows],
                    mode="quant", scale=sc[rows], zero=ze[rows], maxq=15, gpu_codes=c[rows])
    record_stats(f"C3 OBQ 4-bit, {len(rows)} rows, {obc.engine_name}", st)


def test_config4_full_compound_sampled_rows(obc):
    W, spec, Wd, Hinv = _front(obc, "C4", obc.PREC_BF16X3)
    R, d = W.shape
    order = torch.zeros(R, d, dtype=torch.int32, device="cuda")
    loss = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    status = torch.zeros(R, dtype=torch.int32, device="cuda")
    obc.obc_prune_trace(Wd, Hinv, order, loss, status)
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
    assert int(status.abs().sum()) == 0 and int(rs.abs().sum()) == 0
    L, P = loss.cpu().numpy(), order.cpu().numpy()
    oc, om = oracle.global_mask(L, P, k)
    assert k == 1179648 and np.array_equal(counts.cpu().numpy(), oc) and np.array_equal(mask.cpu().numpy(), om)
    rows = _sample(R, 8, 4)
    Hh = Hinv.cpu().numpy()
    st = check_rows(Hh, W[rows], P[rows], L[rows])
    gq, gc, gsc, gze = Wq.cpu().numpy(), codes.cpu().numpy(), scale.cpu().numpy(), zero.cpu().numpy()
    assert np.all(gq[om == 0] == 0.0) and np.all(gc[om == 0] == -1) and gc[om == 1].min() >= 0 and gc.max() <= 254
    H64 = Hh.astype(np.float64)
    for r in rows:
        pruned = P[r, :oc[r]]
        F, wF, HiF = oracle.group_obs_state(H64, W[r], pruned)
        own = oracle.minmax_grid(wF[None, :], 8, True)
        assert np.isclose(gsc[r], own[0][0], rtol=1e-4) and gze[r] == own[1][0]
        pos = {int(j): i for i, j in enumerate(F)}
        nF = len(F)
        forced = np.array([pos[int(j)] for j in qo.cpu().numpy()[r, :nF]], dtype=np.int32)
        sq = check_rows(HiF, wF[None, :], forced[None, :], ql.cpu().numpy()[r:r + 1, :nF], gpu_w=gq[r, F][None, :], mode="quant",
                        scale=np.array([float(gsc[r])]), zero=np.array([float(gze[r])]), maxq=254, gpu_codes=gc[r, F][None, :])
        record_stats(f"C4 OBQ 8-bit on the survivors, row {int(r)}, {obc.engine_name}", sq)
    record_stats(f"C4 prune trace, {len(rows)} rows, {obc.engine_name}", st)


def test_config5_full_trace_sampled_rows(obc):
    W, spec, Wd, Hinv = _front(obc, "C5", obc.PREC_BF16X3)
    R, d = W.shape
    order = torch.zeros(R, d, dtype=torch.int32, device="cuda")
    loss = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    status = torch.zeros(R, dtype=torch.int32, device="cuda")
    trace = torch.empty(R, d + 1, d, dtype=torch.float32, device="cuda")
    obc.obc_prune_trace(Wd, Hinv, order, loss, status, w_trace=trace)
    torch.cuda.synchronize()
    assert int(status.abs().sum()) == 0
    L, P = loss.cpu().numpy(), order.cpu().numpy()
    assert np.array_equal(np.sort(P, axis=1), np.broadcast_to(np.arange(d), (R, d)))
    rows = _sample(R, 8, 5)
    Hh = Hinv.cpu().numpy()
    res = check_rows(Hh, W[rows], P[rows], L[rows], gpu_trace=trace[torch.from_numpy(rows).cuda()].cpu().numpy())
    for s, kk in zip(spec.sparsities, (943718, 1415578, 1887437)):
        k = obc_synth.pruned_count(R, d, s)
        assert k == kk
        counts = torch.zeros(R, dtype=torch.int32, device="cuda")
        mask = torch.zeros(R, d, dtype=torch.uint8, device="cuda")
        obc.obc_select_global_mask(loss, order, k, counts, mask)
        oc, om = oracle.global_mask(L, P, k)
        assert np.array_equal(counts.cpu().numpy(), oc) and np.array_equal(mask.cpu().numpy(), om)
        What = torch.zeros(R, d, dtype=torch.float32, device="cuda")
        obc.obc_prune_apply(Wd, Hinv, order, counts, What, status, w_trace=trace, trace_steps=d)
        want = oracle.weights_from_trace(res["oracle"]["w_trace"], oc[rows])
        got = What.cpu().numpy()
        assert np.all(got[om == 0] == 0.0)
        assert (np.abs(got[rows] - want) / np.abs(W[rows]).max(axis=1, keepdims=True)).max() <= REL_TOL
    record_stats(f"C5 prune trace, {len(rows)} rows, {obc.engine_name}", res)
    # forced-order replay without a trace (the realisation to use when the weight trace does not fit): all rows in
    # one launch at the 60 % counts, sampled rows against the oracle, every row against the trace gather
    k = obc_synth.pruned_count(R, d, 0.6)
    counts = torch.zeros(R, dtype=torch.int32, device="cuda")
    mask = torch.zeros(R, d, dtype=torch.uint8, device="cuda")
    obc.obc_select_global_mask(loss, order, k, counts, mask)
    Wt = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    obc.obc_prune_apply(Wd, Hinv, order, counts, Wt, status, w_trace=trace, trace_steps=d)
    del trace
    torch.cuda.empty_cache()
    Wr = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    rs = torch.zeros(R, dtype=torch.int32, device="cuda")
    obc.obc_prune_apply(Wd, Hinv, order, counts, Wr, rs)
    torch.cuda.synchronize()
    assert int(rs.abs().sum()) == 0
    oc = counts.cpu().numpy()
    want = oracle.weights_from_trace(res["oracle"]["w_trace"], oc[rows])
    wmax = np.abs(W).max(axis=1, keepdims=True)
    got = Wr.cpu().numpy()
    e_or = (np.abs(got[rows] - want) / wmax[rows]).max()
    e_tr = (np.abs(got - Wt.cpu().numpy()) / wmax).max()
    print("C5 replay without trace: vs oracle", e_or, "vs trace gather (all rows)", e_tr)
    assert e_or <= REL_TOL and e_tr <= 2 * REL_TOL
    assert np.all(got[mask.cpu().numpy() == 0] == 0.0)


def test_replay_without_trace_at_d2304(obc):
    """forced-order replay (obc_prune_apply without a trace) at d_col = 2304: rows of C3's layer are pruned (full trace of
    160 rows, more than one wave), per-row counts from 0 to d_col, replayed in one launch, sampled rows against the oracle"""
    W, spec, Wd, Hinv = _front(obc, "C3", obc.PREC_BF16X3)
    R, d = 160, W.shape[1]
    W, Wd = W[:R], Wd[:R]
    order = torch.zeros(R, d, dtype=torch.int32, device="cuda")
    loss = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    status = torch.zeros(R, dtype=torch.int32, device="cuda")
    obc.obc_prune_trace(Wd, Hinv, order, loss, status)
    rng = np.random.default_rng(23)
    cnt = rng.integers(0, d + 1, size=R).astype(np.int32)
    cnt[0], cnt[1], cnt[R - 1] = 0, d, d // 2
    counts = torch.from_numpy(cnt).cuda()
    Wr = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    rs = torch.zeros(R, dtype=torch.int32, device="cuda")
    obc.obc_prune_apply(Wd, Hinv, order, counts, Wr, rs)
    torch.cuda.synchronize()
    assert int(status.abs().sum()) == 0 and int(rs.abs().sum()) == 0
    rows = _sample(R, 8, 6)
    P = order.cpu().numpy()
    res = check_rows(Hinv.cpu().numpy(), W[rows], P[rows], loss.cpu().numpy()[rows])
    record_stats(f"C3-shaped prune trace (d_col 2304), {len(rows)} rows, {obc.engine_name}", res)
    ref = oracle.run_rows(Hinv.cpu().numpy().astype(np.float64), W[rows], forced=P[rows], want_trace=True)
    want = oracle.weights_from_trace(ref["w_trace"], cnt[rows])
    got = Wr.cpu().numpy()
    err = (np.abs(got[rows] - want) / np.abs(W[rows]).max(axis=1, keepdims=True)).max()
    print("replay at d_col 2304 vs oracle:", err)
    assert err <= REL_TOL
    for r in range(R):
        assert np.all(got[r, P[r, :cnt[r]]] == 0.0)
