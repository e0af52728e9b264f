"""Seeded random configurations of the blocked row engine against the oracle: row lengths on both sides of every
internal threshold, every thread count, block lengths from 1 to the maximum, all modes (prune with trace, OBQ with
and without the outlier rule, forced-order replay, compound, N:M, blocks of 4)."""
import numpy as np
import pytest
import torch

import obc_synth
import oracle
from parity import check_rows, REL_TOL, WithEngineOpts

pytestmark = pytest.mark.gpu
DAMP = obc_synth.DAMP_REL


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _padded(a, ld):
    r, c = a.shape
    buf = torch.zeros(r, ld, dtype=torch.float32, device="cuda")
    buf[:, :c] = torch.from_numpy(a)
    return buf[:, :c]


@pytest.mark.parametrize("case", range(28))
def test_random_configuration(case):
    import paper_2208_11580_b200 as m
    m.load_library()
    rng = np.random.default_rng(9000 + case)
    mode = ["prune", "quant", "replay", "compound", "nm", "blocks", "outliers"][case % 7]
    d = int(rng.choice([7, 12, 33, 96, 161, 200, 257, 300, 412, 520, 640, 700]))
    if mode == "blocks":
        d = (d + 3) // 4 * 4
    if mode == "nm":
        d = (d + 7) // 8 * 8
    rows = int(rng.integers(1, 6))
    threads = int(rng.choice([0, 128, 256, 512]))
    pending = int(rng.choice([0, 1, 2, 3, 5, 8, 13, 31, 64]))
    kind = str(rng.choice(["correlated", "relu"]))
    m = WithEngineOpts(m, m.ENGINE_BLOCKED, threads, pending)
    W, X = obc_synth.make_small(rows, d, 3 * d + 64, 7000 + case, kind)
    ld = (d + 3) // 4 * 4
    H = oracle.hessian(X).astype(np.float32)
    Hinv, info = m.obc_hessian_inverse(_padded(H, ld), DAMP)
    assert int(info.item()) == 0
    Hh = Hinv.cpu().numpy()
    Wd = _padded(W, ld)
    i32 = lambda *s, fill=0: torch.full(s, fill, dtype=torch.int32, device="cuda")
    f32 = lambda *s: torch.zeros(*s, dtype=torch.float32, device="cuda")
    order, loss, rs = i32(rows, d, fill=-7), f32(rows, d), i32(rows)
    if mode in ("prune", "replay", "compound"):
        trace = f32(rows, d + 1, d)
        m.obc_prune_trace(Wd, Hinv, order, loss, rs, w_trace=trace)
        torch.cuda.synchronize()
        assert int(rs.abs().sum()) == 0
        st = check_rows(Hh, W, order.cpu().numpy(), loss.cpu().numpy(), gpu_trace=trace.cpu().numpy())
        counts = torch.from_numpy(rng.integers(0, d + 1, size=rows).astype(np.int32)).cuda()
        if mode == "replay":
            out = f32(rows, d)
            m.obc_prune_apply(Wd, Hinv, order, counts, out, rs)
            torch.cuda.synchronize()
            want = oracle.weights_from_trace(st["oracle"]["w_trace"], counts.cpu().numpy())
            assert (np.abs(out.cpu().numpy() - want) / np.abs(W).max(axis=1, keepdims=True)).max() <= REL_TOL
        if mode == "compound":
            counts = torch.clamp(counts, max=d - 1)
            sc, ze, Wq, codes = f32(rows), f32(rows), f32(rows, d), i32(rows, d)
            ql, qo = f32(rows, d), i32(rows, d, fill=-1)
            m.obc_quantize(Wd, Hinv, sc, ze, 4, False, Wq, codes, rs, prune_order=order, prune_counts=counts, loss=ql, qorder=qo)
            torch.cuda.synchronize()
            assert int(rs.abs().sum()) == 0
            o, c = order.cpu().numpy(), counts.cpu().numpy()
            for r in range(rows):
                F, wF, HiF = oracle.group_obs_state(Hh.astype(np.float64), W[r], o[r, :c[r]])
                pos = {int(j): i for i, j in enumerate(F)}
                forced = np.array([pos[int(j)] for j in qo.cpu().numpy()[r, :len(F)]], dtype=np.int32)
                check_rows(HiF, wF[None, :], forced[None, :], ql.cpu().numpy()[r:r + 1, :len(F)],
                           gpu_w=Wq.cpu().numpy()[r, F][None, :], mode="quant", scale=np.array([float(sc[r])]),
                           zero=np.array([float(ze[r])]), maxq=15, gpu_codes=codes.cpu().numpy()[r, F][None, :])
    elif mode in ("quant", "outliers"):
        bits = int(rng.choice([2, 3, 4, 8]))
        sym = bool(rng.integers(0, 2))
        sc, ze, Wq, codes = f32(rows), f32(rows), f32(rows, d), i32(rows, d)
        maxq = m.obc_minmax_grid(Wd, bits, sym, sc, ze)
        flags = 0
        if mode == "outliers":
            sc *= 0.6
            flags = m.FLAG_OUTLIERS
        m.obc_quantize(Wd, Hinv, sc, ze, bits, sym, Wq, codes, rs, flags=flags, loss=loss, qorder=order)
        torch.cuda.synchronize()
        assert int(rs.abs().sum()) == 0
        check_rows(Hh, W, order.cpu().numpy(), loss.cpu().numpy(), gpu_w=Wq.cpu().numpy(), mode="quant",
                   scale=sc.cpu().numpy().astype(np.float64), zero=ze.cpu().numpy().astype(np.float64), maxq=maxq,
                   flags=flags, gpu_codes=codes.cpu().numpy())
    elif mode == "nm":
        n_keep, mb = [(2, 4), (4, 8), (1, 4), (3, 8)][case % 4]
        steps = d // mb * (mb - n_keep)
        out, mask = f32(rows, d), torch.zeros(rows, d, dtype=torch.uint8, device="cuda")
        m.obc_prune_nm(Wd, Hinv, n_keep, mb, out, rs, order=order, loss=loss, mask=mask)
        torch.cuda.synchronize()
        assert int(rs.abs().sum()) == 0
        assert np.all(mask.cpu().numpy().reshape(rows, d // mb, mb).sum(axis=2) == n_keep)
        check_rows(Hh, W, order.cpu().numpy(), loss.cpu().numpy(), gpu_w=out.cpu().numpy(), steps=steps, nm=(n_keep, mb))
    else:   # blocks of 4
        m.obc_prune_blocks(Wd, Hinv, order, loss, rs)
        torch.cuda.synchronize()
        assert int(rs.abs().sum()) == 0
        o, l = order.cpu().numpy(), loss.cpu().numpy().astype(np.float64)
        blocks = o[:, ::4] // 4
        res = oracle.run_rows_blocks(Hh.astype(np.float64), W, 4, forced_blocks=blocks)
        assert np.all(res["status"] == 0)
        assert not ((res["best_block"] != blocks) & (res["forced_gap"] > 1e-6)).any()
        L = res["loss"][:, ::4]
        assert (np.abs(l[:, ::4] - L) / (np.abs(L) + 1e-7 * np.abs(L).max(axis=1, keepdims=True))).max() <= REL_TOL
