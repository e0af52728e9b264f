"""Rows long enough that the blocked engine keeps part of its deferred updates in global memory (d_col > ~2740): every
mode of the engine at such a length against the oracle on sampled rows -- OBQ with more rows than SMs (rows handed over
between blocks), N:M pruning and block pruning.  (Pruning with a full trace at d_col = 3072 is the C5 case of
test_gpu_fullsize.py.)"""
import numpy as np
import pytest
import torch

import obc_synth
import oracle
from parity import check_rows, REL_TOL, WithEngineOpts

pytestmark = pytest.mark.gpu
DAMP = obc_synth.DAMP_REL
D = 2880                      # a multiple of 4 that is no multiple of 64: the last tiles of every pass are ragged


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


@pytest.fixture(scope="module")
def layer():
    import paper_2208_11580_b200 as m
    m.load_library()
    m = WithEngineOpts(m, m.ENGINE_BLOCKED)
    rows = torch.cuda.get_device_properties(0).multi_processor_count + 23
    W, X = obc_synth.make_small(rows, D, D + 512, 2880, "relu")
    H = torch.empty(D, D, dtype=torch.float32, device="cuda")
    m.obc_hessian(_dev(X), H, prec=m.PREC_BF16X3)
    Hinv, info = m.obc_hessian_inverse(H, DAMP)
    assert int(info.item()) == 0
    plan = m.obc_engine_plan(D, False, rows)
    assert plan["l2_vectors"] >= 8 and plan["l2_vectors"] % 8 == 0 and plan["rows_per_sm"] == 1
    return m, W, _dev(W), Hinv, Hinv.cpu().numpy()


def test_obq_long_rows_with_hand_over(layer):
    m, W, Wd, Hinv, Hh = layer
    rows = W.shape[0]
    f32 = lambda *s: torch.zeros(*s, dtype=torch.float32, device="cuda")
    i32 = lambda *s: torch.zeros(*s, dtype=torch.int32, device="cuda")
    scale, zero = f32(rows), f32(rows)
    maxq = m.obc_minmax_grid(Wd, 4, False, scale, zero)
    Wq, codes, ql, qo, rs = f32(rows, D), i32(rows, D), f32(rows, D), i32(rows, D), i32(rows)
    m.obc_quantize(Wd, Hinv, scale, zero, 4, False, Wq, codes, rs, loss=ql, qorder=qo)
    torch.cuda.synchronize()
    assert int(rs.abs().sum()) == 0
    sample = np.array([0, 1, rows // 3, rows // 2, rows - 2, rows - 1])      # first and last blocks' rows, handed-over ones between
    st = check_rows(Hh, W[sample], qo.cpu().numpy()[sample], ql.cpu().numpy()[sample], gpu_w=Wq.cpu().numpy()[sample], mode="quant",
                    scale=scale.cpu().numpy().astype(np.float64)[sample], zero=zero.cpu().numpy().astype(np.float64)[sample],
                    maxq=maxq, gpu_codes=codes.cpu().numpy()[sample])
    assert st["codes_differ"] == 0
    # every row stays on one block: same codes except where a pick was a sub-margin tie
    whole = WithEngineOpts(m._m, m._m.ENGINE_BLOCKED, 0, 0, m._m.ENGINE_WHOLE_WAVES)
    Wq2, codes2 = f32(rows, D), i32(rows, D)
    whole.obc_quantize(Wd, Hinv, scale, zero, 4, False, Wq2, codes2, rs)
    torch.cuda.synchronize()
    assert int(rs.abs().sum()) == 0
    assert float((codes2 == codes).float().mean()) > 0.999


def test_nm_long_rows(layer):
    m, W, Wd, Hinv, Hh = layer
    rows = 4
    order = torch.full((rows, D), -7, dtype=torch.int32, device="cuda")
    loss = torch.full((rows, D), -7.0, dtype=torch.float32, device="cuda")
    Wout = torch.full((rows, D), 9.0, dtype=torch.float32, device="cuda")
    mask = torch.full((rows, D), 9, dtype=torch.uint8, device="cuda")
    rs = torch.full((rows,), -7, dtype=torch.int32, device="cuda")
    m.obc_prune_nm(Wd[:rows], Hinv, 2, 4, Wout, rs, order=order, loss=loss, mask=mask)
    torch.cuda.synchronize()
    assert int(rs.abs().sum()) == 0
    steps = D // 2
    o, mk, wo = order.cpu().numpy(), mask.cpu().numpy(), Wout.cpu().numpy()
    assert np.all(o[:, steps:] == -7) and np.all(mk.reshape(rows, D // 4, 4).sum(axis=2) == 2)
    assert np.all(wo[mk == 0] == 0.0)
    check_rows(Hh, W[:rows], o, loss.cpu().numpy(), gpu_w=wo, steps=steps, nm=(2, 4))


@pytest.mark.parametrize("c", [4, 8])
def test_blocks_long_rows(layer, c):
    m, W, Wd, Hinv, Hh = layer
    rows, nblk = 3, D // (2 * c)              # compared: the first half of the blocks (the passes with vectors in global memory)
    order = torch.full((rows, D), -7, dtype=torch.int32, device="cuda")
    loss = torch.full((rows, D), -7.0, dtype=torch.float32, device="cuda")
    rs = torch.full((rows,), -7, dtype=torch.int32, device="cuda")
    trace = torch.zeros(rows, D + 1, D, dtype=torch.float32, device="cuda")
    m.obc_prune_blocks(Wd[:rows], Hinv, order, loss, rs, block=c, w_trace=trace)
    torch.cuda.synchronize()
    assert int(rs.abs().sum()) == 0
    full = order.cpu().numpy()
    assert all(sorted((full[r, ::c] // c).tolist()) == list(range(D // c)) for r in range(rows))
    assert np.all(trace[:, -1].cpu().numpy() == 0.0)
    o, l = full[:, :c * nblk], loss.cpu().numpy().astype(np.float64)[:, :c * nblk]
    blocks = o[:, ::c] // c
    assert np.array_equal(o, (blocks[:, :, None] * c + np.arange(c)).reshape(rows, c * nblk))
    res = oracle.run_rows_blocks(Hh.astype(np.float64), W[:rows], c, steps=nblk, forced_blocks=blocks)
    assert np.all(res["status"] == 0)
    differ = res["best_block"] != blocks
    assert not (differ & (res["forced_gap"] > 1e-6)).any()
    L = res["loss"][:, ::c]
    floor = 1e-7 * np.abs(L).max(axis=1, keepdims=True)
    assert (np.abs(l[:, ::c] - L) / (np.abs(L) + floor)).max() <= REL_TOL
    wscale = np.abs(W[:rows]).max(axis=1, keepdims=True)
    assert (np.abs(trace[:, c * nblk].cpu().numpy() - res["w"]) / wscale).max() <= REL_TOL
