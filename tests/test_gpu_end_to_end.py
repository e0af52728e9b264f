"""End-to-end check per benchmark configuration: the whole CUDA pipeline (BF16x3 tensor-core Hessian -> FP64-carried
inverse stored in FP32 -> row engine) against the oracle run on its OWN FP64 Hessian and inverse, free-running (no
teacher forcing).  The stage-isolated parity tests feed the oracle the GPU's FP32 inverse; this one shows what the
rounding of the Hessian and of the inverse does to a layer's result.  The greedy orders of the two runs may part ways
(the path is chaotic), so the compared quantity is the layer-error metric of the loss trace, (1/2) sum_t L[r, t]:
over the first half of the eliminations for pruning (over all d_col steps the sum telescopes to (1/2) w0^T H w0
whatever the order), over all steps for OBQ.  Reported per configuration; asserted against a loose bound."""
import numpy as np
import pytest
import torch

import obc_synth
import oracle
from parity import record_stats

pytestmark = pytest.mark.gpu
DAMP = obc_synth.DAMP_REL
E2E_TOL = 5e-3          # relative difference of the partial layer error between the two pipelines


def _rows(R, k, seed):
    rng = np.random.default_rng(seed)
    if R <= k + 2:
        return np.arange(R)
    return np.array(sorted({0, R - 1} | set(rng.choice(np.arange(1, R - 1), size=k, replace=False).tolist())))


@pytest.mark.parametrize("name", ["C1", "C2", "C3", "C4", "C5"])
def test_pipeline_against_oracle_on_its_own_hessian(name):
    import paper_2208_11580_b200 as obc
    obc.load_library()
    W, X, spec = obc_synth.make_layer(name)
    R, d = W.shape
    rows = _rows(R, 6 if d > 1024 else 30, 17)
    Xd = torch.from_numpy(X).cuda()
    H = torch.empty(d, d, dtype=torch.float32, device="cuda")
    obc.obc_hessian(Xd, H, prec=obc.PREC_BF16X3)
    del Xd
    Hinv, info = obc.obc_hessian_inverse(H, DAMP)
    assert int(info.item()) == 0
    Wd = torch.from_numpy(np.ascontiguousarray(W[rows])).cuda()
    n = len(rows)
    order = torch.zeros(n, d, dtype=torch.int32, device="cuda")
    loss = torch.zeros(n, d, dtype=torch.float32, device="cuda")
    status = torch.zeros(n, dtype=torch.int32, device="cuda")
    H64 = oracle.hessian(X)
    Hinv64, oinfo = oracle.inverse(H64, DAMP)
    assert oinfo == 0
    quant = spec.task == "quant"
    if quant:
        scale = torch.zeros(n, dtype=torch.float32, device="cuda")
        zero = torch.zeros(n, dtype=torch.float32, device="cuda")
        maxq = obc.obc_minmax_grid(Wd, spec.bits, spec.symmetric, scale, zero)
        Wq = torch.zeros(n, d, dtype=torch.float32, device="cuda")
        codes = torch.zeros(n, d, dtype=torch.int32, device="cuda")
        obc.obc_quantize(Wd, Hinv, scale, zero, spec.bits, spec.symmetric, Wq, codes, status, loss=loss, qorder=order)
        sc, ze, mq = oracle.minmax_grid(W[rows], spec.bits, spec.symmetric)
        assert mq == maxq
        ref = oracle.run_rows(Hinv64, W[rows], mode="quant", scale=sc, zero=ze, maxq=mq)
        T = d
    else:
        obc.obc_prune_trace(Wd, Hinv, order, loss, status)
        ref = oracle.run_rows(Hinv64, W[rows])
        T = d // 2
    torch.cuda.synchronize()
    assert int(status.abs().sum()) == 0 and np.all(ref["status"] == 0)
    g = 0.5 * loss.cpu().numpy().astype(np.float64)[:, :T].sum(axis=1)
    o = 0.5 * ref["loss"][:, :T].sum(axis=1)
    rel = np.abs(g - o) / np.abs(o)
    same = float((order.cpu().numpy()[:, :T] == ref["order"][:, :T]).mean())
    hin = Hinv.cpu().numpy().astype(np.float64)
    stats = {"rows": int(n), "steps_summed": int(T), "layer_error_rel_diff_max": float(rel.max()),
             "layer_error_rel_diff_median": float(np.median(rel)), "picks_equal_fraction": same,
             "hinv_max_rel_diff": float(np.abs(hin - Hinv64).max() / np.abs(Hinv64).max())}
    record_stats(f"{name} end to end (BF16x3 Hessian, free-running oracle on its FP64 Hessian)", stats)
    assert rel.max() <= E2E_TOL
