"""The bounded device-side waits of the tensor-core Hessian kernels, made to run out on purpose (nothing hangs, nothing
faults): with wait_limit < 0 every wait of the copy / multiply pipeline expires at once, so no product is ever issued;
the kernel must still wait for its own copies in flight, release its tensor memory and return, the call reports
OBC_ERR_TIMEOUT through its info word and fills the result with NaN, and the next ordinary call on the same context
works."""
import numpy as np
import pytest
import torch

import obc_synth
import oracle

pytestmark = pytest.mark.gpu
OBC_ERR_TIMEOUT = 6


@pytest.mark.parametrize("prec", [1, 2])                       # TF32, BF16x3
@pytest.mark.parametrize("d,n", [(64, 256), (200, 1024)])     # fewer / more k-blocks than pipeline stages
def test_hessian_wait_that_runs_out_is_reported(prec, d, n):
    import paper_2208_11580_b200 as obc
    obc.load_library()
    _, X = obc_synth.make_small(1, d, n, 31 + d)
    Xd = torch.from_numpy(X).cuda()
    H = torch.zeros(d, d, dtype=torch.float32, device="cuda")
    info = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    obc.obc_hessian(Xd, H, prec=prec, info=info, wait_limit=-1)         # returns OBC_OK: the failure is data-dependent
    torch.cuda.synchronize()
    assert int(info.item()) == OBC_ERR_TIMEOUT
    assert bool(torch.isnan(H).all())
    assert obc.obc_status_string(OBC_ERR_TIMEOUT) == "device-side wait timed out"
    # the context is intact: the same call with the ordinary limit gives the Hessian, info = 0
    obc.obc_hessian(Xd, H, prec=prec, info=info)
    torch.cuda.synchronize()
    ref = oracle.hessian(X)
    assert int(info.item()) == 0
    assert np.abs(H.cpu().numpy() - ref).max() <= 3e-3 * np.abs(ref).max()
    # a short but sufficient limit also passes (the waits poll: a few thousand polls cover a tile load)
    obc.obc_hessian(Xd, H, prec=prec, info=info, wait_limit=2_000_000)
    torch.cuda.synchronize()
    assert int(info.item()) == 0 and not bool(torch.isnan(H).any())


def test_cross_gram_wait_that_runs_out_is_reported():
    import paper_2208_11580_b200 as obc
    obc.load_library()
    W, X = obc_synth.make_small(40, 96, 512, 77)
    Y = (W @ X).astype(np.float32)
    Yd, Xd = torch.from_numpy(Y).cuda(), torch.from_numpy(X).cuda()
    G = torch.zeros(40, 96, dtype=torch.float32, device="cuda")
    info = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    obc.obc_cross_gram(Yd, Xd, G, prec=obc.PREC_BF16X3, info=info, wait_limit=-1)
    torch.cuda.synchronize()
    assert int(info.item()) == OBC_ERR_TIMEOUT and bool(torch.isnan(G).all())
    obc.obc_cross_gram(Yd, Xd, G, prec=obc.PREC_BF16X3, info=info)
    torch.cuda.synchronize()
    ref = Y.astype(np.float64) @ X.astype(np.float64).T
    assert int(info.item()) == 0 and np.abs(G.cpu().numpy() - ref).max() <= 1e-4 * np.abs(ref).max()
    obc.obc_cross_gram(Yd, Xd, G, prec=obc.PREC_FP32, info=info)        # no waits on this path
    torch.cuda.synchronize()
    assert int(info.item()) == 0
