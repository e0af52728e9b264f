"""Small stand-alone run of the row elimination engine (or the Hessian kernel) for profiler captures.

  python -m paper_2208_11580_b200.profile_case --d 1152 --rows 148 --mode prune --repeat 2

Builds a seeded synthetic layer (d_col = --d, --rows rows), its Hessian and inverse through the library, then
launches the engine --repeat times and prints CUDA-event times and the algorithmic GB/s (8 m^2 bytes per step).
Sized by the caller so that the private inverse-Hessian copies exceed L2 but stay at a few GB.
"""
import argparse
import json
import os
import sys

import numpy as np
import torch

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import obc_synth  # noqa: E402
import paper_2208_11580_b200 as obc  # noqa: E402


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--d", type=int, default=1152)
    ap.add_argument("--rows", type=int, default=148)
    ap.add_argument("--n", type=int, default=0)
    ap.add_argument("--mode", default="prune", choices=["prune", "quant", "nm24", "hessian"])
    ap.add_argument("--prec", default="bf16x3", choices=["fp32", "tf32", "bf16x3"])
    ap.add_argument("--repeat", type=int, default=2)
    ap.add_argument("--engine", default="auto", choices=["auto", "streaming", "blocked"])
    ap.add_argument("--threads", type=int, default=0, help="blocked engine: threads per row (0 = from d)")
    ap.add_argument("--pending", type=int, default=0, help="blocked engine: limit on deferred updates (0 = max)")
    a = ap.parse_args()
    d, R = a.d, a.rows
    obc.obc_set_engine({"auto": obc.ENGINE_AUTO, "streaming": obc.ENGINE_STREAMING, "blocked": obc.ENGINE_BLOCKED}[a.engine],
                       a.threads, a.pending)
    n = a.n or 2 * d
    W, X = obc_synth.make_small(R, d, n, 4242, "relu")
    Wd, Xd = torch.from_numpy(W).cuda(), torch.from_numpy(X).cuda()
    H = torch.empty(d, d, dtype=torch.float32, device="cuda")
    if a.mode == "hessian":
        prec = {"fp32": obc.PREC_FP32, "tf32": obc.PREC_TF32, "bf16x3": obc.PREC_BF16X3}[a.prec]
        ws = torch.empty(obc.obc_workspace_bytes(obc.OP_HESSIAN, 0, d, n), dtype=torch.uint8, device="cuda")
        times = []
        for _ in range(a.repeat):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            obc.obc_hessian(Xd, H, prec=prec, ws=ws)
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        print(json.dumps({"d": d, "n": n, "mode": "hessian", "prec": a.prec, "ms": [round(t, 3) for t in times],
                          "dense_equiv_TFLOPs": round(2.0 * d * d * n / (min(times) * 1e-3) / 1e12, 1)}))
        return
    obc.obc_hessian(Xd, H)
    Hinv, info = obc.obc_hessian_inverse(H, obc_synth.DAMP_REL)
    order = torch.zeros(R, d, dtype=torch.int32, device="cuda")
    loss = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    status = torch.zeros(R, dtype=torch.int32, device="cuda")
    ws = torch.empty(obc.obc_workspace_bytes(obc.OP_PRUNE_TRACE, R, d), dtype=torch.uint8, device="cuda")
    if a.mode == "nm24":
        Wq = torch.zeros(R, d, dtype=torch.float32, device="cuda")
    if a.mode == "quant":
        scale = torch.zeros(R, dtype=torch.float32, device="cuda")
        zero = torch.zeros(R, dtype=torch.float32, device="cuda")
        obc.obc_minmax_grid(Wd, 4, False, scale, zero)
        Wq = torch.zeros(R, d, dtype=torch.float32, device="cuda")
        codes = torch.zeros(R, d, dtype=torch.int32, device="cuda")
    times = []
    for _ in range(a.repeat):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        if a.mode == "prune":
            obc.obc_prune_trace(Wd, Hinv, order, loss, status, ws=ws)
        elif a.mode == "nm24":
            obc.obc_prune_nm(Wd, Hinv, 2, 4, Wq, status, order=order, loss=loss, ws=ws)
        else:
            obc.obc_quantize(Wd, Hinv, scale, zero, 4, False, Wq, codes, status, ws=ws)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    assert int(info.item()) == 0 and int(status.abs().sum()) == 0
    m = np.arange(1, d + 1, dtype=np.float64)
    nbytes = R * float((8 * m * m).sum())
    print(json.dumps({"d": d, "rows": R, "mode": a.mode, "engine": a.engine, "threads": a.threads, "pending": a.pending, "ms": [round(t, 3) for t in times],
                      "algorithmic_GBps": round(nbytes / (min(times) * 1e-3) / 1e9, 1),
                      "private_copies_MB": round(min(R, 148) * d * d * 4 / 1e6, 1)}))


if __name__ == "__main__":
    main()
