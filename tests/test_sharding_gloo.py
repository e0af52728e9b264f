"""Row sharding across ranks, on CPU: the partition arithmetic, and the one exchange step of the multi-GPU path
(all-gather of the per-row loss traces and orders before Algorithm 2) with two gloo processes.  Each rank produces
the traces of its own rows with the FP64 oracle; after the exchange every rank must hold exactly what a single
process computes for the whole layer, and the global mask taken from it must be the single-process mask."""
import os
import socket
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_row_range_partitions_every_row_once():
    from paper_2208_11580_b200.sharding import row_range
    for R in (0, 1, 7, 64, 768, 3072):
        for world in (1, 2, 3, 8):
            spans = [row_range(R, world, r) for r in range(world)]
            assert spans[0][0] == 0 and sum(c for _, c in spans) == R
            for (b0, c0), (b1, _) in zip(spans, spans[1:]):
                assert b0 + c0 == b1
            sizes = [c for _, c in spans]
            assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    with pytest.raises(ValueError):
        row_range(4, 2, 2)


WORKER = r"""
import os, sys
import numpy as np
import torch
import torch.distributed as dist
sys.path.insert(0, os.environ["OBC_ROOT"])
import obc_synth, oracle
from paper_2208_11580_b200.sharding import row_range, gather_traces

dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{os.environ['OBC_PORT']}",
                        rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
rank, world = dist.get_rank(), dist.get_world_size()
R, d = 7, 24                                   # 7 rows over 2 ranks: ranges of 4 and 3 rows (padding in the collective)
W, X = obc_synth.make_small(R, d, 200, 11)
H = oracle.hessian(X)
Hinv, info = oracle.inverse(H, obc_synth.DAMP_REL)
assert info == 0
b, c = row_range(R, world, rank)
loc = oracle.run_rows(Hinv, W[b:b + c])
L, P = gather_traces(torch.from_numpy(loc["loss"].astype(np.float32)), torch.from_numpy(loc["order"]), R)
full = oracle.run_rows(Hinv, W)
assert L.shape == (R, d) and P.shape == (R, d) and P.dtype == torch.int32
assert np.array_equal(P.numpy(), full["order"])
assert np.array_equal(L.numpy(), full["loss"].astype(np.float32))
k = obc_synth.pruned_count(R, d, 0.5)
c1, m1 = oracle.global_mask(L.numpy(), P.numpy(), k)
c0, m0 = oracle.global_mask(full["loss"].astype(np.float32), full["order"], k)
assert np.array_equal(c1, c0) and np.array_equal(m1, m0) and int((m1 == 0).sum()) == k
# every rank agrees on the counts (the selection runs redundantly on all ranks)
t = torch.from_numpy(c1.astype(np.int64))
lo, hi = t.clone(), t.clone()
dist.all_reduce(lo, op=dist.ReduceOp.MIN); dist.all_reduce(hi, op=dist.ReduceOp.MAX)
assert torch.equal(lo, hi)
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_trace_exchange_two_gloo_ranks(tmp_path):
    import oracle
    oracle.build()                                       # compile once, before two processes race for it
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", OBC_PORT=str(port), OBC_ROOT=ROOT, OMP_NUM_THREADS="2")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = []
    for p in procs:
        try:
            out, _ = p.communicate(timeout=240)
        except subprocess.TimeoutExpired:
            p.kill()
            out, _ = p.communicate()
        outs.append(out)
    for rank, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, f"rank {rank} failed:\n{out}"
        assert f"rank {rank} ok" in out
