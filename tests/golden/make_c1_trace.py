"""Writes tests/golden/c1_trace_rows.txt: the FP64 oracle's pruning trace (order, loss) and 4-bit OBQ codes of the first
three rows of the smallest benchmark layer (C1: 32 x 64, seed 0).  It calls only obc_synth and oracle; the stored
values guard the oracle's arithmetic against unintended changes (they are its own output, not an independent pin --
the independent pins are in tests/test_oracle_pins.py).

    python tests/golden/make_c1_trace.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
import obc_synth  # noqa: E402
import oracle  # noqa: E402


def compute():
    W, X, spec = obc_synth.make_layer("C1")
    H = oracle.hessian(X)
    Hinv, info = oracle.inverse(H, obc_synth.DAMP_REL)
    assert info == 0
    rows = W[:3]
    tr = oracle.run_rows(Hinv, rows)
    sc, ze, mq = oracle.minmax_grid(rows, spec.bits, spec.symmetric)
    q = oracle.run_rows(Hinv, rows, mode="quant", scale=sc, zero=ze, maxq=mq)
    return tr["order"], tr["loss"], q["codes"], q["order"]


def main():
    order, loss, codes, qorder = compute()
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "c1_trace_rows.txt")
    with open(path, "w") as f:
        f.write("# Output of tests/golden/make_c1_trace.py (FP64 oracle; layer C1, rows 0-2): Algorithm 1 order and loss,\n")
        f.write("# Algorithm 3 (4-bit symmetric min-max grid) codes and order.  Regenerate with that script only.\n")
        for r in range(3):
            f.write(f"order {r} " + " ".join(str(int(v)) for v in order[r]) + "\n")
            f.write(f"loss {r} " + " ".join(repr(float(v)) for v in loss[r]) + "\n")
            f.write(f"codes {r} " + " ".join(str(int(v)) for v in codes[r]) + "\n")
            f.write(f"qorder {r} " + " ".join(str(int(v)) for v in qorder[r]) + "\n")
    print("wrote", path)


if __name__ == "__main__":
    main()
