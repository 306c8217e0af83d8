"""Writes tests/golden/oracle_checksums.txt from the CPU oracle alone.

Run from the repository root:  python tests/golden/make_golden.py
It calls only ``oracle/`` and the seeded input generators; nothing here touches the CUDA
path.  The stored sums guard the oracle and the input recipe against silent change; they
are regression values, not values printed by the paper (the paper prints no worked
numeric example of the Gated MLP).
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2606_26344_b200 import inputs as I  # noqa: E402

CASES = [
    ("tiny", None),
    ("ragged-M7-plain", None),
    ("ragged-M7-norm", None),
]


def main():
    lines = ["# name  rows  sum(y_ref)  sum(|y_ref|)  y_ref[0,0]  y_ref[-1,-1]  sum(H bits) mod 2^32"]
    for name, _ in CASES:
        w = I.WORKLOADS[name]
        inp = I.make_inputs(w)
        rows = I.sample_rows(w, inp.outlier_rows)
        Y, H = oracle.gmlp_rows(inp.bits("X"), inp.bits("Wg"), inp.bits("Wu"), inp.bits("Wd"), rows=rows,
                                gamma=inp.bits("gamma") if w.rmsnorm else None, eps=w.eps, rmsnorm=w.rmsnorm,
                                want_h=True)
        lines.append(f"{name} {rows.size} {Y.sum():.12e} {np.abs(Y).sum():.12e} {Y[0, 0]:.12e} {Y[-1, -1]:.12e} "
                     f"{int(H.astype(np.uint64).sum() % (1 << 32))}")
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_checksums.txt")
    with open(out, "w") as f:
        f.write("\n".join(lines) + "\n")
    print(open(out).read())


if __name__ == "__main__":
    main()
