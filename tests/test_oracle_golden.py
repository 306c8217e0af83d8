"""Regression guard: the oracle and the input recipe still produce the stored checksums
(written by tests/golden/make_golden.py, which calls only the oracle)."""
import os

import numpy as np

import oracle
from paper_2606_26344_b200 import inputs as I

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "oracle_checksums.txt")


def test_oracle_checksums_unchanged():
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        name, n_rows, s, sa, y00, yll, hsum = line.split()
        w = I.WORKLOADS[name]
        inp = I.make_inputs(w)
        rows = I.sample_rows(w, inp.outlier_rows)
        assert rows.size == int(n_rows)
        Y, H = oracle.gmlp_rows(inp.bits("X"), inp.bits("Wg"), inp.bits("Wu"), inp.bits("Wd"), rows=rows,
                                gamma=inp.bits("gamma") if w.rmsnorm else None, eps=w.eps, rmsnorm=w.rmsnorm,
                                want_h=True)
        assert np.isclose(Y.sum(), float(s), rtol=1e-9, atol=1e-9)
        assert np.isclose(np.abs(Y).sum(), float(sa), rtol=1e-9)
        assert np.isclose(Y[0, 0], float(y00), rtol=1e-9, atol=1e-12)
        assert np.isclose(Y[-1, -1], float(yll), rtol=1e-9, atol=1e-12)
        assert int(H.astype(np.uint64).sum() % (1 << 32)) == int(hsum)
