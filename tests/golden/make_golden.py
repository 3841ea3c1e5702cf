"""Writes tests/golden/oracle_rounds_small.txt: five rounds of the FP64 oracle on one small seeded dense problem
and one small seeded CSC problem (candidate lists, kept lists, changes, objective).

The paper prints no worked numeric example, so these are not the paper's values: they are the oracle's own, frozen,
so that a later edit of the oracle that changes what it computes shows up as a failing test
(tests/test_oracle_golden.py) and has to be justified.  Calls only oracle/ and the seeded input generators.

    python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_1312_5766_b200 import workloads as wl  # noqa: E402

CASES = {
    "dense": dict(kind="dense_iid", n_rows=200, n_cols=600, n_true=12, lam_frac=0.05, n_candidates=48, n_keep=12, rho=0.1),
    "csc": dict(kind="csc_uniform", n_rows=500, n_cols=3000, n_true=20, lam_frac=0.01, nnz_col=12, n_candidates=96,
                n_keep=24, rho=0.1),
}
ROUNDS = 5
OUT = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_rounds_small.txt")


def run_case(cfg):
    """Yields (round, cand, kept, dbeta, objective) for the first ROUNDS rounds from beta = 0."""
    p = wl.make_problem(cfg, seed=7)
    if p.layout == wl.DENSE:
        X = oracle.Matrix.dense(p.values.numpy(), n_rows=p.n_rows)
    else:
        X = oracle.Matrix.csc(p.n_rows, p.n_cols, p.values.numpy(), p.row_idx.numpy(), p.col_ptr.numpy())
    n2, beta, resid, delta = oracle.init(X, p.y.numpy(), 1e4)
    lam, eta, rho = float(np.float32(p.lam)), float(np.float32(p.eta)), float(np.float32(p.rho))
    for t in range(ROUNDS):
        out = oracle.round(X, n2, lam, eta, rho, p.n_candidates, p.n_keep, p.seed, t, beta, resid, delta)
        yield t, out["cand"], out["kept"], out["dbeta"], oracle.objective(resid, beta, lam)


def lines():
    for name, cfg in CASES.items():
        for t, cand, kept, dbeta, f in run_case(cfg):
            yield f"{name} {t} cand " + " ".join(str(int(c)) for c in cand)
            yield f"{name} {t} kept " + " ".join(str(int(k)) for k in kept)
            yield f"{name} {t} dbeta " + " ".join(float(d).hex() for d in dbeta)
            yield f"{name} {t} objective {float(f).hex()}"


if __name__ == "__main__":
    with open(OUT, "w") as fh:
        fh.write("# written by tests/golden/make_golden.py from oracle/ alone (not values of the paper: it prints none)\n")
        for ln in lines():
            fh.write(ln + "\n")
    print(OUT)
