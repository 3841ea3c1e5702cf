"""Shared test plumbing: turn a generated problem into oracle inputs (numpy)."""
import numpy as np

import oracle
from paper_1312_5766_b200 import workloads as wl


def oracle_matrix(p: wl.LassoProblem) -> oracle.Matrix:
    if p.layout == wl.DENSE:
        return oracle.Matrix.dense(p.values.cpu().numpy(), n_rows=p.n_rows)
    return oracle.Matrix.csc(p.n_rows, p.n_cols, p.values.cpu().numpy(), p.row_idx.cpu().numpy(),
                             p.col_ptr.cpu().numpy())


def dense_array(p: wl.LassoProblem) -> np.ndarray:
    """X as a float64 [N, J] numpy array (small problems only)."""
    if p.layout == wl.DENSE:
        return p.values.cpu().numpy().astype(np.float64).T[: p.n_rows]
    X = np.zeros((p.n_rows, p.n_cols))
    v, r, cp = p.values.cpu().numpy(), p.row_idx.cpu().numpy(), p.col_ptr.cpu().numpy()
    for j in range(p.n_cols):
        X[r[cp[j]:cp[j + 1]], j] = v[cp[j]:cp[j + 1]]
    return X


def run_oracle(p: wl.LassoProblem, rounds: int, c_init: float = 1e4, record=None):
    X = oracle_matrix(p)
    n2, beta, resid, delta = oracle.init(X, p.y.cpu().numpy(), c_init)
    for t in range(rounds):
        out = oracle.round(X, n2, p.lam, p.eta, p.rho, p.n_candidates, p.n_keep, p.seed, t, beta, resid, delta)
        if record is not None:
            record(t, out, beta, resid, delta)
    return X, n2, beta, resid, delta
