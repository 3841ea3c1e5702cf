"""Pins for the oracle's update and for the optimum the scheduled iteration reaches (no GPU).

Three independent anchors for Eq. 1 / Eq. 2: the KKT conditions of the Lasso at
convergence, exhaustive search over all sign patterns on tiny problems, and the
closed-form soft-threshold solution on orthogonal designs.
"""
import itertools

import numpy as np
import pytest
import torch

import oracle
from paper_1312_5766_b200 import workloads as wl
from helpers import dense_array, oracle_matrix, run_oracle


def _small_dense(N, J, n_true, seed, n_cand, n_keep, rho=0.3, lam_frac=0.1):
    cfg = dict(kind="dense_iid", n_rows=N, n_cols=J, n_true=n_true, lam_frac=lam_frac,
               n_candidates=n_cand, n_keep=n_keep, rho=rho, rounds=0)
    return wl.make_problem(cfg, seed=seed)


def _small_csc(N, J, nnz_col, n_true, seed, n_cand, n_keep, rho=0.3, lam_frac=0.1, kind="csc_uniform"):
    cfg = dict(kind=kind, n_rows=N, n_cols=J, n_true=n_true, lam_frac=lam_frac, nnz_col=nnz_col,
               n_candidates=n_cand, n_keep=n_keep, rho=rho, rounds=0)
    return wl.make_problem(cfg, seed=seed)


def _kkt_violation(Xd, y, beta, lam):
    """Largest violation of: |x_j^T r| <= lam where beta_j = 0, x_j^T r = lam sign(beta_j) otherwise."""
    r = y - Xd @ beta
    g = Xd.T @ r
    zero = beta == 0
    v0 = np.maximum(np.abs(g[zero]) - lam, 0.0).max(initial=0.0)
    v1 = np.abs(g[~zero] - lam * np.sign(beta[~zero])).max(initial=0.0)
    return max(v0, v1) / lam


@pytest.mark.parametrize("maker,args", [
    (_small_dense, dict(N=60, J=200, n_true=8, seed=0, n_cand=40, n_keep=8)),
    (_small_dense, dict(N=100, J=50, n_true=5, seed=1, n_cand=10, n_keep=4)),
    (_small_csc, dict(N=300, J=400, nnz_col=12, n_true=10, seed=2, n_cand=60, n_keep=16)),
    (_small_csc, dict(N=500, J=300, nnz_col=8, n_true=10, seed=3, n_cand=40, n_keep=12, kind="csc_zipf")),
])
def test_kkt_at_convergence(maker, args):
    p = maker(**args)
    X, n2, beta, resid, delta = run_oracle(p, rounds=6000)
    Xd, y = dense_array(p), p.y.numpy().astype(np.float64)
    assert _kkt_violation(Xd, y, beta, p.lam) < 1e-6
    # the maintained residual equals y - X beta recomputed from scratch
    assert np.abs(resid - (y - Xd @ beta)).max() < 1e-10 * max(1.0, np.abs(y).max())
    # and the gradient routine agrees with numpy on it
    assert np.allclose(oracle.gradient(X, resid), Xd.T @ resid, rtol=0, atol=1e-12)


def _brute_force_lasso(Xd, y, lam):
    """Exhaustive Lasso: for every support A and sign vector s solve the restricted stationarity
    equations beta_A = (X_A^T X_A)^-1 (X_A^T y - lam s) and keep the sign-consistent, KKT-feasible one."""
    J = Xd.shape[1]
    G, c = Xd.T @ Xd, Xd.T @ y
    best = None
    for mask in range(1 << J):
        A = [j for j in range(J) if mask >> j & 1]
        if not A:
            if np.abs(c).max() <= lam * (1 + 1e-12):
                return np.zeros(J)
            continue
        Ginv = np.linalg.inv(G[np.ix_(A, A)])
        signs = np.array(list(itertools.product((-1.0, 1.0), repeat=len(A)))).T     # [|A|, 2^|A|]
        B = Ginv @ (c[A][:, None] - lam * signs)
        ok = np.all(np.sign(B) == signs, axis=0)
        for col in np.nonzero(ok)[0]:
            beta = np.zeros(J)
            beta[A] = B[:, col]
            g = c - G @ beta
            comp = [j for j in range(J) if not (mask >> j & 1)]
            if not comp or np.abs(g[comp]).max() <= lam * (1 + 1e-9):
                best = beta
    return best


@pytest.mark.parametrize("N,J,seed", [(30, 6, 0), (40, 9, 1), (50, 12, 2)])
def test_against_exhaustive_search(N, J, seed):
    p = _small_dense(N, J, n_true=3, seed=seed, n_cand=min(J, 6), n_keep=3, rho=0.25, lam_frac=0.2)
    Xd, y = dense_array(p), p.y.numpy().astype(np.float64)
    want = _brute_force_lasso(Xd, y, p.lam)
    assert want is not None and 0 < np.count_nonzero(want) < J
    X, n2, beta, resid, delta = run_oracle(p, rounds=4000)
    assert np.abs(beta - want).max() < 1e-8
    f_want = 0.5 * np.sum((y - Xd @ want) ** 2) + p.lam * np.abs(want).sum()
    assert abs(oracle.objective(resid, beta, p.lam) - f_want) < 1e-10 * f_want
    f_scratch, r_scratch = oracle.objective_from_scratch(X, p.y.numpy(), beta, p.lam)
    assert abs(f_scratch - f_want) < 1e-10 * f_want


def test_orthogonal_design_closed_form():
    # X^T X = I: beta_j = S(x_j^T y, lam) after the FIRST update of j, and no pair ever conflicts
    rng = np.random.default_rng(0)
    N, J = 64, 40
    Q, _ = np.linalg.qr(rng.standard_normal((N, N)))
    xc = np.ascontiguousarray(Q[:, :J].T.astype(np.float32))          # [J, N], unit orthogonal columns
    y = (Q[:, :J] @ rng.standard_normal(J) * 2 + 0.1 * rng.standard_normal(N)).astype(np.float32)
    X = oracle.Matrix.dense(xc)
    lam, n_cand, n_keep = 0.7, 10, 10
    n2, beta, resid, delta = oracle.init(X, y, 1e4)
    xty = xc.astype(np.float64) @ y.astype(np.float64)
    want = np.sign(xty) * np.maximum(np.abs(xty) - lam, 0.0)
    touched = np.zeros(J, bool)
    for t in range(J // n_keep):
        out = oracle.round(X, n2, lam, 1e-6, 0.1, n_cand, n_keep, 0, t, beta, resid, delta)
        assert out["kept"].tolist() == out["cand"][:n_keep].tolist()      # first P candidates, in order
        touched[out["kept"]] = True
        assert np.abs(beta[touched] - want[touched]).max() < 1e-6           # FP32 columns: ~1e-7 from exact
        assert np.all(beta[~touched] == 0.0)
    assert touched.all()
    # a further round changes nothing
    out = oracle.round(X, n2, lam, 1e-6, 0.1, n_cand, n_keep, 0, 99, beta, resid, delta)
    assert np.abs(out["dbeta"]).max() < 1e-6


def test_single_coordinate_rounds_are_monotone_and_exact():
    # P' = P = 1 is plain stochastic coordinate descent: F never increases, and each step is the
    # exact minimiser of F along that coordinate.
    p = _small_dense(50, 30, n_true=4, seed=4, n_cand=1, n_keep=1)
    X = oracle_matrix(p)
    Xd, y = dense_array(p), p.y.numpy().astype(np.float64)
    n2, beta, resid, delta = oracle.init(X, p.y.numpy(), 1e4)

    def F(b):
        return 0.5 * np.sum((y - Xd @ b) ** 2) + p.lam * np.abs(b).sum()

    prev = F(beta)
    for t in range(300):
        out = oracle.round(X, n2, p.lam, p.eta, p.rho, 1, 1, 0, t, beta, resid, delta)
        cur = F(beta)
        assert cur <= prev + 1e-12
        assert abs(oracle.objective(resid, beta, p.lam) - cur) < 1e-10 * cur
        j = int(out["kept"][0])
        for eps in (1e-4, -1e-4):
            b2 = beta.copy()
            b2[j] += eps
            assert F(b2) >= cur - 1e-13
        assert delta[j] == abs(out["dbeta"][0])
        prev = cur


def test_large_lambda_keeps_beta_at_zero():
    p = _small_dense(40, 60, n_true=4, seed=5, n_cand=20, n_keep=6)
    Xd, y = dense_array(p), p.y.numpy().astype(np.float64)
    lam = float(np.abs(Xd.T @ y).max()) * (1 + 1e-9)
    X = oracle_matrix(p)
    n2, beta, resid, delta = oracle.init(X, p.y.numpy(), 1e4)
    for t in range(30):
        oracle.round(X, n2, lam, p.eta, p.rho, 20, 6, 0, t, beta, resid, delta)
    assert np.all(beta == 0.0) and np.array_equal(resid, y)
    assert np.count_nonzero(delta == 0.0) > 0 and set(np.unique(delta)) <= {0.0, 1e4}


def test_update_uses_one_snapshot_of_the_residual():
    # Jacobi inside a round: every kept coefficient is computed from the pre-round r
    p = _small_dense(30, 10, n_true=3, seed=6, n_cand=10, n_keep=10, rho=2.0)
    X = oracle_matrix(p)
    Xd, y = dense_array(p), p.y.numpy().astype(np.float64)
    n2, beta, resid, delta = oracle.init(X, p.y.numpy(), 1e4)
    kept = np.array([3, 1, 7], dtype=np.int32)
    r0 = resid.copy()
    d = oracle.update(X, n2, p.lam, kept, beta, resid, delta)
    for a, j in enumerate(kept):
        z = Xd[:, j] @ r0 / n2[j]
        want = np.sign(z) * max(abs(z) - p.lam / n2[j], 0.0)
        assert abs(d[a] - want) < 1e-14
    assert np.allclose(resid, r0 - Xd[:, kept] @ d, rtol=0, atol=1e-13)


def test_non_unit_columns_use_the_general_minimiser():
    # columns of arbitrary norm: one full pass of single-coordinate updates still lowers F and the
    # fixed point satisfies KKT
    rng = np.random.default_rng(7)
    N, J = 40, 12
    xc = (rng.standard_normal((J, N)) * rng.uniform(0.2, 3.0, size=(J, 1))).astype(np.float32)
    xc[5] = 0.0                                                             # an all-zero column
    y = rng.standard_normal(N).astype(np.float32)
    X = oracle.Matrix.dense(xc)
    n2, beta, resid, delta = oracle.init(X, y, 1e4)
    lam = 0.8
    for t in range(3000):
        oracle.round(X, n2, lam, 1e-6, 0.5, 4, 2, 0, t, beta, resid, delta)
    assert beta[5] == 0.0
    assert _kkt_violation(xc.astype(np.float64).T, y.astype(np.float64), beta, lam) < 1e-6
