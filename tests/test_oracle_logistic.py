"""Pins for the oracle's logistic-loss mode (no GPU): the optimality conditions of the l1-regularised logistic
regression at convergence, an independent solver on tiny problems, the descent guarantee of the bounded-curvature
step, and the bookkeeping of margin and gradient vector."""
import numpy as np
import pytest
import scipy.optimize

import oracle
from paper_1312_5766_b200 import workloads as wl
from helpers import dense_array, oracle_matrix


def _sigma(m):
    return 1.0 / (1.0 + np.exp(-m))


def _objective(A, y, beta, lam):
    m = A @ beta
    return float(np.sum(np.logaddexp(0.0, m) - y * m) + lam * np.abs(beta).sum())


def _problem(kind, seed, **over):
    cfg = {"dense": dict(kind="dense_iid", n_rows=120, n_cols=200, n_true=8, lam_frac=0.1, n_candidates=40, n_keep=8, rho=0.2),
           "csc": dict(kind="csc_uniform", n_rows=300, n_cols=400, n_true=10, lam_frac=0.1, nnz_col=12, n_candidates=60,
                       n_keep=10, rho=0.2)}[kind]
    cfg.update(over)
    return wl.to_logistic(wl.make_problem(cfg, seed=seed), lam_frac=0.2)


@pytest.mark.parametrize("kind", ["dense", "csc"])
def test_kkt_at_convergence(kind):
    p = _problem(kind, 3)
    X, y = oracle_matrix(p), p.y.numpy()
    n2, beta, margin, resid, delta = oracle.init_logistic(X, y, 1e4)
    lam = float(p.lam)
    for t in range(6000):
        oracle.round_logistic(X, y, n2, lam, 1e-6, p.rho, p.n_candidates, p.n_keep, 5, t, beta, margin, resid, delta)
    A = dense_array(p)
    g = A.T @ (y - _sigma(A @ beta))                       # minus the gradient of the loss, from beta alone
    zero = beta == 0
    assert np.count_nonzero(~zero) > 0
    assert np.all(np.abs(g[zero]) <= lam * (1 + 1e-6))
    assert np.allclose(g[~zero], lam * np.sign(beta[~zero]), rtol=1e-6, atol=1e-9)
    # bookkeeping: the maintained margin and gradient vector are those of beta
    assert np.allclose(margin, A @ beta, rtol=0, atol=1e-10)
    assert np.allclose(resid, y - _sigma(A @ beta), rtol=0, atol=1e-12)
    assert abs(oracle.objective_logistic(y, margin, beta, lam) - _objective(A, y, beta, lam)) < 1e-10


def test_optimum_against_an_independent_solver():
    # tiny problem: L-BFGS-B on beta = u - v, u, v >= 0 (smooth objective, bound constraints)
    p = _problem("dense", 7, n_rows=60, n_cols=9, n_true=3, n_candidates=9, n_keep=1)
    X, y, A = oracle_matrix(p), p.y.numpy().astype(np.float64), dense_array(p)
    lam = float(p.lam)
    J = p.n_cols

    def f(w):
        b = w[:J] - w[J:]
        m = A @ b
        val = np.sum(np.logaddexp(0.0, m) - y * m) + lam * w.sum()
        gb = A.T @ (_sigma(m) - y)
        return val, np.concatenate([gb + lam, -gb + lam])

    res = scipy.optimize.minimize(f, np.zeros(2 * J), jac=True, method="L-BFGS-B", bounds=[(0, None)] * (2 * J),
                                  options=dict(maxiter=5000, ftol=1e-15, gtol=1e-12))
    n2, beta, margin, resid, delta = oracle.init_logistic(X, p.y.numpy(), 1e4)
    for t in range(8000):
        oracle.round_logistic(X, p.y.numpy(), n2, lam, 1e-6, p.rho, p.n_candidates, p.n_keep, 1, t, beta, margin, resid, delta)
    f_oracle = oracle.objective_logistic(p.y.numpy(), margin, beta, lam)
    assert abs(f_oracle - res.fun) <= 1e-8 * abs(res.fun), (f_oracle, res.fun)
    assert np.allclose(beta, res.x[:J] - res.x[J:], atol=1e-4)


def test_single_coordinate_steps_descend_and_minimise_the_bound():
    p = _problem("dense", 11, n_candidates=1, n_keep=1)
    X, y, A = oracle_matrix(p), p.y.numpy(), dense_array(p)
    n2, beta, margin, resid, delta = oracle.init_logistic(X, y, 1e4)
    lam = float(p.lam)
    f_prev = oracle.objective_logistic(y, margin, beta, lam)
    moved = 0
    for t in range(600):
        b_before = beta.copy()
        g_all = A.T @ (y - _sigma(A @ b_before))
        out = oracle.round_logistic(X, y, n2, lam, 1e-6, p.rho, 1, 1, 2, t, beta, margin, resid, delta)
        f = oracle.objective_logistic(y, margin, beta, lam)
        assert f <= f_prev + 1e-12                          # the curvature bound n_j / 4 makes every step a descent step
        f_prev = f
        j = int(out["kept"][0])
        # beta_j' minimises  -g (b - b0) + (n_j / 8) (b - b0)^2 + lambda |b|  over b
        q = lambda b: -g_all[j] * (b - b_before[j]) + n2[j] / 8.0 * (b - b_before[j]) ** 2 + lam * abs(b)
        for eps in (1e-6, -1e-6, 1e-3, -1e-3):
            assert q(beta[j]) <= q(beta[j] + eps) + 1e-15
        moved += out["dbeta"][0] != 0.0
    assert moved > 50


def test_large_lambda_keeps_beta_at_zero():
    p = _problem("csc", 13)
    X, y, A = oracle_matrix(p), p.y.numpy(), dense_array(p)
    lam = float(np.abs(A.T @ (y - 0.5)).max()) * 1.0001
    n2, beta, margin, resid, delta = oracle.init_logistic(X, y, 1e4)
    assert np.array_equal(resid, y - 0.5) and not margin.any()
    for t in range(50):
        oracle.round_logistic(X, y, n2, lam, 1e-6, p.rho, p.n_candidates, p.n_keep, 3, t, beta, margin, resid, delta)
    assert not beta.any() and not margin.any()


def test_round_is_sample_filter_update_from_one_snapshot():
    p = _problem("dense", 17)
    X, y = oracle_matrix(p), p.y.numpy()
    n2, beta, margin, resid, delta = oracle.init_logistic(X, y, 1e4)
    lam = float(p.lam)
    for t in range(5):
        b0, m0, r0, d0 = beta.copy(), margin.copy(), resid.copy(), delta.copy()
        out = oracle.round_logistic(X, y, n2, lam, 1e-6, p.rho, p.n_candidates, p.n_keep, 9, t, beta, margin, resid, delta)
        cand = oracle.sample(d0, 1e-6, 9, t, p.n_candidates)
        kept, ne, _ = oracle.filter(X, n2, cand, p.n_keep, p.rho)
        assert np.array_equal(out["cand"], cand) and np.array_equal(out["kept"], kept)
        # every change from the round's first gradient vector (Jacobi), not from one updated on the way
        A = dense_array(p)
        for a, j in enumerate(kept):
            z = b0[j] + 4.0 * (A[:, j] @ r0) / n2[j]
            want = np.sign(z) * max(abs(z) - 4.0 * lam / n2[j], 0.0) - b0[j]
            assert abs(out["dbeta"][a] - want) <= 1e-12 * max(1.0, abs(want))
