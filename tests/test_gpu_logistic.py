"""Logistic loss (STRADS_FLAG_LOGISTIC) through the C ABI against the oracle's logistic mode: initial state, whole
rounds from identical state, the free-running objective, and strads_run against rounds one by one."""
import numpy as np
import pytest
import torch

import oracle
from paper_1312_5766_b200 import workloads as wl
from helpers import oracle_matrix
from test_gpu_parity import HALF_ULP32, RTOL_DBETA, RTOL_OBJ, _small_problems

pytestmark = pytest.mark.gpu


def _b():
    from paper_1312_5766_b200 import binding
    return binding


def _problem(name, seed):
    return wl.to_logistic(wl.make_problem(_small_problems()[name], seed=seed), lam_frac=0.1)


@pytest.mark.parametrize("name", ["dense", "dense_grouped", "csc", "csc_zipf"])
def test_logistic_rounds_teacher_forced(name):
    b = _b()
    p = _problem(name, 51)
    X, y = oracle_matrix(p), p.y.numpy()
    s = b.StradsLasso.from_problem(p, device="cuda", flags=b.FLAG_LOGISTIC)
    n2, beta, margin, resid, delta = oracle.init_logistic(X, y, 1e4)
    lam, eta, rho = float(np.float32(p.lam)), float(np.float32(p.eta)), float(np.float32(p.rho))
    assert np.array_equal(s.resid.cpu().numpy(), (y - 0.5).astype(np.float32)) and not s.margin().any()
    f0 = s.objective()
    assert abs(f0 - oracle.objective_logistic(y, margin, beta, lam)) <= 1e-12 * f0
    assert abs(f0 - p.n_rows * np.log(2.0)) <= 1e-9 * f0
    t = 0
    sweep = p.n_cols // p.n_keep + 2
    for run_to, n_check in [(0, 5), (sweep, 5), (2 * sweep, 5)]:
        s.run(run_to - t)
        t = run_to
        for _ in range(n_check):
            beta[:] = s.beta.cpu().numpy(); margin[:] = s.margin().cpu().numpy(); delta[:] = s.delta.cpu().numpy()
            resid[:] = s.resid.cpu().numpy()
            cand_d, kept_d, dbeta_d, counts_d = s.round()
            counts = counts_d.cpu().numpy(); nk = int(counts[2])
            want = oracle.round_logistic(X, y, n2, lam, eta, rho, p.n_candidates, p.n_keep, p.seed, t, beta, margin, resid, delta)
            assert np.array_equal(cand_d.cpu().numpy(), want["cand"]), t
            assert np.array_equal(kept_d.cpu().numpy()[:nk], want["kept"]), t
            tol = RTOL_DBETA * np.abs(want["dbeta"]) + HALF_ULP32 * np.abs(beta[want["kept"]])
            assert np.all(np.abs(dbeta_d.cpu().numpy()[:nk] - want["dbeta"]) <= tol), t
            # the new margin and gradient vector (FP32 on the device) against the oracle's, from the same start
            mmax = max(np.abs(margin).max(), 1e-30)
            assert np.abs(s.margin().cpu().numpy() - margin).max() <= 2e-7 * mmax + 1e-7 * np.abs(beta).max()
            assert np.abs(s.resid.cpu().numpy() - resid).max() <= 2e-7 + 3e-7 * mmax
            t += 1
    assert s.status() == (0, 0) and s.get_round() == t


@pytest.mark.parametrize("name,rounds", [("dense", 600), ("csc", 900)])
def test_logistic_objective_after_fixed_rounds(name, rounds):
    b = _b()
    p = _problem(name, 52)
    X, y = oracle_matrix(p), p.y.numpy()
    n2, beta, margin, resid, delta = oracle.init_logistic(X, y, 1e4)
    lam, eta, rho = float(np.float32(p.lam)), float(np.float32(p.eta)), float(np.float32(p.rho))
    for t in range(rounds):
        oracle.round_logistic(X, y, n2, lam, eta, rho, p.n_candidates, p.n_keep, p.seed, t, beta, margin, resid, delta)
    f_want = oracle.objective_logistic(y, margin, beta, lam)
    s = b.StradsLasso.from_problem(p, device="cuda", flags=b.FLAG_LOGISTIC)
    f0 = s.objective()
    s.run(rounds)
    f_got = s.objective()
    assert f_want < 0.9 * f0 and abs(f_got - f_want) <= RTOL_OBJ * f_want, (f_got, f_want)
    # the maintained FP32 margin has not drifted from X beta
    b64 = s.beta.cpu().numpy().astype(np.float64)
    m_scratch = np.zeros(p.n_rows)
    if p.layout == wl.DENSE:
        m_scratch = p.values.numpy().astype(np.float64)[:, : p.n_rows].T @ b64
    else:
        v, r, cp = p.values.numpy(), p.row_idx.numpy(), p.col_ptr.numpy()
        for j in np.flatnonzero(b64):
            m_scratch[r[cp[j]:cp[j + 1]]] += v[cp[j]:cp[j + 1]].astype(np.float64) * b64[j]
    assert np.abs(s.margin().cpu().numpy() - m_scratch).max() <= 1e-4 * max(np.abs(m_scratch).max(), 1e-30)


@pytest.mark.parametrize("name,S", [("dense_grouped", 1), ("csc_zipf", 1), ("dense", 4)])
def test_logistic_run_equals_rounds(name, S):
    b = _b()
    p = _problem(name, 53)
    a, ref = (b.StradsLasso.from_problem(p, device="cuda", flags=b.FLAG_LOGISTIC, n_schedulers=S) for _ in range(2))
    n = 70
    a.run(n)
    for _ in range(n):
        ref.round()
    for x, y in ((a.beta, ref.beta), (a.resid, ref.resid), (a.delta, ref.delta), (a.margin(), ref.margin())):
        assert torch.equal(x, y)
    assert a.totals() == ref.totals() and a.status()[0] == 0


def test_logistic_from_nonzero_beta_and_host_round_refused():
    b = _b()
    for name in ("dense", "csc"):
        p = _problem(name, 54)
        b0 = torch.zeros(p.n_cols)
        idx = torch.randperm(p.n_cols, generator=torch.Generator().manual_seed(0))[:30]
        b0[idx] = torch.randn(30, generator=torch.Generator().manual_seed(1))
        s = b.StradsLasso.from_problem(p, device="cuda", flags=b.FLAG_LOGISTIC, beta0=b0)
        X, y = oracle_matrix(p), p.y.numpy()
        n2, beta, margin, resid, delta = oracle.init_logistic(X, y, 1e4)
        # the oracle's state for this beta: apply it as one update from zero with a huge step budget is not the same
        # thing, so build margin and gradient vector directly
        beta[:] = b0.numpy()
        margin[:] = 0.0
        if p.layout == wl.DENSE:
            margin[:] = p.values.numpy().astype(np.float64)[:, : p.n_rows].T @ beta
        else:
            v, r, cp = p.values.numpy(), p.row_idx.numpy(), p.col_ptr.numpy()
            for j in np.flatnonzero(beta):
                margin[r[cp[j]:cp[j + 1]]] += v[cp[j]:cp[j + 1]].astype(np.float64) * beta[j]
        f_want = oracle.objective_logistic(y, margin, beta, float(np.float32(p.lam)))
        assert np.abs(s.margin().cpu().numpy() - margin).max() <= 2e-7 * np.abs(margin).max()
        assert abs(s.objective() - f_want) <= 1e-6 * f_want
        h = [t.cpu().pin_memory() for t in (s.beta, s.resid, s.delta)]
        with pytest.raises(b.StradsError) as e:
            s.round_host(*h)
        assert e.value.code == -7
    plain = b.StradsLasso.from_problem(wl.make_problem(_small_problems()["dense"], seed=1), device="cuda")
    with pytest.raises(b.StradsError):
        plain.margin()
