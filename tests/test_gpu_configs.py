"""The benchmark configurations against the oracle at sizes it can run in full.

c1 (1,000 x 10,000 dense, P' = 200, P = 32, 1,000 rounds) is run whole: teacher-forced rounds from identical
state (candidates bit-exact, kept list equal, coefficient changes within tolerance) in the first sweep and
in the late phase, and the free-running objective after all 1,000 rounds.  c2 .. c5 are too large for the
oracle to run whole, so their free-running objective is checked on replicas with N, J, the true support, P'
and P divided by ten, after a tenth of their rounds (their full sizes are checked round by round in
test_gpu_fullsize.py).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1312_5766_b200 import workloads as wl
from helpers import oracle_matrix

pytestmark = pytest.mark.gpu

RTOL_DBETA = 1e-5          # relative tolerance on a coefficient change
HALF_ULP32 = 2.0 ** -24    # the device stores beta in FP32: the change it makes is fl32(beta') - beta
RHO_EXCUSE = 1e-6
RTOL_OBJ = 1e-4


def _solver(p, **kw):
    from paper_1312_5766_b200 import binding
    return binding.StradsLasso.from_problem(p, device="cuda", **kw)


def _kept_matches(X, n2, cand, n_keep, rho, got_kept, got_examined):
    want, ne, mm = oracle.filter(X, n2, cand, n_keep, rho)
    if not np.array_equal(got_kept, want):
        assert mm <= RHO_EXCUSE, ("kept differs without a borderline pair", mm)
        want, ne, _ = oracle.filter(X, n2, cand, n_keep, rho, follow=got_kept, tol=RHO_EXCUSE)
        assert np.array_equal(got_kept, want)
    assert got_examined == ne


def _teacher_forced_round(p, X, n2, s, t):
    lam, eta, rho = float(np.float32(p.lam)), float(np.float32(p.eta)), float(np.float32(p.rho))
    beta = s.beta.cpu().numpy().astype(np.float64)
    resid = s.resid.cpu().numpy().astype(np.float64)
    delta = s.delta.cpu().numpy().astype(np.float64)
    cand_d, kept_d, dbeta_d, counts_d = s.round()
    counts = counts_d.cpu().numpy(); nk = int(counts[2])
    cand = cand_d.cpu().numpy(); kept = kept_d.cpu().numpy()[:nk]; d_got = dbeta_d.cpu().numpy()[:nk]
    assert np.array_equal(cand, oracle.sample(delta, eta, p.seed, t, p.n_candidates)), t
    _kept_matches(X, n2, cand, p.n_keep, rho, kept, int(counts[1]))
    b_old = beta[kept].copy()
    d_want = oracle.update(X, n2, lam, kept, beta, resid, delta)
    # entry by entry: 1e-5 of the change itself, plus the rounding of the new coefficient to FP32 (half an ulp of it)
    tol = RTOL_DBETA * np.abs(d_want) + HALF_ULP32 * 1.001 * np.abs(b_old + d_want)
    assert np.all(np.abs(d_got - d_want) <= tol), (t, np.abs(d_got - d_want).max())
    assert int(counts[3]) == int(np.count_nonzero(d_got))
    return nk


def test_c1_teacher_forced_rounds():
    p = wl.make_problem("c1", seed=0)
    X = oracle_matrix(p)
    n2 = oracle.colnorm2(X)
    s = _solver(p)
    t, kept = 0, 0
    # first sweep (every priority still C), the rounds in which the sweep ends (J / P = 312.5), the late phase
    for run_to, n_check in [(0, 6), (308, 8), (900, 6)]:
        s.run(run_to - t)
        t = run_to
        for _ in range(n_check):
            kept += _teacher_forced_round(p, X, n2, s, t)
            t += 1
    assert s.get_round() == t and kept > 0 and s.status() == (0, 0)


def test_c1_objective_after_all_rounds():
    p = wl.make_problem("c1", seed=0)
    assert p.rounds == 1000
    X = oracle_matrix(p)
    n2, beta, resid, delta = oracle.init(X, p.y.numpy(), 1e4)
    lam, eta, rho = float(np.float32(p.lam)), float(np.float32(p.eta)), float(np.float32(p.rho))
    f_mid = None
    for t in range(p.rounds):
        oracle.round(X, n2, lam, eta, rho, p.n_candidates, p.n_keep, p.seed, t, beta, resid, delta)
        if t == 399:
            f_mid = oracle.objective(resid, beta, lam)
    f_want = oracle.objective(resid, beta, lam)
    s = _solver(p)
    s.run(400)
    assert abs(s.objective() - f_mid) <= RTOL_OBJ * f_mid
    s.run(p.rounds - 400)
    f_got = s.objective()
    assert abs(f_got - f_want) <= RTOL_OBJ * f_want, (f_got, f_want)
    # the maintained FP32 residual still is y - X beta
    f_scratch, r_scratch = oracle.objective_from_scratch(X, p.y.numpy(), s.beta.cpu().numpy().astype(np.float64), lam)
    assert abs(f_scratch - f_got) <= 1e-5 * f_want
    assert np.abs(s.resid.cpu().numpy() - r_scratch).max() <= 1e-4 * np.abs(r_scratch).max()
    assert s.totals()["rounds"] == p.rounds and s.status() == (0, 0)


@pytest.mark.parametrize("name", ["c2", "c3", "c4", "c5"])
def test_tenth_size_replicas_objective(name):
    cfg = wl.scaled(name, 10)
    rounds = cfg["rounds"] // 10
    p = wl.make_problem(dict(cfg, name=name + "/10"), seed=0)
    X = oracle_matrix(p)
    n2, beta, resid, delta = oracle.init(X, p.y.numpy(), 1e4)
    lam, eta, rho = float(np.float32(p.lam)), float(np.float32(p.eta)), float(np.float32(p.rho))
    kept_want = 0
    for t in range(rounds):
        kept_want += int(oracle.round(X, n2, lam, eta, rho, p.n_candidates, p.n_keep, p.seed, t, beta, resid, delta)["counts"][2])
    f_want = oracle.objective(resid, beta, lam)
    f0 = oracle.objective(p.y.numpy().astype(np.float64), np.zeros(p.n_cols), lam)
    assert f_want < f0
    s = _solver(p)
    s.run(rounds)
    f_got = s.objective()
    assert abs(f_got - f_want) <= RTOL_OBJ * f_want, (name, f_got, f_want)
    tot = s.totals()
    assert tot["rounds"] == rounds and s.status()[0] == 0
    # the two runs made (nearly) the same number of updates: a borderline correlation may move a few
    assert abs(tot["kept"] - kept_want) <= 0.002 * kept_want + 2
    f_scratch, _ = oracle.objective_from_scratch(X, p.y.numpy(), s.beta.cpu().numpy().astype(np.float64), lam)
    assert abs(f_scratch - f_got) <= 1e-5 * f_want
