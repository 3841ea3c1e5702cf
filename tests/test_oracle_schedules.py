"""Pins for the oracle's other schedules (no GPU).

  - the importance distribution of Algorithm 1 as printed, p(j) ~ |beta_j^(t_j-2) - beta_j^(t_j-1)| + eta,
    and the uniform draw of the static and random schedulers the paper compares with (Section 5.1);
  - no dependency check (the random scheduler);
  - dependencies dropped at run time (Section 1, "Dynamic Block Structures"; SAP step 4).
Each is checked against something other than itself: the exact successive-sampling probabilities of the
weights, numpy correlations and a greedy walk written out here, the Lasso optimum every schedule must reach.
"""
import itertools
import math

import numpy as np
import pytest

import oracle
from paper_1312_5766_b200 import workloads as wl
from helpers import dense_array, oracle_matrix


def test_abs_weight_key_is_its_definition():
    rng = np.random.default_rng(0)
    for _ in range(200):
        d, eta, x = float(rng.choice([0.0, 1e-4, 0.3, 2.0, 1e4])), float(rng.choice([1e-6, 1e-4, 0.05])), int(rng.integers(0, 2**32))
        E = np.float32(oracle.unit_exponential(x))
        want = E / (np.abs(np.float32(d)) + np.float32(eta))            # binary32 operations, as specified
        assert np.float32(oracle.race_key_mode(d, eta, x, "abs")) == np.float32(want)
        assert np.float32(oracle.race_key_mode(d, eta, x, "uniform")) == E
        assert oracle.race_key_mode(d, eta, x, "square") == oracle.race_key(d, eta, x)


def test_abs_weight_ordered_pairs_follow_successive_sampling():
    # J = 6, P' = 2: ordered-pair frequencies against w_a / W * w_b / (W - w_a) with w = |delta| + eta
    delta = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 0.25])
    eta = 0.05
    w = np.array([float(np.float32(d) + np.float32(eta)) for d in delta])
    W = w.sum()
    rounds = 120000
    counts = {}
    for t in range(rounds):
        a, b = oracle.sample(delta, eta, seed=13, t=t, n_cand=2, weight="abs").tolist()
        counts[(a, b)] = counts.get((a, b), 0) + 1
    chi2 = 0.0
    for a, b in itertools.permutations(range(6), 2):
        expect = rounds * w[a] / W * w[b] / (W - w[a])
        chi2 += (counts.get((a, b), 0) - expect) ** 2 / expect
    assert chi2 < 29 + 5 * math.sqrt(58), chi2                           # 29 dof
    # and it is not the squared weight: the two distributions differ far beyond that bound
    w2 = np.array([float(np.float32(d) * np.float32(d) + np.float32(eta)) for d in delta])
    chi2_sq = sum((counts.get((a, b), 0) - rounds * w2[a] / w2.sum() * w2[b] / (w2.sum() - w2[a])) ** 2
                  / (rounds * w2[a] / w2.sum() * w2[b] / (w2.sum() - w2[a])) for a, b in itertools.permutations(range(6), 2))
    assert chi2_sq > 1000


def test_uniform_draw_ignores_the_priorities():
    rng = np.random.default_rng(1)
    J = 3000
    delta = rng.choice([0.0, 1e-3, 1.0, 1e4], size=J)
    for t in range(3):
        got = oracle.sample(delta, 1e-6, seed=2, t=t, n_cand=100, weight="uniform")
        assert np.array_equal(got, oracle.sample(np.ones(J), 0.0, seed=2, t=t, n_cand=100))    # w = 1 exactly


def _walk(corr, cand, n_keep, rho, dormant):
    """Greedy first-fit written out on a matrix of correlations; a pair with a dormant member does not couple."""
    kept = []
    examined = 0
    for c in cand:
        if len(kept) == n_keep:
            break
        examined += 1
        if dormant[c] or all(dormant[k] or abs(corr[c, k]) < rho for k in kept):
            kept.append(int(c))
    return np.array(kept, dtype=np.int32), examined


@pytest.mark.parametrize("kind", ["dense_grouped", "csc_zipf"])
def test_dynamic_filter_against_a_walk_on_numpy_correlations(kind):
    cfg = {"dense_grouped": dict(kind="dense_grouped", n_rows=300, n_cols=400, n_true=10, lam_frac=0.05, n_candidates=200,
                                 n_keep=60, rho=0.1, group=20),
           "csc_zipf": dict(kind="csc_zipf", n_rows=400, n_cols=500, n_true=10, lam_frac=0.05, nnz_col=8,
                            n_candidates=250, n_keep=80, rho=0.05)}[kind]
    p = wl.make_problem(cfg, seed=31)
    X = oracle_matrix(p)
    n2 = oracle.colnorm2(X)
    A = dense_array(p)
    nrm = np.sqrt((A * A).sum(axis=0))
    corr = (A.T @ A) / np.outer(nrm, nrm)
    rng = np.random.default_rng(5)
    for trial in range(6):
        beta = np.where(rng.random(p.n_cols) < 0.3, rng.normal(size=p.n_cols), 0.0)
        delta = np.where(rng.random(p.n_cols) < 0.5, 0.0, np.abs(rng.normal(size=p.n_cols)))
        if trial == 0:
            delta[:] = 1e4; beta[:] = 0.0                                  # nothing updated yet: nobody is dormant
        if trial == 1:
            delta[:] = 0.0; beta[:] = 0.0                                  # everybody dormant
        dormant = (beta == 0.0) & (delta == 0.0)
        cand = rng.permutation(p.n_cols)[: p.n_candidates].astype(np.int32)
        if kind == "dense_grouped" and trial % 2 == 0:
            cand = np.arange(p.n_candidates, dtype=np.int32)               # whole groups side by side
        kept, ne = oracle.filter_dynamic(X, n2, cand, p.n_keep, p.rho, beta, delta)
        want, want_ne = _walk(corr, cand, p.n_keep, p.rho, dormant)
        assert np.array_equal(kept, want) and ne == want_ne, trial
        # what the modified coupling demands: active kept pairs are below rho; every rejected candidate is active and
        # conflicts with an earlier kept active one; dormant candidates inside the examined range are all kept
        act = [k for k in kept if not dormant[k]]
        for a, b in itertools.combinations(act, 2):
            assert abs(corr[a, b]) < p.rho
        pos = {int(c): i for i, c in enumerate(cand)}
        for c in cand[:ne]:
            if c in kept:
                continue
            assert not dormant[c]
            assert any(abs(corr[c, k]) >= p.rho and pos[int(k)] < pos[int(c)] for k in act)
        if trial == 0:                                                     # reduces to Algorithm 1's filter
            plain, plain_ne, _ = oracle.filter(X, n2, cand, p.n_keep, p.rho)
            assert np.array_equal(kept, plain) and ne == plain_ne
        if trial == 1:
            assert np.array_equal(kept, cand[: p.n_keep])
    # on this data the two filters do differ once coefficients have gone dormant
    beta = np.zeros(p.n_cols); delta = np.zeros(p.n_cols); delta[::2] = 0.3
    cand = np.arange(p.n_candidates, dtype=np.int32)
    assert len(oracle.filter_dynamic(X, n2, cand, p.n_keep, p.rho, beta, delta)[0]) >= len(oracle.filter(X, n2, cand, p.n_keep, p.rho)[0])


def test_no_filter_keeps_the_first_candidates():
    p = wl.make_problem(dict(kind="dense_grouped", n_rows=200, n_cols=400, n_true=10, lam_frac=0.05, n_candidates=100,
                             n_keep=30, rho=0.1, group=20), seed=3)
    X = oracle_matrix(p)
    n2, beta, resid, delta = oracle.init(X, p.y.numpy(), 1e4)
    out = oracle.round(X, n2, p.lam, p.eta, p.rho, p.n_candidates, p.n_keep, 1, 0, beta, resid, delta, weight="uniform", filter="none")
    assert np.array_equal(out["kept"], out["cand"][: p.n_keep]) and out["counts"].tolist()[:3] == [100, 30, 30]
    assert np.array_equal(out["cand"], oracle.sample(np.ones(p.n_cols), 0.0, 1, 0, p.n_candidates))


@pytest.mark.parametrize("weight,filt", [("abs", "rho"), ("uniform", "rho"), ("square", "dynamic"), ("abs", "dynamic")])
def test_every_schedule_reaches_the_lasso_optimum(weight, filt):
    """A schedule changes the path, not the fixed point: KKT at convergence (Eq. 1's optimality conditions)."""
    p = wl.make_problem(dict(kind="dense_grouped", n_rows=120, n_cols=200, n_true=8, lam_frac=0.1, n_candidates=40,
                             n_keep=8, rho=0.2, group=10), seed=9)
    X = oracle_matrix(p)
    n2, beta, resid, delta = oracle.init(X, p.y.numpy(), 1e4)
    lam = float(p.lam)
    for t in range(4000):
        oracle.round(X, n2, lam, 1e-6, p.rho, p.n_candidates, p.n_keep, 7, t, beta, resid, delta, weight=weight, filter=filt)
    g = oracle.gradient(X, resid)
    zero = beta == 0
    assert np.all(np.abs(g[zero]) <= lam * (1 + 1e-6))
    assert np.allclose(g[~zero], lam * np.sign(beta[~zero]), rtol=1e-6, atol=1e-9)
    f_scratch, r_scratch = oracle.objective_from_scratch(X, p.y.numpy(), beta, lam)
    assert np.allclose(r_scratch, resid, rtol=0, atol=1e-10)
