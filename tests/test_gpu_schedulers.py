"""Round-robin scheduler threads (Section 3) on the device: every round against the oracle's scheduler
mode from identical state, and the pipelined strads_run against the same rounds run one by one."""
import numpy as np
import pytest
import torch

import oracle
from paper_1312_5766_b200 import workloads as wl
from helpers import oracle_matrix
from test_gpu_parity import (HALF_ULP32, RTOL_DBETA, RTOL_OBJ, _assert_kept_matches, _small_problems, _solver)

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,S", [("dense", 2), ("dense", 4), ("dense_grouped", 3), ("csc", 4), ("csc_zipf", 2)])
def test_rounds_teacher_forced_with_schedulers(name, S):
    """Round t is dispatched by scheduler t mod S: candidates bit-exact and all of its own coefficients,
    kept equal, changes within tolerance, from the device's state before every round."""
    p = wl.make_problem(_small_problems()[name], seed=6)
    X = oracle_matrix(p)
    s = _solver(p, n_schedulers=S)
    n2, beta, resid, delta = oracle.init(X, p.y.numpy(), 1e4)
    lam, eta, rho = float(np.float32(p.lam)), float(np.float32(p.eta)), float(np.float32(p.rho))
    n_rounds = 6 * S + 1
    for t in range(n_rounds):
        beta[:] = s.beta.cpu().numpy(); resid[:] = s.resid.cpu().numpy(); delta[:] = s.delta.cpu().numpy()
        cand_d, kept_d, dbeta_d, counts_d = s.round()
        counts = counts_d.cpu().numpy(); nk = int(counts[2])
        cand = cand_d.cpu().numpy(); kept = kept_d.cpu().numpy()[:nk]; d_got = dbeta_d.cpu().numpy()[:nk]
        assert np.all(cand % S == t % S)
        assert np.array_equal(cand, oracle.sample_part(delta, eta, p.seed, t, S, t % S, p.n_candidates)), t
        _assert_kept_matches(X, n2, cand, p.n_keep, rho, kept, int(counts[1]))
        d_want = oracle.update(X, n2, lam, kept, beta, resid, delta)
        assert np.all(np.abs(d_got - d_want) <= RTOL_DBETA * np.abs(d_want) + HALF_ULP32 * np.abs(beta[kept])), t
    assert s.get_round() == n_rounds
    tot = s.totals()
    assert tot["rounds"] == n_rounds and tot["kept"] > 0
    assert s.status() == (0, 0)


@pytest.mark.parametrize("name,S,n_keep,n_cand", [("dense", 2, 24, 1024), ("dense", 4, 48, 300), ("dense_grouped", 4, 120, 400),
                                                  ("dense_grouped", 3, 40, 600), ("csc", 4, 100, 1000),
                                                  ("csc_zipf", 2, 300, 1500), ("csc_zipf", 8, 400, 1500)])
def test_pipelined_run_equals_rounds_one_by_one(name, S, n_keep, n_cand):
    """strads_run prepares the blocks of later rounds on the schedulers' own streams while an update runs
    (captured sequences of 16 turns each, the rest enqueued directly); the state must be bit-identical to
    strads_round called the same number of times, whatever the split into calls."""
    cfg = dict(_small_problems()[name], n_keep=n_keep, n_candidates=n_cand)
    p = wl.make_problem(cfg, seed=15)
    a, b = _solver(p, n_schedulers=S), _solver(p, n_schedulers=S)
    calls = [3, 16 * S + 5, 1, 2 * 16 * S, S + 2]     # unaligned head, a captured sequence + tail, single round, ...
    for n in calls:
        a.run(n)
    n_total = sum(calls)
    kept_total = 0
    for _ in range(n_total):
        kept_total += int(b.round()[3][2])
    assert a.get_round() == b.get_round() == n_total
    for x, y in ((a.beta, b.beta), (a.resid, b.resid), (a.delta, b.delta)):
        assert torch.equal(x, y)
    assert a.totals() == b.totals() and a.totals()["kept"] == kept_total
    assert a.status()[0] == 0 and b.status()[0] == 0
    # rounds mixed with runs on one handle, and a resumed handle
    a.round(); a.run(2 * S + 1)
    for _ in range(2 * S + 2):
        b.round()
    assert torch.equal(a.beta, b.beta) and torch.equal(a.delta, b.delta) and torch.equal(a.resid, b.resid)
    c = _solver(p, n_schedulers=S)
    c.beta.copy_(b.beta); c.resid.copy_(b.resid); c.delta.copy_(b.delta)
    c.set_round(b.get_round())
    b.run(S + 3); c.run(S + 3)
    assert torch.equal(c.beta, b.beta) and torch.equal(c.delta, b.delta) and torch.equal(c.resid, b.resid)


@pytest.mark.parametrize("name,rounds,S", [("dense", 800, 4), ("csc", 1200, 2)])
def test_objective_after_fixed_rounds_with_schedulers(name, rounds, S):
    p = wl.make_problem(_small_problems()[name], seed=3)
    X = oracle_matrix(p)
    s = _solver(p, n_schedulers=S)
    s.run(rounds)
    got = s.objective()
    n2, beta, resid, delta = oracle.init(X, p.y.numpy(), 1e4)
    lam, eta, rho = float(np.float32(p.lam)), float(np.float32(p.eta)), float(np.float32(p.rho))
    for t in range(rounds):
        oracle.round(X, n2, lam, eta, rho, p.n_candidates, p.n_keep, p.seed, t, beta, resid, delta, n_sched=S)
    want = oracle.objective(resid, beta, lam)
    assert abs(got - want) <= RTOL_OBJ * abs(want)
    scratch, _ = oracle.objective_from_scratch(X, p.y.numpy(), s.beta.cpu().numpy().astype(np.float64), lam)
    assert abs(got - scratch) <= RTOL_OBJ * abs(scratch)


def test_scheduler_arguments():
    p = wl.make_problem(_small_problems()["dense"], seed=1)       # J = 3000, P' = 300
    with pytest.raises(Exception):
        _solver(p, n_schedulers=9)                                # beyond STRADS_MAX_SCHEDULERS
    with pytest.raises(Exception):
        _solver(dataclass_replace(p, n_candidates=1501), n_schedulers=2)   # P' > J / S
    s = _solver(p, n_schedulers=2)
    with pytest.raises(Exception):
        s.profile_begin(4)                                        # step timing needs one scheduler


def dataclass_replace(p, **kw):
    import copy
    q = copy.copy(p)
    for k, v in kw.items():
        setattr(q, k, v)
    return q
