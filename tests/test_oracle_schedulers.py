"""Pins of the oracle's round-robin scheduler mode (STRADS, "Implementation Overview": S scheduler
threads, each owning a fixed disjoint set of J/S coefficients, taking turns to dispatch a block).

None of these calls the CUDA library."""
import itertools
import math

import numpy as np
import pytest

import oracle


def _delta(J, seed=0):
    rng = np.random.default_rng(seed)
    d = np.abs(rng.normal(size=J))
    d[rng.random(J) < 0.3] = 0.0          # coefficients that did not move: weight eta
    return d


def test_one_scheduler_is_the_plain_sampler():
    d = _delta(300)
    for t in (0, 5, 2**33 + 1):
        assert oracle.sample_part(d, 1e-6, 9, t, 1, 0, 40).tolist() == oracle.sample(d, 1e-6, 9, t, 40).tolist()


@pytest.mark.parametrize("J,S", [(300, 2), (301, 3), (302, 4), (303, 4), (97, 8)])
def test_a_scheduler_ranks_its_own_coefficients_like_the_global_ranking(J, S):
    # the keys do not depend on S: thread s's list is the global ranking of ALL J keys with the
    # coefficients of the other threads struck out
    d = _delta(J, seed=J)
    full = oracle.sample(d, 1e-6, 3, 17, J)
    for s in range(S):
        own = [j for j in full.tolist() if j % S == s]
        n = min(len(own), 25)
        got = oracle.sample_part(d, 1e-6, 3, 17, S, s, n).tolist()
        assert got == own[:n]
        assert all(j % S == s for j in got)
    # the whole of a partition can be asked for, one more cannot
    members0 = len(range(0, J, S))
    assert sorted(oracle.sample_part(d, 1e-6, 3, 17, S, 0, members0).tolist()) == list(range(0, J, S))
    with pytest.raises(ValueError):
        oracle.sample_part(d, 1e-6, 3, 17, S, 0, members0 + 1)


def test_bad_scheduler_arguments_are_rejected():
    d = _delta(20)
    for S, s in ((0, 0), (2, 2), (2, -1)):
        with pytest.raises(ValueError):
            oracle.sample_part(d, 1e-6, 1, 0, S, s, 2)


def test_a_scheduler_samples_from_its_own_importance_distribution():
    # J = 8, S = 2, thread 1 owns {1, 3, 5, 7}: ordered pairs must follow successive sampling with the
    # weights of those four coefficients alone (p_s(j) of the paper), whatever the other weights are
    delta = np.array([9.0, 0.0, 7.0, 0.5, 3.0, 1.0, 8.0, 1.5])
    eta = 0.05
    own = [1, 3, 5, 7]
    w = {j: float(np.float32(delta[j]) * np.float32(delta[j]) + np.float32(eta)) for j in own}
    W = sum(w.values())
    rounds = 60000
    counts = {}
    for t in range(rounds):
        a, b = oracle.sample_part(delta, eta, 21, t, 2, 1, 2).tolist()
        counts[(a, b)] = counts.get((a, b), 0) + 1
    assert set(j for ab in counts for j in ab) <= set(own)
    chi2 = 0.0
    for a, b in itertools.permutations(own, 2):
        expect = rounds * w[a] / W * w[b] / (W - w[a])
        chi2 += (counts.get((a, b), 0) - expect) ** 2 / expect
    assert chi2 < 11 + 5 * math.sqrt(22), chi2      # 11 dof


def _small_problem(J=60, N=40, seed=4):
    rng = np.random.default_rng(seed)
    x = rng.normal(size=(J, N))
    x -= x.mean(axis=1, keepdims=True)
    x /= np.linalg.norm(x, axis=1, keepdims=True)
    x = x.astype(np.float32)
    bstar = np.zeros(J)
    bstar[rng.choice(J, 6, replace=False)] = rng.normal(size=6) * 2
    y = (x.T.astype(np.float64) @ bstar + 0.05 * rng.normal(size=N)).astype(np.float32)
    lam = 0.05 * float(np.abs(x.astype(np.float64) @ y.astype(np.float64)).max())
    return oracle.Matrix.dense(x), y, lam


@pytest.mark.parametrize("S", [2, 3])
def test_turn_taking_and_preparing_a_block_ahead_changes_nothing(S):
    # Round t belongs to thread t mod S; only that thread's coefficients may change in it.  And since
    # nobody else touches delta of thread s between its turns, the block of round t can be prepared
    # as soon as round t - S is over: the candidates drawn from the state S - 1 rounds earlier are
    # the ones drawn at the start of round t.
    X, y, lam = _small_problem()
    n2, beta, resid, delta = oracle.init(X, y, 1e4)
    J = X.n_cols
    snapshots = []
    for t in range(40):
        snapshots.append(delta.copy())
        b0, d0 = beta.copy(), delta.copy()
        out = oracle.round(X, n2, lam, 1e-6, 0.3, 8, 3, 5, t, beta, resid, delta, n_sched=S)
        s = t % S
        assert all(j % S == s for j in out["cand"].tolist())
        changed = np.nonzero((beta != b0) | (delta != d0))[0]
        assert all(j % S == s for j in changed.tolist())
        early = snapshots[max(0, t - S + 1)]
        assert oracle.sample_part(early, 1e-6, 5, t, S, s, 8).tolist() == out["cand"].tolist()
    # the maintained residual is still y - X beta
    scratch, r = oracle.objective_from_scratch(X, y, beta, lam)
    assert np.allclose(r, resid, rtol=0, atol=1e-12)
    assert abs(oracle.objective(resid, beta, lam) - scratch) <= 1e-12 * max(1.0, abs(scratch))


def test_round_robin_reaches_the_same_optimum():
    # the schedule changes the path, not the fixed point: KKT of eq. 1 at convergence
    X, y, lam = _small_problem(J=40, N=60, seed=8)
    n2, beta, resid, delta = oracle.init(X, y, 1e4)
    for t in range(4000):
        oracle.round(X, n2, lam, 1e-6, 0.5, 6, 2, 1, t, beta, resid, delta, n_sched=4)
    g = oracle.gradient(X, resid)
    zero = beta == 0
    assert np.all(np.abs(g[zero]) <= lam * (1 + 1e-6))
    assert np.allclose(g[~zero], lam * np.sign(beta[~zero]), rtol=1e-6, atol=1e-9)
