"""Pins for the oracle's candidate sampler (Algorithm 1, "draw a set of P' coefficients").

The ranking of race keys must realise sampling WITHOUT replacement with
probabilities proportional to w_j = delta_j^2 + eta (successive sampling /
Plackett-Luce).  Checked by exact enumeration on tiny J, by the uniform special
case, and by the full-sweep behaviour the paper describes for the first phase.
"""
import itertools
import math

import numpy as np

import oracle


def test_sample_is_the_sorted_prefix_of_the_keys():
    rng = np.random.default_rng(0)
    J = 5000
    delta = rng.choice([0.0, 1e-3, 0.1, 1.0, 1e4], size=J)
    cand, keys = oracle.sample(delta, 1e-6, seed=7, t=3, n_cand=300, return_keys=True)
    # keys are the per-coefficient race keys
    for j in (0, 1, 2, 3, 4, 4999):
        assert keys[j] == np.float32(oracle.race_key(delta[j], 1e-6, oracle.draw_word(7, 3, j)))
    order = np.lexsort((np.arange(J), keys))          # by key, ties by index
    assert np.array_equal(cand, order[:300].astype(np.int32))
    assert len(set(cand.tolist())) == 300


def test_ties_go_to_the_smaller_index():
    # infinite priority makes every race time exactly 0: a complete tie
    J = 1000
    delta = np.full(J, np.inf)
    cand = oracle.sample(delta, 1e-6, seed=1, t=0, n_cand=17)
    assert cand.tolist() == list(range(17))
    delta[:500] = 0.0                                   # finite times lose against the zeros
    cand = oracle.sample(delta, 1e-6, seed=1, t=0, n_cand=17)
    assert cand.tolist() == list(range(500, 517))


def test_ordered_pairs_follow_successive_sampling():
    # J = 6, P' = 2: compare ordered-pair frequencies with w_a/W * w_b/(W - w_a)
    delta = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 0.25])
    eta = 0.05
    w = np.array([float(np.float32(d) * np.float32(d) + np.float32(eta)) for d in delta])
    W = w.sum()
    rounds = 120000
    counts = {}
    for t in range(rounds):
        a, b = oracle.sample(delta, eta, seed=11, t=t, n_cand=2).tolist()
        counts[(a, b)] = counts.get((a, b), 0) + 1
    chi2 = 0.0
    for a, b in itertools.permutations(range(6), 2):
        expect = rounds * w[a] / W * w[b] / (W - w[a])
        chi2 += (counts.get((a, b), 0) - expect) ** 2 / expect
    # 29 dof: mean 29, sd 7.6
    assert chi2 < 29 + 5 * math.sqrt(58), chi2


def test_equal_weights_give_uniform_subsets():
    J, k, rounds = 7, 3, 70000
    delta = np.full(J, 0.3)
    first = np.zeros(J)
    member = np.zeros(J)
    for t in range(rounds):
        c = oracle.sample(delta, 1e-6, seed=5, t=t, n_cand=k)
        first[c[0]] += 1
        member[c] += 1
    chi_first = ((first - rounds / J) ** 2 / (rounds / J)).sum()
    assert chi_first < 6 + 5 * math.sqrt(12), chi_first
    # inclusion probability k/J for every coefficient
    p = k / J
    z = (member - rounds * p) / math.sqrt(rounds * p * (1 - p))
    assert np.abs(z).max() < 4.5, z


def test_first_phase_is_a_full_sweep():
    # With delta = C everywhere, coefficients that were updated (delta drops to O(1) or 0) lose
    # to the never-updated ones, so all J are visited once before any is visited twice.
    J, k, C = 600, 50, 1e4
    delta = np.full(J, C)
    seen = set()
    for t in range(J // k):
        cand = oracle.sample(delta, 1e-6, seed=3, t=t, n_cand=k)
        assert not (set(cand.tolist()) & seen)
        seen |= set(cand.tolist())
        delta[cand] = 0.7                                # pretend all candidates were updated
    assert len(seen) == J


def test_bad_arguments_are_rejected():
    import pytest
    with pytest.raises(ValueError):
        oracle.sample(np.ones(4), 1e-6, 0, 0, n_cand=5)
