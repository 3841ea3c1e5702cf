"""Pins for the oracle's dependency filter (Algorithm 1, the rho condition), no GPU.

The kept set is checked through properties that need no second implementation
(validity, first-fit maximality, the stop at P), through a construction whose
answer is known (groups of strongly correlated columns), and the correlations
through numpy / scipy on the same columns.
"""
import numpy as np
import scipy.sparse as sp

import oracle
from paper_1312_5766_b200 import workloads as wl
from helpers import dense_array, oracle_matrix


def _check_first_fit(corr_abs, cand, kept, n_examined, n_keep, rho):
    kept = list(kept)
    pos = {c: i for i, c in enumerate(cand)}
    assert len(set(kept)) == len(kept) <= n_keep and all(k in pos for k in kept)
    assert [pos[k] for k in kept] == sorted(pos[k] for k in kept)            # keep order = walk order
    for a in kept:                                                            # validity
        for b in kept:
            if a != b:
                assert corr_abs[a, b] < rho
    if len(kept) == n_keep:                                                   # stops exactly at P
        assert n_examined == pos[kept[-1]] + 1
    else:
        assert n_examined == len(cand)
    for c in cand[:n_examined]:                                               # maximality
        if c not in kept:
            earlier = [k for k in kept if pos[k] < pos[c]]
            assert any(corr_abs[c, k] >= rho for k in earlier)


def test_dense_filter_properties():
    p = wl.make_problem(dict(kind="dense_iid", n_rows=40, n_cols=300, n_true=5, lam_frac=0.1,
                             n_candidates=120, n_keep=25, rho=0.2), seed=0)
    X = oracle_matrix(p)
    n2 = oracle.colnorm2(X)
    Xd = dense_array(p)
    corr = np.abs((Xd.T @ Xd) / np.sqrt(np.outer(n2, n2)))
    assert np.allclose(n2, (Xd ** 2).sum(0), rtol=1e-12)
    rng = np.random.default_rng(0)
    saw_full, saw_short = False, False
    for trial in range(30):
        n_keep = [6, 200][trial % 2]
        cand = rng.permutation(300)[:120].astype(np.int32)
        kept, ne, mm = oracle.filter(X, n2, cand, n_keep, p.rho)
        _check_first_fit(corr, cand.tolist(), kept.tolist(), ne, n_keep, p.rho)
        saw_full |= len(kept) == n_keep
        saw_short |= len(kept) < n_keep
        assert 0 < len(kept) < 120                                            # rejections do occur
    assert saw_full and saw_short
    assert abs(oracle.corr(X, n2, 3, 17) - (Xd[:, 3] @ Xd[:, 17]) / np.sqrt(n2[3] * n2[17])) < 1e-14


def test_grouped_design_keeps_one_column_per_group():
    # columns of one group correlate ~0.8, columns of different groups ~N(0, 1/N): with rho = 0.3
    # exactly the first candidate of every group survives
    p = wl.make_problem(dict(kind="dense_grouped", n_rows=2000, n_cols=200, n_true=5, lam_frac=0.1,
                             n_candidates=200, n_keep=200, rho=0.3, group=20), seed=1)
    X = oracle_matrix(p)
    n2 = oracle.colnorm2(X)
    assert 0.7 < oracle.corr(X, n2, 0, 1) < 0.9 and abs(oracle.corr(X, n2, 0, 20)) < 0.15
    cand = np.random.default_rng(1).permutation(200).astype(np.int32)
    kept, ne, mm = oracle.filter(X, n2, cand, 200, p.rho)
    first = {}
    for c in cand.tolist():
        first.setdefault(c // 20, c)
    assert kept.tolist() == [c for c in cand.tolist() if first[c // 20] == c]
    assert ne == 200 and len(kept) == 10


def test_csc_correlations_match_scipy():
    for kind in ("csc_uniform", "csc_zipf"):
        p = wl.make_problem(dict(kind=kind, n_rows=400, n_cols=500, n_true=5, lam_frac=0.1, nnz_col=10,
                                 n_candidates=100, n_keep=40, rho=0.1), seed=2)
        X = oracle_matrix(p)
        n2 = oracle.colnorm2(X)
        S = sp.csc_matrix((p.values.numpy().astype(np.float64), p.row_idx.numpy(), p.col_ptr.numpy()),
                          shape=(p.n_rows, p.n_cols))
        G = (S.T @ S).toarray()
        assert np.allclose(n2, np.diag(G), rtol=1e-12)
        corr = np.abs(G / np.sqrt(np.outer(n2, n2)))
        rng = np.random.default_rng(3)
        for j, k in rng.integers(0, 500, size=(200, 2)):
            assert abs(abs(oracle.corr(X, n2, j, k)) - corr[j, k]) < 1e-13
        cand = rng.permutation(500)[:100].astype(np.int32)
        kept, ne, mm = oracle.filter(X, n2, cand, 40, p.rho)
        _check_first_fit(corr, cand.tolist(), kept.tolist(), ne, 40, p.rho)
        assert np.isfinite(mm)


def test_threshold_is_strict_and_margin_is_reported():
    # two identical directions at a chosen angle: corr = cos(theta)
    N = 8
    e0, e1 = np.zeros(N), np.zeros(N)
    e0[0], e1[1] = 1.0, 1.0
    c = 0.25                                                  # exactly representable
    x2 = c * e0 + np.sqrt(1 - c * c) * e1
    xc = np.stack([e0, x2, e1]).astype(np.float32)
    X = oracle.Matrix.dense(xc)
    n2 = oracle.colnorm2(X)
    corr01 = oracle.corr(X, n2, 0, 1)
    assert abs(corr01 - 0.25) < 1e-7
    cand = np.array([0, 1, 2], dtype=np.int32)
    kept, ne, mm = oracle.filter(X, n2, cand, 3, rho=corr01)             # |corr| == rho: NOT < rho
    assert kept.tolist() == [0, 2] and mm == 0.0
    kept, ne, mm = oracle.filter(X, n2, cand, 3, rho=np.nextafter(corr01, 1.0))
    assert kept.tolist() == [0] or kept.tolist() == [0, 1]               # 1 passes vs 0 ...
    assert 1 in kept.tolist()                                             # ... and then 2 conflicts with 1
    kept, ne, mm = oracle.filter(X, n2, cand, 2, rho=2.0)                # stop at P
    assert kept.tolist() == [0, 1] and ne == 2


def test_follow_mode_only_bends_borderline_decisions():
    N = 8
    e = np.eye(N)
    c = 0.25
    xc = np.stack([e[0], c * e[0] + np.sqrt(1 - c * c) * e[1], e[2]]).astype(np.float32)
    X = oracle.Matrix.dense(xc)
    n2 = oracle.colnorm2(X)
    cand = np.array([0, 1, 2], dtype=np.int32)
    rho = oracle.corr(X, n2, 0, 1) + 5e-7                                 # pair (0,1) within 1e-6 of rho
    assert oracle.filter(X, n2, cand, 3, rho)[0].tolist() == [0, 1, 2]
    # the other implementation rejected 1: the replay follows it on the borderline pair only
    assert oracle.filter(X, n2, cand, 3, rho, follow=[0, 2], tol=1e-6)[0].tolist() == [0, 2]
    assert oracle.filter(X, n2, cand, 3, rho, follow=[0, 1, 2], tol=1e-6)[0].tolist() == [0, 1, 2]
    # a claim that is NOT borderline is not followed
    assert oracle.filter(X, n2, cand, 3, rho, follow=[0], tol=1e-6)[0].tolist() == [0, 2]
    assert oracle.filter(X, n2, cand, 3, 0.1, follow=[0, 1, 2], tol=1e-6)[0].tolist() == [0, 2]
