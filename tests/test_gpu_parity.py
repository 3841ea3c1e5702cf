"""Parity of the CUDA library with the FP64 CPU oracle, element by element, through the C ABI.

Three levels, as the round has three kinds of output:
  1. candidates: bit-exact ordered lists from identical (delta, seed, t);
  2. one round from identical (beta, r, delta): same kept list (decisions within 1e-6 of rho are
     replayed by the oracle and must then agree), dbeta within 1e-5 relative + half an FP32 ulp of the
     coefficient's own new value (the device stores beta in FP32 and reports the change that makes);
  3. free-running objective within 1e-4 relative after a fixed number of rounds.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1312_5766_b200 import workloads as wl
from helpers import oracle_matrix

pytestmark = pytest.mark.gpu

RTOL_DBETA = 1e-5        # relative tolerance on a coefficient change (FP64 accumulation on both sides)
HALF_ULP32 = 2.0 ** -24 * 1.001   # times |beta_j'|: the device's change is fl32(beta_j') - beta_j, the oracle's beta_j' - beta_j
RHO_EXCUSE = 1e-6        # |corr| this close to rho may fall either way (FP32 Gram vs FP64 oracle)
RTOL_OBJ = 1e-4


def _binding():
    from paper_1312_5766_b200 import binding
    return binding


def _solver(p, **kw):
    return _binding().StradsLasso.from_problem(p, device="cuda", **kw)


# --------------------------------------------------------------------------------------------------
# level 1: sampler
# --------------------------------------------------------------------------------------------------
def _delta_cases(J, rng):
    C = 1e4
    sweep = np.full(J, C, dtype=np.float32)
    part = sweep.copy()
    part[rng.random(J) < 0.7] = 0.0
    late = (rng.random(J) < 0.05) * rng.exponential(0.05, J)
    mixed = np.where(rng.random(J) < 0.1, C, late)
    wide = 10.0 ** rng.uniform(-8, 3, J)
    return {"sweep": sweep, "partial_sweep": part, "late": late.astype(np.float32),
            "mixed": mixed.astype(np.float32), "wide": wide.astype(np.float32),
            "zeros": np.zeros(J, dtype=np.float32)}


@pytest.mark.parametrize("J,n_cand", [(10_000, 200), (100_000, 2048), (99_997, 1000), (1_000_003, 8192),
                                      (37, 37), (5, 1), (4096, 4096), (2_000_001, 16384)])
def test_candidates_bit_exact(J, n_cand):
    rng = np.random.default_rng(J)
    p = wl.make_problem(dict(kind="csc_uniform", n_rows=64, n_cols=J, n_true=1, lam_frac=0.1, nnz_col=2,
                             n_candidates=n_cand, n_keep=1, rho=0.1), seed=0)
    cases = _delta_cases(J, rng)
    names = list(cases) if J <= 100_000 else ["sweep", "mixed", "late"]
    for seed, t in [(0, 0), ((0xABCDEF01 << 32) | 0x2345, 7), (42, (1 << 32) + 5)]:
        p.seed = seed
        s = _solver(p)
        s.set_round(t)
        for name in names:
            d = cases[name]
            s.delta.copy_(torch.from_numpy(d))
            got = s.sample().cpu().numpy()
            want = oracle.sample(d.astype(np.float64), p.eta, seed, t, n_cand)
            assert np.array_equal(got, want), (name, seed, t, np.flatnonzero(got != want)[:5])
        assert s.status()[0] == 0
        s.close()


def test_sampler_refinement_path_is_exact():
    # every race time is exactly 0 for the coefficients with infinite priority: one histogram bin
    # holds far more keys than the boundary buffer, so the select must refine down to the index bits
    J, n_cand = 200_000, 300
    p = wl.make_problem(dict(kind="csc_uniform", n_rows=64, n_cols=J, n_true=1, lam_frac=0.1, nnz_col=2,
                             n_candidates=n_cand, n_keep=1, rho=0.1), seed=0)
    d = np.zeros(J, dtype=np.float32)
    d[1000:150_000] = np.inf
    s = _solver(p)
    s.delta.copy_(torch.from_numpy(d))
    got = s.sample().cpu().numpy()
    want = oracle.sample(d.astype(np.float64), p.eta, 0, 0, n_cand)
    assert np.array_equal(got, want) and want.tolist() == list(range(1000, 1300))
    rc, bits = s.status()
    assert rc == 0 and bits & 1                      # informational "refined" bit
    # and the next ordinary draw is unaffected by the detour
    d2 = np.full(J, 1e4, dtype=np.float32)
    s.delta.copy_(torch.from_numpy(d2))
    assert np.array_equal(s.sample().cpu().numpy(), oracle.sample(d2.astype(np.float64), p.eta, 0, 0, n_cand))


def test_guided_first_pass_is_exact_when_the_guide_is_good_bad_or_absent():
    """For J >= 2^19 the sampler's first pass leaves out the keys certainly above four times the previous
    round's boundary and repeats itself in full when too few keys lie below it.  Same candidates as ranking
    all J keys, whatever the previous round was like."""
    J, n_cand = 4_400_000, 1500
    cfg = dict(kind="csc_uniform", n_rows=2000, n_cols=J, n_true=50, lam_frac=0.01, nnz_col=4,
               n_candidates=n_cand, n_keep=64, rho=0.1)
    p = wl.make_problem(cfg, seed=2)
    s = _solver(p)
    rng = np.random.default_rng(4)
    base = np.abs(rng.normal(size=J)).astype(np.float32)
    steps = [("initial C everywhere", None), ("same again: guided", None), ("weights / 1e6: guide far too low", base * 1e-3),
             ("weights x 1e6: guide far too high", base), ("mostly zero changes", np.where(rng.random(J) < 0.99, 0, base).astype(np.float32)),
             ("same again: guided", None)]
    for t, (what, delta) in enumerate(steps):
        if delta is not None:
            s.delta.copy_(torch.from_numpy(delta))
        s.set_round(t)
        got = s.sample().cpu().numpy()
        want = oracle.sample(s.delta.cpu().numpy(), float(np.float32(p.eta)), p.seed, t, n_cand)
        assert np.array_equal(got, want), what
    assert s.status()[0] == 0


def test_uniform_draw_flag_ignores_delta():
    b = _binding()
    J, n_cand = 50_000, 500
    p = wl.make_problem(dict(kind="csc_uniform", n_rows=64, n_cols=J, n_true=1, lam_frac=0.1, nnz_col=2,
                             n_candidates=n_cand, n_keep=1, rho=0.1), seed=3)
    s = _solver(p, flags=b.FLAG_UNIFORM_DRAW)
    s.delta.copy_(torch.rand(J, device="cuda"))
    got = s.sample().cpu().numpy()
    # uniform weights = any constant delta with eta chosen so that w = 1 exactly
    want = oracle.sample(np.ones(J), 0.0, 3, 0, n_cand)
    assert np.array_equal(got, want)


# --------------------------------------------------------------------------------------------------
# init
# --------------------------------------------------------------------------------------------------
def _small_problems():
    return {
        "dense": dict(kind="dense_iid", n_rows=1000, n_cols=3000, n_true=30, lam_frac=0.05,
                      n_candidates=300, n_keep=48, rho=0.1),
        "dense_grouped": dict(kind="dense_grouped", n_rows=2000, n_cols=2000, n_true=20, lam_frac=0.02,
                              n_candidates=400, n_keep=64, rho=0.1, group=20),
        "csc": dict(kind="csc_uniform", n_rows=5000, n_cols=20000, n_true=100, lam_frac=0.01, nnz_col=50,
                    n_candidates=1000, n_keep=128, rho=0.1),
        "csc_zipf": dict(kind="csc_zipf", n_rows=20000, n_cols=50000, n_true=100, lam_frac=0.01, nnz_col=20,
                         n_candidates=1500, n_keep=400, rho=0.05),
    }


@pytest.mark.parametrize("name", list(_small_problems()))
def test_init_state(name):
    p = wl.make_problem(_small_problems()[name], seed=1)
    X = oracle_matrix(p)
    n2, beta, resid, delta = oracle.init(X, p.y.numpy(), 1e4)
    s = _solver(p)
    assert np.allclose(s.colnorm2().cpu().numpy(), n2, rtol=1e-13, atol=0)
    assert np.array_equal(s.resid.cpu().numpy(), p.y.numpy())
    assert np.all(s.delta.cpu().numpy() == np.float32(1e4)) and np.all(s.beta.cpu().numpy() == 0)
    f = s.objective()
    assert abs(f - oracle.objective(resid, beta, p.lam)) < 1e-12 * f
    assert s.get_round() == 0


@pytest.mark.parametrize("name", ["dense", "csc"])
def test_init_from_nonzero_beta(name):
    p = wl.make_problem(_small_problems()[name], seed=2)
    X = oracle_matrix(p)
    b0 = torch.zeros(p.n_cols)
    idx = torch.randperm(p.n_cols, generator=torch.Generator().manual_seed(0))[:40]
    b0[idx] = torch.randn(40, generator=torch.Generator().manual_seed(1))
    s = _solver(p, beta0=b0)
    f_want, r_want = oracle.objective_from_scratch(X, p.y.numpy(), b0.numpy().astype(np.float64), p.lam)
    assert np.allclose(s.resid.cpu().numpy(), r_want, rtol=0, atol=2e-7 * np.abs(r_want).max())
    assert abs(s.objective() - f_want) < 1e-6 * f_want


# --------------------------------------------------------------------------------------------------
# level 2: filter and update from identical state
# --------------------------------------------------------------------------------------------------
def _assert_kept_matches(X, n2, cand, n_keep, rho, got_kept, got_examined):
    want, ne, mm = oracle.filter(X, n2, cand, n_keep, rho)
    if not np.array_equal(got_kept, want):
        assert mm <= RHO_EXCUSE, ("kept differs without a borderline pair", mm)
        want, ne, _ = oracle.filter(X, n2, cand, n_keep, rho, follow=got_kept, tol=RHO_EXCUSE)
        assert np.array_equal(got_kept, want)
    assert got_examined == ne
    return want


@pytest.mark.parametrize("name", list(_small_problems()))
def test_filter_matches_oracle(name):
    cfg = _small_problems()[name]
    p = wl.make_problem(cfg, seed=3)
    X = oracle_matrix(p)
    n2 = oracle.colnorm2(X)
    s = _solver(p)
    rho = float(np.float32(p.rho))
    rng = np.random.default_rng(0)
    rejected = 0
    for trial in range(4):
        n_cand = [p.n_candidates, p.n_candidates, 33, 1][trial]
        cand = rng.permutation(p.n_cols)[:n_cand].astype(np.int32)
        if name == "dense_grouped" and trial == 0:
            cand = np.arange(n_cand, dtype=np.int32)          # whole groups side by side: many rejections
        kept_d, counts_d, gram = s.filter(torch.from_numpy(cand).cuda(), want_gram=True)
        counts = counts_d.cpu().numpy()
        kept = kept_d.cpu().numpy()
        nk = int(counts[2])
        assert np.all(kept[nk:] == -1) and counts[0] == n_cand
        _assert_kept_matches(X, n2, cand, p.n_keep, rho, kept[:nk], int(counts[1]))
        rejected += int(counts[1]) - nk
        # the Gram itself against FP64 dot products on sampled pairs
        g = gram.cpu().numpy()
        for a, b in rng.integers(0, n_cand, size=(300, 2)):
            want = oracle.corr(X, n2, cand[a], cand[b]) * np.sqrt(n2[cand[a]] * n2[cand[b]])
            assert abs(g[a, b] - want) < 2e-6 + 4e-6 * abs(want), (a, b, g[a, b], want)
    if name in ("dense_grouped", "csc_zipf", "dense"):
        assert rejected > 0


CSC_GRAM_CASES = {
    # most pairs share no row: the Gram comes from the row buckets (a few candidates per row)
    "few_per_row": (dict(kind="csc_uniform", n_rows=5000, n_cols=20000, n_true=100, lam_frac=0.01, nnz_col=50,
                         n_candidates=1024, n_keep=128, rho=0.1), [1024, 700, 33, 2]),
    # rows of Zipf frequency hold far more candidates than a bucket does: all pairs instead
    "crowded_rows": (dict(kind="csc_zipf", n_rows=2000, n_cols=30000, n_true=100, lam_frac=0.01, nnz_col=20,
                          n_candidates=1024, n_keep=128, rho=0.1, zipf_a=1.1), [1024, 300]),
    # no bucket overflows (16 candidates in all), but every candidate shares ~40 rows with every other: more terms
    # than one candidate's sort takes, all pairs instead
    "everyone_meets_everyone": (dict(kind="csc_uniform", n_rows=48, n_cols=64, n_true=4, lam_frac=0.01, nnz_col=44,
                                     n_candidates=16, n_keep=8, rho=0.1), [16, 12]),
}


@pytest.mark.parametrize("case", list(CSC_GRAM_CASES))
def test_csc_filter_without_gram_output(case):
    """The filter as the rounds run it (no Gram matrix asked for, so the CSC path may take its inner products from the
    row buckets), on designs that keep to the buckets, overflow them, or collect too many terms for one candidate."""
    cfg, sizes = CSC_GRAM_CASES[case]
    p = wl.make_problem(cfg, seed=5)
    X = oracle_matrix(p)
    n2 = oracle.colnorm2(X)
    s = _solver(p)
    rho = float(np.float32(p.rho))
    rng = np.random.default_rng(1)
    rejected = 0
    for rep in range(3):                                    # (a failed attempt changes what the next call tries first)
        for n_cand in sizes:
            cand = rng.permutation(p.n_cols)[:n_cand].astype(np.int32)
            kept_d, counts_d = s.filter(torch.from_numpy(cand).cuda(), want_gram=False)
            counts = counts_d.cpu().numpy()
            kept = kept_d.cpu().numpy()
            nk = int(counts[2])
            assert np.all(kept[nk:] == -1) and counts[0] == n_cand
            _assert_kept_matches(X, n2, cand, p.n_keep, rho, kept[:nk], int(counts[1]))
            rejected += int(counts[1]) - nk
    assert rejected > 0


@pytest.mark.parametrize("name", list(_small_problems()))
def test_update_matches_oracle(name):
    p = wl.make_problem(_small_problems()[name], seed=4)
    X = oracle_matrix(p)
    s = _solver(p)
    n2, beta, resid, delta = oracle.init(X, p.y.numpy(), 1e4)
    rng = np.random.default_rng(1)
    lam = float(np.float32(p.lam))
    for step in range(6):
        n_kept = [p.n_keep, p.n_keep, 1, 0, p.n_keep // 2, p.n_keep][step]
        kept = rng.permutation(p.n_cols)[:n_kept].astype(np.int32)
        # identical state on both sides
        beta[:] = s.beta.cpu().numpy(); resid[:] = s.resid.cpu().numpy(); delta[:] = s.delta.cpu().numpy()
        d_got = s.update(torch.from_numpy(kept).cuda()).cpu().numpy()
        d_want = oracle.update(X, n2, lam, kept, beta, resid, delta)
        bmax = max(np.abs(beta).max(), 1e-30)
        tol = RTOL_DBETA * np.abs(d_want) + HALF_ULP32 * np.abs(beta[kept])      # (beta now holds the new values)
        assert np.all(np.abs(d_got[:n_kept] - d_want) <= tol)
        assert np.all(d_got[n_kept:] == 0)
        assert np.allclose(s.beta.cpu().numpy(), beta, rtol=0, atol=1.2e-7 * bmax)
        assert np.allclose(s.resid.cpu().numpy(), resid, rtol=0, atol=2e-7 * np.abs(resid).max() + 1e-7 * bmax)
        dl = s.delta.cpu().numpy()
        assert np.all(np.abs(dl[kept] - np.abs(d_want)) <= tol)
        untouched = np.ones(p.n_cols, bool); untouched[kept] = False
        assert np.all(dl[untouched] == delta[untouched].astype(np.float32))
    assert s.get_round() == 0                      # split-phase calls do not advance t


@pytest.mark.parametrize("name", list(_small_problems()))
def test_rounds_teacher_forced(name):
    """Whole rounds; before each one the oracle is given the device's state, so every round is checked
    from identical inputs (candidates exact, kept equal, dbeta within tolerance)."""
    p = wl.make_problem(_small_problems()[name], seed=5)
    X = oracle_matrix(p)
    s = _solver(p)
    n2, beta, resid, delta = oracle.init(X, p.y.numpy(), 1e4)
    lam, eta, rho = float(np.float32(p.lam)), float(np.float32(p.eta)), float(np.float32(p.rho))
    n_rounds = 40
    for t in range(n_rounds):
        beta[:] = s.beta.cpu().numpy(); resid[:] = s.resid.cpu().numpy(); delta[:] = s.delta.cpu().numpy()
        cand_d, kept_d, dbeta_d, counts_d = s.round()
        counts = counts_d.cpu().numpy(); nk = int(counts[2])
        cand = cand_d.cpu().numpy(); kept = kept_d.cpu().numpy()[:nk]; d_got = dbeta_d.cpu().numpy()[:nk]
        want_cand = oracle.sample(delta, eta, p.seed, t, p.n_candidates)
        assert np.array_equal(cand, want_cand), t
        _assert_kept_matches(X, n2, cand, p.n_keep, rho, kept, int(counts[1]))
        d_want = oracle.update(X, n2, lam, kept, beta, resid, delta)
        assert np.all(np.abs(d_got - d_want) <= RTOL_DBETA * np.abs(d_want) + HALF_ULP32 * np.abs(beta[kept])), t
        assert int(counts[3]) == int(np.count_nonzero(d_got))
    assert s.get_round() == n_rounds
    tot = s.totals()
    assert tot["rounds"] == n_rounds and tot["kept"] > 0
    assert s.status() == (0, 0)


# --------------------------------------------------------------------------------------------------
# level 3: free-running objective
# --------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("name,rounds", [("dense", 600), ("csc", 900), ("dense_grouped", 500)])
def test_objective_after_fixed_rounds(name, rounds):
    p = wl.make_problem(_small_problems()[name], seed=6)
    X = oracle_matrix(p)
    n2, beta, resid, delta = oracle.init(X, p.y.numpy(), 1e4)
    lam, eta, rho = float(np.float32(p.lam)), float(np.float32(p.eta)), float(np.float32(p.rho))
    for t in range(rounds):
        oracle.round(X, n2, lam, eta, rho, p.n_candidates, p.n_keep, p.seed, t, beta, resid, delta)
    f_want = oracle.objective(resid, beta, lam)
    s = _solver(p)
    s.run(rounds)
    f_got = s.objective()
    assert abs(f_got - f_want) <= RTOL_OBJ * f_want, (f_got, f_want)
    # the maintained FP32 residual has not drifted from y - X beta
    f_scratch, r_scratch = oracle.objective_from_scratch(X, p.y.numpy(), s.beta.cpu().numpy().astype(np.float64), lam)
    assert abs(f_scratch - f_got) <= 1e-5 * f_want
    assert np.abs(s.resid.cpu().numpy() - r_scratch).max() <= 1e-4 * np.abs(r_scratch).max()


def test_same_seed_gives_identical_bits():
    for name in ("dense", "csc_zipf"):
        p = wl.make_problem(_small_problems()[name], seed=7)
        outs = []
        for rep in range(2):
            s = _solver(p)
            s.run(60)
            outs.append((s.beta.cpu().numpy().copy(), s.resid.cpu().numpy().copy(), s.delta.cpu().numpy().copy()))
        for a, b in zip(*outs):
            assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


def test_round_on_host_state_equals_round_on_device_state():
    p = wl.make_problem(_small_problems()["dense"], seed=8)
    a, b = _solver(p), _solver(p)
    beta_h = torch.zeros(p.n_cols).pin_memory(); resid_h = p.y.clone().pin_memory()
    delta_h = torch.full((p.n_cols,), 1e4).pin_memory()
    kept_h = torch.zeros(p.n_keep, dtype=torch.int32).pin_memory()
    dbeta_h = torch.zeros(p.n_keep).pin_memory(); counts_h = torch.zeros(4, dtype=torch.int32).pin_memory()
    for t in range(5):
        cand, kept, dbeta, counts = a.round()
        b.round_host(beta_h, resid_h, delta_h, kept_h, dbeta_h, counts_h)
        assert torch.equal(kept.cpu(), kept_h) and torch.equal(dbeta.cpu(), dbeta_h) and torch.equal(counts.cpu(), counts_h)
        assert torch.equal(a.beta.cpu(), beta_h) and torch.equal(a.resid.cpu(), resid_h) and torch.equal(a.delta.cpu(), delta_h)


def test_resume_from_saved_state():
    p = wl.make_problem(_small_problems()["csc"], seed=9)
    a = _solver(p)
    a.run(10)
    saved = (a.beta.clone(), a.resid.clone(), a.delta.clone(), a.get_round())
    a.run(10)
    b = _solver(p)
    b.beta.copy_(saved[0]); b.resid.copy_(saved[1]); b.delta.copy_(saved[2]); b.set_round(saved[3])
    b.run(10)
    assert torch.equal(a.beta, b.beta) and torch.equal(a.resid, b.resid) and torch.equal(a.delta, b.delta)


def test_no_filter_flag_keeps_first_candidates():
    b = _binding()
    p = wl.make_problem(_small_problems()["dense_grouped"], seed=10)
    s = _solver(p, flags=b.FLAG_NO_FILTER)
    cand, kept, dbeta, counts = s.round()
    assert torch.equal(kept, cand[: p.n_keep]) and counts.cpu().tolist()[1:3] == [p.n_keep, p.n_keep]


def test_ragged_rows_and_padding():
    # N not a multiple of 4 or of any tile, ld > N with NaN in the padding: nothing may leak in
    cfg = dict(kind="dense_iid", n_rows=1003, n_cols=777, n_true=10, lam_frac=0.05, n_candidates=131, n_keep=19,
               rho=0.1)
    p = wl.make_problem(cfg, seed=11)
    ld = 1008
    vals = torch.full((p.n_cols, ld), float("nan"))
    vals[:, : p.n_rows] = p.values
    b = _binding()
    s = b.StradsLasso(wl.DENSE, p.n_rows, p.n_cols, vals.cuda(), p.y.cuda(), p.lam, p.eta, p.rho, p.n_candidates,
                      p.n_keep, seed=p.seed)
    X = oracle_matrix(p)
    n2, beta, resid, delta = oracle.init(X, p.y.numpy(), 1e4)
    lam, eta, rho = float(np.float32(p.lam)), float(np.float32(p.eta)), float(np.float32(p.rho))
    assert np.allclose(s.colnorm2().cpu().numpy(), n2, rtol=1e-13)
    for t in range(12):
        beta[:] = s.beta.cpu().numpy(); resid[:] = s.resid.cpu().numpy(); delta[:] = s.delta.cpu().numpy()
        cand_d, kept_d, dbeta_d, counts_d = s.round()
        counts = counts_d.cpu().numpy(); nk = int(counts[2])
        cand = cand_d.cpu().numpy(); kept = kept_d.cpu().numpy()[:nk]
        assert np.array_equal(cand, oracle.sample(delta, eta, p.seed, t, p.n_candidates))
        _assert_kept_matches(X, n2, cand, p.n_keep, rho, kept, int(counts[1]))
        d_want = oracle.update(X, n2, lam, kept, beta, resid, delta)
        assert np.all(np.abs(dbeta_d.cpu().numpy()[:nk] - d_want) <= RTOL_DBETA * np.abs(d_want) + HALF_ULP32 * np.abs(beta[kept]))
    assert torch.isfinite(s.resid).all() and s.status() == (0, 0)


def test_degenerate_sizes():
    # P' = P = J = 1 and a single row
    b = _binding()
    vals = torch.tensor([[2.0, 0.0, 0.0, 0.0]]).cuda()
    y = torch.tensor([3.0]).cuda()
    s = b.StradsLasso(wl.DENSE, 1, 1, vals, y, lam=1.0, eta=1e-6, rho=0.1, n_candidates=1, n_keep=1)
    cand, kept, dbeta, counts = s.round()
    # n = 4, g = 6: beta = S(6/4, 1/4) = 1.25, r = 3 - 2*1.25 = 0.5
    assert cand.tolist() == [0] and kept.tolist() == [0] and abs(float(dbeta[0]) - 1.25) < 1e-7
    assert abs(float(s.resid[0]) - 0.5) < 1e-7 and abs(s.objective() - (0.125 + 1.25)) < 1e-7
    # an all-zero column never moves and never conflicts
    vals = torch.zeros((3, 8)); vals[1, :4] = 0.5
    s = b.StradsLasso(wl.DENSE, 8, 3, vals.cuda(), torch.ones(8).cuda(), lam=0.1, eta=1e-6, rho=0.1,
                      n_candidates=3, n_keep=3)
    cand, kept, dbeta, counts = s.round()
    assert counts.cpu().tolist() == [3, 3, 3, 1] and sorted(kept.tolist()) == [0, 1, 2]
    assert s.beta.cpu().tolist()[0] == 0.0 and s.beta.cpu().tolist()[2] == 0.0 and s.status() == (0, 0)


# --------------------------------------------------------------------------------------------------
# tensor-core Gram (3xTF32, tcgen05) against the oracle and against the FP32 SIMT kernel
# --------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("cfg", [
    dict(kind="dense_iid", n_rows=1000, n_cols=3000, n_true=30, lam_frac=0.05, n_candidates=300, n_keep=300, rho=0.1),
    dict(kind="dense_grouped", n_rows=2000, n_cols=2000, n_true=20, lam_frac=0.02, n_candidates=640, n_keep=640,
         rho=0.1, group=20),
    dict(kind="dense_iid", n_rows=1003, n_cols=900, n_true=10, lam_frac=0.05, n_candidates=131, n_keep=131, rho=0.05),
    dict(kind="dense_iid", n_rows=24, n_cols=600, n_true=5, lam_frac=0.05, n_candidates=513, n_keep=513, rho=0.3),
])
def test_tensor_core_gram_decisions(cfg):
    b = _binding()
    p = wl.make_problem(cfg, seed=12)
    ld = (p.n_rows + 3) // 4 * 4
    vals = torch.full((p.n_cols, ld), float("nan"))
    vals[:, : p.n_rows] = p.values
    X = oracle_matrix(p)
    n2 = oracle.colnorm2(X)
    rho = float(np.float32(p.rho))
    mk = lambda flags: b.StradsLasso(wl.DENSE, p.n_rows, p.n_cols, vals.cuda(), p.y.cuda(), p.lam, p.eta, p.rho,
                                     p.n_candidates, p.n_keep, seed=p.seed, flags=flags)
    tc, simt, tc3 = mk(0), mk(b.FLAG_SIMT_GRAM), mk(b.FLAG_GRAM_3XTF32)
    rng = np.random.default_rng(5)
    for trial in range(3):
        cand = rng.permutation(p.n_cols)[: p.n_candidates].astype(np.int32)
        if cfg["kind"] == "dense_grouped" and trial == 0:
            cand = np.arange(p.n_candidates, dtype=np.int32)
        cd = torch.from_numpy(cand).cuda()
        kept_tc, counts_tc = tc.filter(cd)
        c = counts_tc.cpu().numpy(); nk = int(c[2])
        _assert_kept_matches(X, n2, cand, p.n_keep, rho, kept_tc.cpu().numpy()[:nk], int(c[1]))
        kept_s, counts_s = simt.filter(cd)
        assert torch.equal(kept_tc, kept_s) and torch.equal(counts_tc, counts_s)
        kept_3, counts_3 = tc3.filter(cd)
        assert torch.equal(kept_tc, kept_3) and torch.equal(counts_tc, counts_3)
    assert tc.status() == (0, 0) and tc3.status() == (0, 0)


@pytest.mark.parametrize("J,n_keep", [(1536, 64), (4096, 800)])
def test_tensor_core_screen_overflow_falls_back_to_3xtf32(J, n_keep):
    # every pair correlates at ~rho: x_j = sqrt(rho) z + sqrt(1 - rho) e_j, so hundreds of thousands of pairs
    # fall inside the screen's "too close to call" band and its list overflows -- in the whole-list Gram of the
    # retry (first case) or already in the candidate window, which then hands over to the retry (second case)
    b = _binding()
    N, rho = 12_000, 0.25
    g = torch.Generator().manual_seed(3)
    z = torch.randn(N, generator=g)
    x = (rho ** 0.5) * z[None, :] + ((1 - rho) ** 0.5) * torch.randn((J, N), generator=g)
    x -= x.mean(dim=1, keepdim=True)
    x /= x.norm(dim=1, keepdim=True)
    y = torch.randn(N, generator=g)
    mk = lambda flags: b.StradsLasso(wl.DENSE, N, J, x.cuda(), y.cuda(), 0.1, 1e-6, rho, J, n_keep, seed=0, flags=flags)
    tc, simt = mk(0), mk(b.FLAG_SIMT_GRAM)
    cand = torch.randperm(J, generator=g).to(torch.int32).cuda()
    kept_tc, counts_tc = tc.filter(cand)
    kept_s, counts_s = simt.filter(cand)
    X = oracle.Matrix.dense(x.numpy())
    n2 = oracle.colnorm2(X)
    c = counts_tc.cpu().numpy(); nk = int(c[2])
    _assert_kept_matches(X, n2, cand.cpu().numpy(), n_keep, float(np.float32(rho)), kept_tc.cpu().numpy()[:nk], int(c[1]))
    # the two FP32-accurate kernels may differ only on pairs within 1e-6 of rho; on this data they agree
    assert torch.equal(kept_tc, kept_s) and torch.equal(counts_tc, counts_s)
    assert tc.status() == (0, 8)                     # informational bit: the fallback did run


# --------------------------------------------------------------------------------------------------
# candidate window: the default (window first, whole list only if the walk runs out) against the
# whole-list Gram, on data where the window suffices and on data where it does not
# --------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("name,n_keep", [("dense", 24), ("dense_grouped", 24), ("dense_grouped", 120), ("csc", 100),
                                         ("csc_zipf", 60), ("csc_zipf", 300)])
def test_window_equals_full_gram(name, n_keep):
    b = _binding()
    cfg = dict(_small_problems()[name], n_keep=n_keep)
    cfg["n_candidates"] = 1024 if "dense" in name else cfg["n_candidates"]
    p = wl.make_problem(cfg, seed=13)
    X = oracle_matrix(p)
    n2 = oracle.colnorm2(X)
    rho = float(np.float32(p.rho))
    lazy, full = _solver(p), _solver(p, flags=b.FLAG_FULL_GRAM)
    rng = np.random.default_rng(6)
    shorts = 0
    for trial in range(4):
        cand = rng.permutation(p.n_cols)[: p.n_candidates].astype(np.int32)
        if name == "dense_grouped" and trial % 2 == 0:
            cand = np.arange(p.n_candidates, dtype=np.int32)       # whole groups side by side: the window runs short
        cd = torch.from_numpy(cand).cuda()
        kept_l, counts_l = lazy.filter(cd)
        kept_f, counts_f = full.filter(cd)
        assert torch.equal(kept_l, kept_f) and torch.equal(counts_l, counts_f), (name, trial)
        c = counts_l.cpu().numpy(); nk = int(c[2])
        _assert_kept_matches(X, n2, cand, p.n_keep, rho, kept_l.cpu().numpy()[:nk], int(c[1]))
        shorts += nk < p.n_keep
    if (name, n_keep) in (("dense_grouped", 120), ("csc_zipf", 300)):
        assert shorts > 0                        # these did exercise the whole-list retry
    assert lazy.status()[0] == 0


@pytest.mark.parametrize("name,n_keep,n_cand", [("dense", 24, 1024), ("dense_grouped", 120, 1024), ("dense_grouped", 40, 1024),
                                                ("csc", 100, 1000), ("csc_zipf", 300, 1500)])
def test_graph_replay_equals_round_by_round(name, n_keep, n_cand):
    """strads_run replays a captured round in which the whole-list retry and its 3xTF32 fallback are launches
    that return at once unless the window was too short; the state it leaves must be bit-identical to calling
    strads_round the same number of times."""
    cfg = dict(_small_problems()[name], n_keep=n_keep, n_candidates=n_cand)
    p = wl.make_problem(cfg, seed=14)
    a, b = _solver(p), _solver(p)
    n = 70                                            # crosses round 64, where a skipped window is tried again
    a.run(n)
    kept_total = 0
    for _ in range(n):
        kept_total += int(b.round()[3][2])
    assert a.get_round() == b.get_round() == n
    for x, y in ((a.beta, b.beta), (a.resid, b.resid), (a.delta, b.delta)):
        assert torch.equal(x, y)
    assert a.totals() == b.totals() and a.totals()["kept"] == kept_total
    assert a.status()[0] == 0 and b.status()[0] == 0


# --------------------------------------------------------------------------------------------------
# sampling ahead: strads_run (one scheduler) draws the candidates of round t + 1 during round t and corrects the
# list for the coefficients round t updates.  The result must be the list a draw made at the round's start
# gives: state after mixed sequences of strads_run and other calls == the same rounds one by one (strads_round
# draws at the round's start and is itself checked against the oracle above).
# --------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("name,cfg_over,flags", [
    ("dense", dict(n_cols=1500, n_candidates=256, n_keep=64), 0),          # the first sweep ends after ~24 rounds
    ("dense", dict(n_cols=300, n_candidates=256, n_keep=64), 0),           # P' + P > J: the early list is everything
    ("dense_grouped", dict(n_candidates=512, n_keep=120), 0),              # heavy rejection, whole-list retries
    ("csc", dict(n_cols=6000, n_candidates=1000, n_keep=128), 0),
    ("csc_zipf", dict(), 0),
    ("dense", dict(n_cols=1500, n_candidates=256, n_keep=64), "uniform"),
])
def test_sampling_ahead_equals_round_by_round(name, cfg_over, flags):
    b = _binding()
    cfg = dict(_small_problems()[name], **cfg_over)
    cfg["n_true"] = min(cfg["n_true"], cfg["n_cols"] // 10)
    p = wl.make_problem(cfg, seed=21)
    kw = dict(flags=b.FLAG_UNIFORM_DRAW) if flags == "uniform" else {}
    a, ref = _solver(p, **kw), _solver(p, **kw)
    done = 0

    def check():
        assert a.get_round() == ref.get_round() == done
        for x, y in ((a.beta, ref.beta), (a.resid, ref.resid), (a.delta, ref.delta)):
            assert torch.equal(x, y), (name, done)

    # runs of several lengths; between them calls that leave the early list stale or unusable
    # (strads_run replays sequences of 8 rounds and, for what is left over, of 4, 2 and 1: 7 = 4 + 2 + 1 from a list in place)
    for step in (3, 1, 40, "round", 2, "filter", 25, "set_round", 30, "round_host", 12, 7):
        if step == "round":
            a.round(); n = 1
        elif step == "filter":
            a.filter(torch.arange(p.n_candidates, dtype=torch.int32, device="cuda")); n = 0   # overwrites kept / counts
        elif step == "set_round":
            a.set_round(done); n = 0
        elif step == "round_host":
            hb, hr, hd = (t.cpu().pin_memory() for t in (a.beta, a.resid, a.delta))
            a.round_host(hb, hr, hd); n = 1
        else:
            a.run(step); n = step
        for _ in range(n):
            ref.round()
        done += n
        check()
    assert a.totals() == ref.totals()
    assert a.status()[0] == 0 and ref.status()[0] == 0


# --------------------------------------------------------------------------------------------------
# short columns: correlations scatter widely around rho, so the BF16 screen leaves many pairs open.  With few
# of them the last CTA of the split-K reduce kernel rechecks them itself; beyond its budget the window is handed
# to the whole-list retry, whose Gram has a recheck kernel (and, past its list, the 3xTF32 fallback).  Every path
# must give the decisions of an exact Gram.
# --------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("n_rows,n_keep", [(64, 64), (64, 256), (300, 256), (24, 256)])
def test_many_open_pairs_in_the_window(n_rows, n_keep):
    b = _binding()
    cfg = dict(kind="dense_iid", n_rows=n_rows, n_cols=4000, n_true=8, lam_frac=0.05, n_candidates=1024,
               n_keep=n_keep, rho=0.1)
    p = wl.make_problem(cfg, seed=17)
    X = oracle_matrix(p)
    n2 = oracle.colnorm2(X)
    rho = float(np.float32(p.rho))
    lazy, full = _solver(p), _solver(p, flags=b.FLAG_FULL_GRAM)
    rng = np.random.default_rng(8)
    for trial in range(3):
        cand = rng.permutation(p.n_cols)[: p.n_candidates].astype(np.int32)
        cd = torch.from_numpy(cand).cuda()
        kept_l, counts_l = lazy.filter(cd)
        kept_f, counts_f = full.filter(cd)
        assert torch.equal(kept_l, kept_f) and torch.equal(counts_l, counts_f), (n_rows, n_keep, trial)
        c = counts_l.cpu().numpy(); nk = int(c[2])
        _assert_kept_matches(X, n2, cand, p.n_keep, rho, kept_l.cpu().numpy()[:nk], int(c[1]))
    assert lazy.status()[0] == 0 and full.status()[0] == 0
    # and whole rounds through strads_run equal rounds one by one on such data too
    a, ref = _solver(p), _solver(p)
    a.run(20)
    for _ in range(20):
        ref.round()
    for x, y in ((a.beta, ref.beta), (a.resid, ref.resid), (a.delta, ref.delta)):
        assert torch.equal(x, y)


# --------------------------------------------------------------------------------------------------
# x_c^T r of the default dense round is accumulated in pairs of floats (exact product and sum errors kept
# in a low word) while the candidate columns stream through the pack kernel.  Adversarial cancellation: r is
# orthogonal to every column up to its own FP32 rounding, so x_c^T r is ~1e-8 of sum |x_i r_i|; the result
# must stay within 2^-44 of that sum of magnitudes (four times the pair arithmetic's bound), which plain
# FP32 accumulation misses by orders of magnitude.
# --------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("n_rows", [4096, 4093])
def test_inner_products_survive_cancellation(n_rows):
    b = _binding()
    J = 256
    p = wl.make_problem(dict(kind="dense_iid", n_rows=n_rows, n_cols=J, n_true=4, lam_frac=0.05, n_candidates=J,
                             n_keep=J, rho=0.9), seed=19)
    X64 = p.values.numpy().astype(np.float64)[:, :n_rows]                  # [J, N]: row j is column x_j
    z = np.random.default_rng(2).normal(size=n_rows)
    coef = np.linalg.solve(X64 @ X64.T, X64 @ z)
    r = z - X64.T @ coef                                                   # orthogonal to all J columns
    y = torch.from_numpy((1e3 * r / np.abs(r).max()).astype(np.float32))
    vals = torch.full((J, (n_rows + 3) // 4 * 4), float("nan"))           # ld a multiple of 4, padding must not leak in
    vals[:, :n_rows] = p.values
    s = b.StradsLasso(wl.DENSE, n_rows, J, vals.cuda(), y.cuda(), 0.0, p.eta, p.rho, J, J, seed=5)
    cand, kept, dbeta, counts = s.round()
    nk = int(counts[2])
    assert nk > J // 2
    kept = kept.cpu().numpy()[:nk]; d_got = dbeta.cpu().numpy()[:nk].astype(np.float64)
    y64 = y.numpy().astype(np.float64)
    n2 = (X64 * X64).sum(axis=1)
    g_want = X64[kept] @ y64                                               # lambda = 0, beta = 0: dbeta = fl32(g / n)
    mag = np.abs(X64[kept]) @ np.abs(y64)
    assert np.median(np.abs(g_want) / mag) < 1e-6                          # the cancellation is there
    bound = 2.0 ** -44 * mag / n2[kept] + 2.0 ** -23 * np.abs(g_want / n2[kept])
    assert np.all(np.abs(d_got - g_want / n2[kept]) <= bound), np.max(np.abs(d_got - g_want / n2[kept]) / bound)
    # the test has teeth: the same sums accumulated in FP32 miss the bound
    g32 = np.array([np.cumsum(p.values.numpy()[j, :n_rows] * y.numpy(), dtype=np.float32)[-1] for j in kept], dtype=np.float64)
    assert np.mean(np.abs(g32 - g_want) / n2[kept] > bound) > 0.9
    assert s.status() == (0, 0)


def test_state_written_by_the_caller_between_runs():
    """strads_run keeps a list drawn ahead for its next round; a caller who rewrites the priorities between two
    runs calls strads_set_round (the header's rule), after which the rounds are those of the new state."""
    cfg = dict(_small_problems()["dense"], n_cols=1500, n_candidates=256, n_keep=64)
    p = wl.make_problem(cfg, seed=23)
    a, ref = _solver(p), _solver(p)
    a.run(30)
    for _ in range(30):
        ref.round()
    g = torch.Generator(device="cuda").manual_seed(5)
    new_delta = torch.rand(p.n_cols, generator=g, device="cuda") ** 4
    a.delta.copy_(new_delta); ref.delta.copy_(new_delta)
    a.set_round(30)                                   # same index: only discards the list drawn from the old priorities
    a.run(25)
    for _ in range(25):
        ref.round()
    for x, y in ((a.beta, ref.beta), (a.resid, ref.resid), (a.delta, ref.delta)):
        assert torch.equal(x, y)
    assert a.get_round() == ref.get_round() == 55


@pytest.mark.parametrize("name", ["csc", "csc_zipf"])
def test_csc_residual_update_is_exact_to_fp32_rounding(name):
    """CSC residual update: contributions are added as 64-bit fixed-point integers (unit 2^-(61 - e), 2^e above the
    largest possible row sum), so what reaches a row is the exact sum to ~2^-60 of that bound, whatever the order of
    the additions -- hot rows of the Zipf design collect hundreds of terms.  The new residual must therefore be the
    FP32 rounding of the exact one: equal to it, or one ulp off where the exact value sits on a rounding boundary."""
    p = wl.make_problem(_small_problems()[name], seed=61)
    s = _solver(p)
    v, r_idx, cp = p.values.numpy().astype(np.float64), p.row_idx.numpy(), p.col_ptr.numpy()
    rng = np.random.default_rng(3)
    for step in range(4):
        s.run(3)                                            # some state with non-trivial beta
        kept = rng.permutation(p.n_cols)[: p.n_keep].astype(np.int32)
        b_old = s.beta.cpu().numpy().astype(np.float64)
        r_old = s.resid.cpu().numpy().astype(np.float64)
        s.update(torch.from_numpy(kept).cuda())
        d = s.beta.cpu().numpy().astype(np.float64) - b_old                  # the changes, exactly (differences of floats)
        assert np.count_nonzero(d) > p.n_keep // 4 and not d[np.setdiff1d(np.arange(p.n_cols), kept)].any()
        moved = np.zeros(p.n_rows)
        for j in np.flatnonzero(d):
            np.add.at(moved, r_idx[cp[j]:cp[j + 1]], v[cp[j]:cp[j + 1]] * d[j])
        want = (r_old - moved).astype(np.float32)
        got = s.resid.cpu().numpy()
        ulp = np.spacing(np.abs(want).astype(np.float32))
        assert np.all(np.abs(got.astype(np.float64) - want.astype(np.float64)) <= ulp)
        assert np.mean(got != want) < 1e-3                  # (ties of the last bit only)
    assert s.status() == (0, 0)


# --------------------------------------------------------------------------------------------------
# The walk from the list of conflicting pairs settles first-fit in passes, one per link of the longest chain of
# decisions that depend on each other, and hands over to the walk over the bit rows past 24 passes.  Columns
# c_k = (z_k + z_{k+1}) / sqrt(2) with orthonormal z make such chains: neighbours correlate at 0.5, everybody else at
# 0.  In list order k = 0, 1, 2, ... every decision waits for the one before it (one chain as long as the list: the
# hand-over); in random order the chains are short; blocks of a few neighbours give chains of every length below the
# limit.  Every case must give the oracle's kept list, stop at P included.
# --------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("n_links,n_keep", [(200, 200), (200, 37), (700, 512)])
def test_walk_settles_chains_of_dependent_decisions(n_links, n_keep):
    b = _binding()
    rng = np.random.default_rng(31)
    n_rows = ((n_links + 1 + 63) // 64) * 64
    z, _ = np.linalg.qr(rng.normal(size=(n_rows, n_links + 1)))
    cols = ((z[:, :-1] + z[:, 1:]) / np.sqrt(2.0)).T.astype(np.float32)          # [J, N]: row k is column c_k
    y = torch.from_numpy(rng.normal(size=n_rows).astype(np.float32))
    J = n_links
    s = b.StradsLasso(wl.DENSE, n_rows, J, torch.from_numpy(cols).contiguous().cuda(), y.cuda(), 0.01, 1e-6, 0.1, J, n_keep, seed=3)
    X = oracle.Matrix.dense(cols, n_rows=n_rows)
    n2 = oracle.colnorm2(X)
    rho = float(np.float32(0.1))
    # blocks of 2 .. 30 consecutive links, the blocks shuffled: chains of every length up to the pass limit and past it
    blocks, at = [], 0
    while at < J:
        n = int(rng.integers(2, 31))
        blocks.append(np.arange(at, min(at + n, J)))
        at += n
    orders = {
        "in_order": np.arange(J),
        "reversed": np.arange(J)[::-1].copy(),
        "random": rng.permutation(J),
        "blocks": np.concatenate([blocks[i] for i in rng.permutation(len(blocks))]),
    }
    for name, order in orders.items():
        cand = order.astype(np.int32)[:J]
        kept_d, counts_d = s.filter(torch.from_numpy(cand).cuda())
        c = counts_d.cpu().numpy(); nk = int(c[2])
        want = _assert_kept_matches(X, n2, cand, n_keep, rho, kept_d.cpu().numpy()[:nk], int(c[1]))
        assert nk == len(want) and (nk == n_keep or int(c[1]) == J), name
        if name == "in_order" and n_keep >= J:
            assert nk == (J + 1) // 2                       # every other link
    assert s.status()[0] == 0
    # whole rounds (candidate window, walk by the Gram kernel's last CTA, retry) against rounds one by one
    a, ref = (b.StradsLasso(wl.DENSE, n_rows, J, torch.from_numpy(cols).contiguous().cuda(), y.cuda(), 0.01, 1e-6, 0.1,
                            J, min(n_keep, J // 4), seed=3) for _ in range(2))
    a.run(12)
    for _ in range(12):
        ref.round()
    for u, v in ((a.beta, ref.beta), (a.resid, ref.resid), (a.delta, ref.delta)):
        assert torch.equal(u, v)
