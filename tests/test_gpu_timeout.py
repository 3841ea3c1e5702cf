"""A bounded device-side wait that does run out: the launch returns, strads_status reports
STRADS_ERR_TIMEOUT, and after strads_recover the same handle works again.

Nothing here faults or hangs: with a limit of a few thousand iterations in force, strads_inject_stall makes
the next wait expire (an arrival counter no barrier completes from; operand loads that are withheld), and the
kernels' own expiry path does the rest -- raise the status bit, stop issuing work, free tensor memory, return.
"""
import numpy as np
import pytest
import torch

from paper_1312_5766_b200 import workloads as wl

pytestmark = pytest.mark.gpu

ERR_INVALID_ARG, ERR_TIMEOUT, WAIT_EXPIRED = -1, -6, 4


def _binding():
    from paper_1312_5766_b200 import binding
    return binding


def test_stall_is_refused_without_a_short_limit():
    b = _binding()
    p = wl.make_problem(dict(kind="dense_iid", n_rows=256, n_cols=512, n_true=4, lam_frac=0.05, n_candidates=128,
                             n_keep=16, rho=0.1), seed=0)
    s = b.StradsLasso.from_problem(p, device="cuda")
    for limit in (0, 1 << 20):
        s.set_wait_limit(limit)
        with pytest.raises(b.StradsError) as e:
            s.inject_stall(b.STALL_GRAM_LOADS)
        assert e.value.code == ERR_INVALID_ARG
    s.set_wait_limit(4096)
    with pytest.raises(b.StradsError):
        s.inject_stall(b.STALL_WALK_BARRIER)          # a dense problem has no walk barrier
    s.round()
    assert s.status() == (0, 0)


def test_csc_walk_barrier_gives_up_and_the_handle_recovers():
    b = _binding()
    # skewed rows: most candidate pairs conflict, so the window runs short and the whole list is walked on demand
    cfg = dict(kind="csc_zipf", n_rows=20000, n_cols=50000, n_true=100, lam_frac=0.01, nnz_col=20,
               n_candidates=1500, n_keep=300, rho=0.05)
    p = wl.make_problem(cfg, seed=13)
    cand = torch.from_numpy(np.random.default_rng(6).permutation(p.n_cols)[: p.n_candidates].astype(np.int32)).cuda()
    ref = b.StradsLasso.from_problem(p, device="cuda")
    kept_want, counts_want = (t.clone() for t in ref.filter(cand))
    assert int(counts_want[2]) < p.n_keep                                   # the walk did go over the whole list

    s = b.StradsLasso.from_problem(p, device="cuda")
    s.set_wait_limit(4096)
    s.inject_stall(b.STALL_WALK_BARRIER)
    s.filter(cand)                                                          # returns: every CTA's wait gives up
    rc, bits = s.status()
    assert rc == ERR_TIMEOUT and bits & WAIT_EXPIRED
    s.filter(cand)                                                          # still flagged; the walk stays out
    assert s.status()[0] == ERR_TIMEOUT
    s.recover()
    assert s.status() == (0, 0)
    kept, counts = s.filter(cand)
    assert torch.equal(kept, kept_want) and torch.equal(counts, counts_want)
    # whole rounds afterwards equal those of a handle that never saw the stall
    s.set_wait_limit(0)
    s.run(12); ref.run(12)
    for x, y in ((s.beta, ref.beta), (s.resid, ref.resid), (s.delta, ref.delta)):
        assert torch.equal(x, y)
    assert s.status()[0] == 0


def test_dense_gram_pipeline_gives_up_and_the_handle_recovers():
    b = _binding()
    cfg = dict(kind="dense_grouped", n_rows=2000, n_cols=2000, n_true=20, lam_frac=0.02, n_candidates=640, n_keep=64,
               rho=0.1, group=20)
    p = wl.make_problem(cfg, seed=3)
    cand = torch.arange(p.n_candidates, dtype=torch.int32, device="cuda")
    ref = b.StradsLasso.from_problem(p, device="cuda")
    kept_want, counts_want = (t.clone() for t in ref.filter(cand))

    s = b.StradsLasso.from_problem(p, device="cuda")
    saved = (s.beta.clone(), s.resid.clone(), s.delta.clone())
    s.set_wait_limit(2048)
    s.inject_stall(b.STALL_GRAM_LOADS)
    s.filter(cand)                                   # the MMA warp's wait for operands runs out in every CTA
    rc, bits = s.status()
    assert rc == ERR_TIMEOUT and bits & WAIT_EXPIRED
    s.run(3)                                         # rounds on a stalled handle also end, flagged
    assert s.status()[0] == ERR_TIMEOUT
    # recovery as the header prescribes: state from the caller's copy, recover, round index
    s.beta.copy_(saved[0]); s.resid.copy_(saved[1]); s.delta.copy_(saved[2])
    s.recover()
    s.set_round(0)
    assert s.status() == (0, 0)
    kept, counts = s.filter(cand)
    assert torch.equal(kept, kept_want) and torch.equal(counts, counts_want)
    s.set_wait_limit(0)
    s.run(20); ref.run(20)
    for x, y in ((s.beta, ref.beta), (s.resid, ref.resid), (s.delta, ref.delta)):
        assert torch.equal(x, y)
    assert s.status()[0] == 0 and s.get_round() == 20
