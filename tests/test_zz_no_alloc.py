"""strads_sample_static: the candidate draw for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is off limits -- inside another framework's memory pool,
or in a loop that must not touch the allocator -- so this entry point keeps its scratch memory in a fixed
array inside the library.  It must give exactly the list the handle-based strads_sample gives, also when
called twice in a row (the array keeps the previous call's contents), and refuse sizes its array cannot
hold.  The list is also compared with the CPU oracle's ranking of all keys.  Collected last on purpose: a run that stops at the first failure has then run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1312_5766_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_static_sampler_matches_the_handle_based_one_twice_in_a_row():
    from paper_1312_5766_b200 import binding as b
    J, n_cand, seed = 300_007, 4096, (7 << 32) | 99
    p = wl.make_problem(dict(kind="csc_uniform", n_rows=64, n_cols=J, n_true=1, lam_frac=0.1, nnz_col=2,
                             n_candidates=n_cand, n_keep=1, rho=0.1), seed=0)
    p.seed = seed
    s = b.StradsLasso.from_problem(p, device="cuda")
    g = torch.Generator(device="cuda").manual_seed(1)
    out = torch.empty(n_cand, dtype=torch.int32, device="cuda")
    for call, t in enumerate([0, 5, (1 << 32) + 3]):
        # a fresh priority vector each time: never-updated, settled and active coefficients mixed
        u = torch.rand(J, generator=g, device="cuda")
        delta = torch.where(u < 0.3, torch.full_like(u, 1e4), torch.where(u < 0.8, torch.zeros_like(u), u))
        s.delta.copy_(delta)
        s.set_round(t)
        want = s.sample().clone()
        got = b.sample_static(delta, p.eta, seed, t, n_cand, out=out)
        assert torch.equal(got, want), (call, t)
        assert np.array_equal(got.cpu().numpy(), oracle.sample(delta.cpu().numpy().astype(np.float64), p.eta, seed, t, n_cand))
        # and again, straight after, on the array the previous call left behind
        got2 = b.sample_static(delta, p.eta, seed, t, n_cand, out=out)
        assert torch.equal(got2, want), (call, t)
    # a smaller request after a larger one, and the refinement path (one bin overflows the key buffer)
    delta = torch.zeros(J, device="cuda")
    delta[1000:200_000] = float("inf")
    s.delta.copy_(delta)
    s.set_round(1)
    want = s.sample()[:300].clone()
    s300 = b.StradsLasso(wl.CSC, p.n_rows, J, p.values.cuda(), p.y.cuda(), p.lam, p.eta, p.rho, 300, 1, seed=seed,
                         row_idx=p.row_idx.cuda(), col_ptr=p.col_ptr.cuda())
    s300.delta.copy_(delta)
    s300.set_round(1)
    want300 = s300.sample().clone()
    assert torch.equal(want300, want)
    got300 = b.sample_static(delta, p.eta, seed, 1, 300)
    assert torch.equal(got300, want300)
    assert np.array_equal(got300.cpu().numpy(), oracle.sample(delta.cpu().numpy().astype(np.float64), p.eta, seed, 1, 300))


def test_static_sampler_rejects_what_its_array_cannot_hold():
    from paper_1312_5766_b200 import binding as b
    delta = torch.ones(100_000, device="cuda")
    with pytest.raises(b.StradsError) as e:
        b.sample_static(delta, 1e-6, 0, 0, b.STATIC_MAX_CANDIDATES + 1)
    assert e.value.code == -7
    with pytest.raises(b.StradsError) as e:
        b.sample_static(delta[:10], 1e-6, 0, 0, 11)
    assert e.value.code == -1
    # the largest allowed size works
    got = b.sample_static(delta, 1e-6, 3, 4, b.STATIC_MAX_CANDIDATES)
    assert np.array_equal(got.cpu().numpy(), oracle.sample(np.ones(100_000), 1e-6, 3, 4, b.STATIC_MAX_CANDIDATES))
