"""The oracle against its own frozen output (tests/golden/oracle_rounds_small.txt, written by
tests/golden/make_golden.py from oracle/ alone): candidate and kept lists exactly, changes and objective to
1e-12 relative.  The paper prints no worked numeric example; the pins that tie the oracle to the paper and the
mathematics are in the other test_oracle_*.py files.  This one makes an unintended change of the oracle's
arithmetic visible."""
import importlib.util
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))


def _load_maker():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_oracle_reproduces_its_frozen_rounds():
    mk = _load_maker()
    with open(mk.OUT) as fh:
        stored = [ln.rstrip("\n") for ln in fh if not ln.startswith("#")]
    fresh = list(mk.lines())
    assert len(stored) == len(fresh) and len(fresh) == 4 * mk.ROUNDS * len(mk.CASES)
    for want, got in zip(stored, fresh):
        w, g = want.split(), got.split()
        assert w[:3] == g[:3]
        if w[2] in ("cand", "kept"):
            assert w[3:] == g[3:], want[:40]
        else:
            a = np.array([float.fromhex(x) for x in w[3:]]); b = np.array([float.fromhex(x) for x in g[3:]])
            assert a.shape == b.shape and np.all(np.abs(a - b) <= 1e-12 * np.maximum(np.abs(a), 1e-300)), want[:40]
    # the frozen rounds are not trivial: candidates full, something kept and moved every round
    for ln in stored:
        f = ln.split()
        if f[2] == "kept":
            assert len(f) > 3


import pytest


@pytest.mark.gpu
@pytest.mark.parametrize("name", ["dense", "csc"])
def test_gpu_first_round_matches_the_frozen_oracle_round(name):
    """Round 0 of the CUDA path (from the same initial state) against the stored oracle round: candidates and
    kept list exactly, changes within the tolerance of the parity tests."""
    import torch
    from paper_1312_5766_b200 import binding, workloads as wl
    mk = _load_maker()
    with open(mk.OUT) as fh:
        stored = {tuple(ln.split()[:3]): ln.split()[3:] for ln in fh if not ln.startswith("#")}
    p = wl.make_problem(mk.CASES[name], seed=7)
    s = binding.StradsLasso.from_problem(p, device="cuda")
    cand, kept, dbeta, counts = s.round()
    nk = int(counts[2])
    assert [str(int(c)) for c in cand.cpu().numpy()] == stored[(name, "0", "cand")]
    assert [str(int(k)) for k in kept.cpu().numpy()[:nk]] == stored[(name, "0", "kept")]
    want = np.array([float.fromhex(x) for x in stored[(name, "0", "dbeta")]])
    got = dbeta.cpu().numpy()[:nk].astype(np.float64)
    assert np.all(np.abs(got - want) <= 1e-5 * np.abs(want) + 1e-7 * max(1.0, float(np.abs(want).max())))
    assert s.status() == (0, 0)
    s.close()
