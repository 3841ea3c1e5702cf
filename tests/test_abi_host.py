"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the header
declares, and rejects bad arguments before anything is launched."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_1312_5766_b200 import build, binding
    build.build()
    return binding.load()


def _declared():
    text = open(os.path.join(ROOT, "include", "strads.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(strads_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_1312_5766_b200 import binding
    names = _declared()
    assert len(names) >= 19
    for n in names:
        assert hasattr(lib, n), n
    assert set(binding.EXPORTS) <= set(names)


def test_error_strings(lib):
    assert lib.strads_error_string(0) == b"ok"
    for code in range(-7, 0):
        assert lib.strads_error_string(code) not in (b"ok", b"unknown error")
    assert lib.strads_error_string(-99) == b"unknown error"


def test_workspace_query_and_size_checks(lib):
    from paper_1312_5766_b200 import binding as b
    assert b.workspace_bytes(0, 10_000, 100_000, 2048, 256) > 8 * 100_000
    bad = [dict(layout=7), dict(n_rows=0), dict(n_cols=0), dict(ld=999), dict(ld=1002), dict(n_candidates=0),
           dict(n_candidates=200_000), dict(n_keep=0), dict(n_keep=3000), dict(n_cols=2**31)]
    for kw in bad:
        cfg = b.Config()
        cfg.layout, cfg.n_rows, cfg.n_cols, cfg.ld, cfg.n_candidates, cfg.n_keep = 0, 1000, 100_000, 1000, 2048, 256
        for k, v in kw.items():
            setattr(cfg, k, v)
        out = C.c_size_t(0)
        assert lib.strads_workspace_bytes(C.byref(cfg), C.byref(out)) < 0, kw
    cfg = b.Config()
    cfg.layout, cfg.n_rows, cfg.n_cols, cfg.ld, cfg.n_candidates, cfg.n_keep = 0, 1000, 100_000, 1000, 20_000, 256
    out = C.c_size_t(0)
    assert lib.strads_workspace_bytes(C.byref(cfg), C.byref(out)) == -7          # beyond STRADS_MAX_CANDIDATES
    assert lib.strads_workspace_bytes(None, C.byref(out)) == -1
    assert lib.strads_workspace_bytes(C.byref(cfg), None) == -1
    # scheduler threads: every one has its own slice (the column norms are shared), S and P' <= J / S are checked
    sizes = []
    for S in (0, 1, 2, 4):
        cfg = b.Config()
        cfg.layout, cfg.n_rows, cfg.n_cols, cfg.ld, cfg.n_candidates, cfg.n_keep = 0, 1000, 100_000, 1000, 2048, 256
        cfg.n_schedulers = S
        assert lib.strads_workspace_bytes(C.byref(cfg), C.byref(out)) == 0
        sizes.append(out.value)
    assert sizes[0] == sizes[1] < sizes[2] < sizes[3]
    # a further scheduler's slice (no column norms); the one-scheduler layout also holds the buffers of the early draw
    rest = (sizes[3] - sizes[2]) // 2
    assert sizes[3] - sizes[2] == 2 * rest and sizes[2] - sizes[1] <= rest < sizes[1] - 8 * 100_000 + 4096
    assert rest - (sizes[2] - sizes[1]) < 256 * 1024
    for S, n_cand in ((-1, 2048), (9, 2048), (4, 16_384 + 0), (8, 12_501)):
        cfg = b.Config()
        cfg.layout, cfg.n_rows, cfg.n_cols, cfg.ld, cfg.n_candidates, cfg.n_keep = 0, 1000, 100_000 if S != 4 else 65_000, 1000, n_cand, 256
        cfg.n_schedulers = S
        assert lib.strads_workspace_bytes(C.byref(cfg), C.byref(out)) == -1, (S, n_cand)


def test_init_rejects_bad_pointers_and_parameters_without_touching_the_gpu(lib):
    from paper_1312_5766_b200 import binding as b

    def cfg_ok():
        cfg = b.Config()
        cfg.layout, cfg.n_rows, cfg.n_cols, cfg.ld, cfg.n_candidates, cfg.n_keep = 0, 1000, 5000, 1000, 100, 10
        for f in ("x_values", "y", "beta", "resid", "delta", "workspace"):
            setattr(cfg, f, 0x10000)                    # aligned, never dereferenced on the host
        cfg.lam, cfg.eta, cfg.rho, cfg.c_init = 0.1, 1e-6, 0.1, 1e4
        cfg.workspace_bytes = 1 << 30
        return cfg

    h = C.c_void_p(None)
    for field, value, want in [("x_values", None, -1), ("y", None, -1), ("workspace", None, -1),
                               ("x_values", 0x10004, -1), ("delta", 0x10008, -1), ("workspace", 0x10010, -1),
                               ("eta", 0.0, -1), ("rho", -0.1, -1), ("lam", -1.0, -1), ("c_init", 0.0, -1),
                               ("lam", float("nan"), -1), ("workspace_bytes", 16, -3), ("layout", 3, -2),
                               # C^2 + eta must stay finite in binary32 (else every first-phase race time is 0)
                               ("c_init", 2e18, -1), ("c_init", float("inf"), -1)]:
        cfg = cfg_ok()
        setattr(cfg, field, value)
        assert lib.strads_lasso_init(C.byref(cfg), C.byref(h)) == want, field
        assert not h.value
    cfg = cfg_ok()
    cfg.layout = 1                                       # CSC without index arrays
    assert lib.strads_lasso_init(C.byref(cfg), C.byref(h)) == -1
    assert lib.strads_lasso_init(C.byref(cfg_ok()), None) == -1
    # NULL handles
    assert lib.strads_round(None, None) == -1 and lib.strads_run(None, 1) == -1
    assert lib.strads_objective(None, None) == -1 and lib.strads_destroy(None) == -1
    assert lib.strads_set_wait_limit(None, 10) == -1 and lib.strads_inject_stall(None, 1) == -1
    assert lib.strads_recover(None) == -1
