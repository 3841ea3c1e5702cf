"""Thin ctypes binding of libstrads_b200.so (see include/strads.h for the contract).

Argument marshalling only: every step of the scheduled round runs in the CUDA kernels of the
library.  PyTorch is used for device memory and streams.  There is no CPU fallback: if the library
has not been built, importing its symbols raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import workloads as wl

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libstrads_b200.so")

OK = 0
FLAG_UNIFORM_DRAW = 1
FLAG_NO_FILTER = 2
FLAG_SIMT_GRAM = 4
FLAG_GRAM_3XTF32 = 8
FLAG_FULL_GRAM = 16
FLAG_ABS_WEIGHT = 32
FLAG_DYNAMIC_DEPS = 64
FLAG_LOGISTIC = 128
MAX_CANDIDATES = 16384
STALL_WALK_BARRIER, STALL_GRAM_LOADS = 1, 2

EXPORTS = [
    "strads_workspace_bytes", "strads_lasso_init", "strads_round", "strads_run", "strads_round_host",
    "strads_objective", "strads_sample", "strads_filter", "strads_update", "strads_get_round",
    "strads_set_round", "strads_totals", "strads_status", "strads_colnorm2", "strads_destroy",
    "strads_error_string", "strads_last_cuda_error", "strads_profile_begin", "strads_profile_end",
    "strads_sample_static", "strads_set_wait_limit", "strads_inject_stall", "strads_recover", "strads_margin",
]


class Config(C.Structure):
    _fields_ = [
        ("layout", C.c_int32),
        ("n_rows", C.c_int64), ("n_cols", C.c_int64), ("nnz", C.c_int64), ("ld", C.c_int64),
        ("x_values", C.c_void_p), ("x_row_idx", C.c_void_p), ("x_col_ptr", C.c_void_p),
        ("y", C.c_void_p), ("beta", C.c_void_p), ("resid", C.c_void_p), ("delta", C.c_void_p),
        ("lam", C.c_float), ("eta", C.c_float), ("rho", C.c_float), ("c_init", C.c_float),
        ("n_candidates", C.c_int32), ("n_keep", C.c_int32),
        ("seed", C.c_uint64),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
        ("stream", C.c_void_p),
        ("flags", C.c_uint32),
        ("n_schedulers", C.c_int32),
    ]


class RoundOut(C.Structure):
    _fields_ = [("cand", C.c_void_p), ("kept", C.c_void_p), ("dbeta", C.c_void_p), ("counts", C.c_void_p),
                ("gram", C.c_void_p)]


_lib = None


def load() -> C.CDLL:
    """Loads the CUDA library; raises if it has not been built (no fallback of any kind)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_1312_5766_b200.build` "
                "(nvcc, sm_100a). This package has no CPU or PyTorch fallback.")
        lib = C.CDLL(LIB_PATH)
        lib.strads_error_string.restype = C.c_char_p
        lib.strads_last_cuda_error.restype = C.c_char_p
        lib.strads_workspace_bytes.argtypes = [C.POINTER(Config), C.POINTER(C.c_size_t)]
        lib.strads_lasso_init.argtypes = [C.POINTER(Config), C.POINTER(C.c_void_p)]
        lib.strads_round.argtypes = [C.c_void_p, C.POINTER(RoundOut)]
        lib.strads_run.argtypes = [C.c_void_p, C.c_int64]
        lib.strads_round_host.argtypes = [C.c_void_p] + [C.c_void_p] * 6
        lib.strads_objective.argtypes = [C.c_void_p, C.POINTER(C.c_double)]
        lib.strads_sample.argtypes = [C.c_void_p, C.c_void_p]
        lib.strads_filter.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
        lib.strads_update.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
        lib.strads_get_round.argtypes = [C.c_void_p, C.POINTER(C.c_int64)]
        lib.strads_set_round.argtypes = [C.c_void_p, C.c_int64]
        lib.strads_totals.argtypes = [C.c_void_p, C.POINTER(C.c_int64)]
        lib.strads_status.argtypes = [C.c_void_p, C.POINTER(C.c_uint32)]
        lib.strads_colnorm2.argtypes = [C.c_void_p, C.POINTER(C.c_void_p)]
        lib.strads_destroy.argtypes = [C.c_void_p]
        lib.strads_profile_begin.argtypes = [C.c_void_p, C.c_int64]
        lib.strads_set_wait_limit.argtypes = [C.c_void_p, C.c_uint32]
        lib.strads_inject_stall.argtypes = [C.c_void_p, C.c_int32]
        lib.strads_recover.argtypes = [C.c_void_p]
        lib.strads_margin.argtypes = [C.c_void_p, C.POINTER(C.c_void_p)]
        lib.strads_sample_static.argtypes = [C.c_void_p, C.c_int64, C.c_float, C.c_uint64, C.c_uint64, C.c_int32,
                                             C.c_uint32, C.c_void_p, C.c_void_p]
        lib.strads_profile_end.argtypes = [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
        _lib = lib
    return _lib


class StradsError(RuntimeError):
    def __init__(self, code: int, where: str):
        lib = load()
        msg = lib.strads_error_string(code).decode()
        cuda = lib.strads_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} ({code})" + (f" [{cuda}]" if code == -4 and cuda else ""))
        self.code = code


def _check(code: int, where: str) -> None:
    if code != OK:
        raise StradsError(code, where)


def _ptr(t: torch.Tensor | None):
    return None if t is None else C.c_void_p(t.data_ptr())


def workspace_bytes(layout, n_rows, n_cols, n_candidates, n_keep, nnz=0, ld=None) -> int:
    cfg = Config()
    cfg.layout, cfg.n_rows, cfg.n_cols, cfg.nnz = layout, n_rows, n_cols, nnz
    cfg.ld = ld if ld is not None else (n_rows + 3) // 4 * 4
    cfg.n_candidates, cfg.n_keep = n_candidates, n_keep
    out = C.c_size_t(0)
    _check(load().strads_workspace_bytes(C.byref(cfg), C.byref(out)), "strads_workspace_bytes")
    return int(out.value)


STATIC_MAX_CANDIDATES = 4096


def sample_static(delta: torch.Tensor, eta: float, seed: int, t: int, n_candidates: int, flags: int = 0,
                  out: torch.Tensor | None = None) -> torch.Tensor:
    """Candidate draw without a handle or workspace (strads_sample_static): for callers that cannot
    allocate device memory.  `out` (int32 [n_candidates], device) is allocated here only if not given."""
    assert delta.is_cuda and delta.dtype == torch.float32 and delta.is_contiguous()
    if out is None:
        out = torch.empty(n_candidates, dtype=torch.int32, device=delta.device)
    with torch.cuda.device(delta.device):
        stream = torch.cuda.current_stream().cuda_stream
        _check(load().strads_sample_static(_ptr(delta), int(delta.numel()), float(eta), int(seed), int(t),
                                           int(n_candidates), int(flags), _ptr(out), C.c_void_p(stream)),
               "strads_sample_static")
    return out


class StradsLasso:
    """One Lasso problem resident on a CUDA device, stepped by the library's kernels.

    x_values / row_idx / col_ptr / y are torch CUDA tensors owned by the caller (kept alive here);
    beta, resid, delta and the workspace are allocated here as torch tensors.
    """

    def __init__(self, layout, n_rows, n_cols, values, y, lam, eta, rho, n_candidates, n_keep, seed=0,
                 row_idx=None, col_ptr=None, c_init=1e4, flags=0, beta0=None, stream=None, n_schedulers=1):
        lib = load()
        dev = values.device
        assert dev.type == "cuda", "the design matrix must live on a CUDA device"
        self.layout, self.N, self.J = int(layout), int(n_rows), int(n_cols)
        self.n_candidates, self.n_keep = int(n_candidates), int(n_keep)
        self.values, self.row_idx, self.col_ptr, self.y = values, row_idx, col_ptr, y
        self.lam, self.eta, self.rho = float(lam), float(eta), float(rho)
        assert values.dtype == torch.float32 and y.dtype == torch.float32 and values.is_contiguous()
        ld = int(values.shape[1]) if layout == wl.DENSE else 0
        nnz = int(values.numel()) if layout == wl.CSC else 0
        if layout == wl.CSC:
            assert row_idx.dtype == torch.int32 and col_ptr.dtype == torch.int64
        self.beta = torch.zeros(self.J, dtype=torch.float32, device=dev) if beta0 is None else \
            beta0.to(device=dev, dtype=torch.float32).contiguous().clone()
        self.resid = torch.empty(self.N, dtype=torch.float32, device=dev)
        self.delta = torch.empty(self.J, dtype=torch.float32, device=dev)
        self.stream = stream
        cfg = Config()
        cfg.layout, cfg.n_rows, cfg.n_cols, cfg.nnz, cfg.ld = self.layout, self.N, self.J, nnz, ld
        cfg.n_candidates, cfg.n_keep = self.n_candidates, self.n_keep
        self.n_schedulers = cfg.n_schedulers = int(n_schedulers)
        cfg.flags = flags                      # (the logistic loss adds the margin to the workspace)
        need = C.c_size_t(0)
        _check(lib.strads_workspace_bytes(C.byref(cfg), C.byref(need)), "strads_workspace_bytes")
        self.workspace = torch.empty(int(need.value), dtype=torch.uint8, device=dev)
        cfg.x_values, cfg.x_row_idx, cfg.x_col_ptr = values.data_ptr(), \
            (row_idx.data_ptr() if row_idx is not None else None), (col_ptr.data_ptr() if col_ptr is not None else None)
        cfg.y, cfg.beta, cfg.resid, cfg.delta = y.data_ptr(), self.beta.data_ptr(), self.resid.data_ptr(), \
            self.delta.data_ptr()
        cfg.lam, cfg.eta, cfg.rho, cfg.c_init = lam, eta, rho, c_init
        cfg.seed = seed
        cfg.workspace, cfg.workspace_bytes = self.workspace.data_ptr(), int(need.value)
        cfg.stream = None if stream is None else stream.cuda_stream
        cfg.flags = flags
        self._cfg = cfg
        self._h = C.c_void_p(None)
        with torch.cuda.device(dev):
            _check(lib.strads_lasso_init(C.byref(cfg), C.byref(self._h)), "strads_lasso_init")
        self._dev = dev
        # per-round output buffers (device)
        self.cand = torch.empty(self.n_candidates, dtype=torch.int32, device=dev)
        self.kept = torch.empty(self.n_keep, dtype=torch.int32, device=dev)
        self.dbeta = torch.empty(self.n_keep, dtype=torch.float32, device=dev)
        self.counts = torch.zeros(4, dtype=torch.int32, device=dev)

    @classmethod
    def from_problem(cls, p: wl.LassoProblem, device="cuda", **kw):
        mv = lambda t: None if t is None else t.to(device)
        return cls(p.layout, p.n_rows, p.n_cols, mv(p.values), mv(p.y), p.lam, p.eta, p.rho, p.n_candidates,
                   p.n_keep, seed=p.seed, row_idx=mv(p.row_idx), col_ptr=mv(p.col_ptr), **kw)

    # ---- whole rounds ----
    def round(self, want_gram: bool = False):
        """One round; returns (cand, kept, dbeta, counts) device tensors (reused between calls)."""
        out = RoundOut(self.cand.data_ptr(), self.kept.data_ptr(), self.dbeta.data_ptr(), self.counts.data_ptr(), None)
        gram = None
        if want_gram:
            gram = torch.zeros((self.n_candidates, self.n_candidates), dtype=torch.float32, device=self._dev)
            out.gram = gram.data_ptr()
        _check(load().strads_round(self._h, C.byref(out)), "strads_round")
        return (self.cand, self.kept, self.dbeta, self.counts) + ((gram,) if want_gram else ())

    def run(self, n_rounds: int) -> None:
        _check(load().strads_run(self._h, int(n_rounds)), "strads_run")

    def round_host(self, beta_h, resid_h, delta_h, kept_h=None, dbeta_h=None, counts_h=None) -> None:
        """One round on state held in (pinned) host tensors; see strads_round_host."""
        _check(load().strads_round_host(self._h, _ptr(beta_h), _ptr(resid_h), _ptr(delta_h), _ptr(kept_h),
                                        _ptr(dbeta_h), _ptr(counts_h)), "strads_round_host")

    def objective(self) -> float:
        out = C.c_double(0.0)
        _check(load().strads_objective(self._h, C.byref(out)), "strads_objective")
        return float(out.value)

    # ---- split-phase ----
    def sample(self) -> torch.Tensor:
        _check(load().strads_sample(self._h, _ptr(self.cand)), "strads_sample")
        return self.cand

    def filter(self, cand: torch.Tensor, want_gram: bool = False):
        n = int(cand.numel())
        gram = torch.zeros((n, n), dtype=torch.float32, device=self._dev) if want_gram else None
        _check(load().strads_filter(self._h, _ptr(cand), n, _ptr(self.kept), _ptr(self.counts), _ptr(gram)),
               "strads_filter")
        return (self.kept, self.counts) + ((gram,) if want_gram else ())

    def update(self, kept: torch.Tensor) -> torch.Tensor:
        _check(load().strads_update(self._h, _ptr(kept), int(kept.numel()), _ptr(self.dbeta)), "strads_update")
        return self.dbeta

    # ---- bookkeeping ----
    def get_round(self) -> int:
        t = C.c_int64(0)
        _check(load().strads_get_round(self._h, C.byref(t)), "strads_get_round")
        return int(t.value)

    def set_round(self, t: int) -> None:
        _check(load().strads_set_round(self._h, int(t)), "strads_set_round")

    def totals(self) -> dict:
        t = (C.c_int64 * 4)()
        _check(load().strads_totals(self._h, t), "strads_totals")
        return {"rounds": t[0], "examined": t[1], "kept": t[2], "nonzero": t[3]}

    def status(self) -> tuple[int, int]:
        bits = C.c_uint32(0)
        rc = load().strads_status(self._h, C.byref(bits))
        return rc, int(bits.value)

    def set_wait_limit(self, iterations: int) -> None:
        _check(load().strads_set_wait_limit(self._h, int(iterations)), "strads_set_wait_limit")

    def inject_stall(self, which: int) -> None:
        _check(load().strads_inject_stall(self._h, int(which)), "strads_inject_stall")

    def recover(self) -> None:
        _check(load().strads_recover(self._h), "strads_recover")

    def colnorm2(self) -> torch.Tensor:
        """||x_j||^2 (FP64), a view into the workspace."""
        ptr = C.c_void_p(None)
        _check(load().strads_colnorm2(self._h, C.byref(ptr)), "strads_colnorm2")
        off = ptr.value - self.workspace.data_ptr()
        return self.workspace[off:off + 8 * self.J].view(torch.float64)

    def margin(self) -> torch.Tensor:
        """The margin X beta (FP32), a view into the workspace (logistic loss only)."""
        ptr = C.c_void_p(None)
        _check(load().strads_margin(self._h, C.byref(ptr)), "strads_margin")
        off = ptr.value - self.workspace.data_ptr()
        return self.workspace[off:off + 4 * self.N].view(torch.float32)

    def profile_begin(self, max_rounds: int) -> None:
        _check(load().strads_profile_begin(self._h, int(max_rounds)), "strads_profile_begin")

    def profile_end(self) -> dict:
        ms = (C.c_double * 5)()
        n = C.c_int64(0)
        _check(load().strads_profile_end(self._h, ms, C.byref(n)), "strads_profile_end")
        return {"rounds": int(n.value), "sample_ms": ms[0], "pack_ms": ms[1], "gram_ms": ms[2], "walk_ms": ms[3],
                "update_ms": ms[4]}

    def close(self) -> None:
        if self._h:
            load().strads_destroy(self._h)
            self._h = C.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
