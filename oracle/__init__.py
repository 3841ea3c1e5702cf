"""ctypes binding of the FP64 CPU oracle (``strads_oracle.c``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU
baseline call this; the CUDA library and its Python binding never do, and this
package imports nothing from them.  All arithmetic lives in the C file; this
module only marshals numpy arrays.

Paper: "Structure-Aware Dynamic Scheduler for Parallel Machine Learning",
Section 2.1 (Algorithm 1, Eq. 1, Eq. 2).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "strads_oracle.c")
_LIB = os.path.join(_HERE, "libstrads_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (strict IEEE, no contraction). Returns the .so path."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(
            ["gcc", "-O2", "-std=c99", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
             "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


class _SoMatrix(C.Structure):
    _fields_ = [
        ("layout", C.c_int32),
        ("n_rows", C.c_int64),
        ("n_cols", C.c_int64),
        ("ld", C.c_int64),
        ("values", C.c_void_p),
        ("row_idx", C.c_void_p),
        ("col_ptr", C.c_void_p),
    ]


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = C.CDLL(build())
            lib.so_unit_exponential_f32.restype = C.c_float
            lib.so_unit_exponential_f32.argtypes = [C.c_uint32]
            lib.so_race_key.restype = C.c_float
            lib.so_race_key.argtypes = [C.c_float, C.c_float, C.c_uint32]
            lib.so_race_key_mode.restype = C.c_float
            lib.so_race_key_mode.argtypes = [C.c_float, C.c_float, C.c_uint32, C.c_int32]
            lib.so_draw_word.restype = C.c_uint32
            lib.so_draw_word.argtypes = [C.c_uint64, C.c_uint64, C.c_uint64]
            lib.so_corr.restype = C.c_double
            lib.so_objective.restype = C.c_double
            lib.so_objective_from_scratch.restype = C.c_double
            lib.so_objective_logistic.restype = C.c_double
            _lib = lib
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


class Matrix:
    """Design matrix X (N x J) in FP32 storage: dense column-major or CSC."""

    def __init__(self, layout, n_rows, n_cols, values, row_idx=None, col_ptr=None, ld=None):
        self.layout = int(layout)
        self.n_rows, self.n_cols = int(n_rows), int(n_cols)
        self.values = np.ascontiguousarray(values, dtype=np.float32)
        self.row_idx = None if row_idx is None else np.ascontiguousarray(row_idx, dtype=np.int32)
        self.col_ptr = None if col_ptr is None else np.ascontiguousarray(col_ptr, dtype=np.int64)
        self.ld = int(ld if ld is not None else n_rows)
        self._c = _SoMatrix(self.layout, self.n_rows, self.n_cols, self.ld,
                            _p(self.values), _p(self.row_idx), _p(self.col_ptr))

    @classmethod
    def dense(cls, x_cols, n_rows=None):
        """x_cols: array of shape [J, ld] (row j of the array is column j of X)."""
        x_cols = np.ascontiguousarray(x_cols, dtype=np.float32)
        J, ld = x_cols.shape
        return cls(0, ld if n_rows is None else n_rows, J, x_cols, ld=ld)

    @classmethod
    def csc(cls, n_rows, n_cols, values, row_idx, col_ptr):
        return cls(1, n_rows, n_cols, values, row_idx, col_ptr)

    @property
    def ref(self):
        return C.byref(self._c)


def _f64(a):
    a = np.ascontiguousarray(a, dtype=np.float64)
    return a


def philox4x32_10(ctr, key):
    lib = _load()
    c = (C.c_uint32 * 4)(*[int(v) & 0xFFFFFFFF for v in ctr])
    k = (C.c_uint32 * 2)(*[int(v) & 0xFFFFFFFF for v in key])
    o = (C.c_uint32 * 4)()
    lib.so_philox4x32_10(c, k, o)
    return [int(v) for v in o]


def draw_word(seed, t, j):
    return int(_load().so_draw_word(int(seed), int(t), int(j)))


def unit_exponential(x):
    return float(_load().so_unit_exponential_f32(int(x) & 0xFFFFFFFF))


def race_key(delta_j, eta, x):
    return float(_load().so_race_key(float(delta_j), float(eta), int(x) & 0xFFFFFFFF))


WEIGHT_MODES = {"square": 0, "abs": 1, "uniform": 2}     # p(j) ~ delta^2 + eta | |delta| + eta | 1
FILTER_MODES = {"rho": 0, "none": 1, "dynamic": 2}        # Algorithm 1's test | first P candidates | dormant coefficients do not couple


def race_key_mode(delta_j, eta, x, weight):
    return float(_load().so_race_key_mode(float(delta_j), float(eta), int(x) & 0xFFFFFFFF, WEIGHT_MODES[weight]))


def sample(delta, eta, seed, t, n_cand, return_keys=False, weight="square"):
    lib = _load()
    delta = _f64(delta)
    J = delta.shape[0]
    cand = np.empty(n_cand, dtype=np.int32)
    if weight != "square":
        assert not return_keys
        rc = lib.so_sample_mode(C.c_int64(J), _p(delta), C.c_double(eta), C.c_uint64(seed), C.c_uint64(t),
                                C.c_int32(n_cand), C.c_int32(WEIGHT_MODES[weight]), _p(cand))
        if rc:
            raise ValueError(f"so_sample_mode failed: {rc}")
        return cand
    keys = np.empty(J, dtype=np.float32) if return_keys else None
    rc = lib.so_sample(C.c_int64(J), _p(delta), C.c_double(eta), C.c_uint64(seed), C.c_uint64(t),
                       C.c_int32(n_cand), _p(cand), _p(keys))
    if rc:
        raise ValueError(f"so_sample failed: {rc}")
    return (cand, keys) if return_keys else cand


def sample_part(delta, eta, seed, t, n_sched, sched, n_cand):
    """Candidates of scheduler thread `sched` of `n_sched` (it owns j = sched mod n_sched), best first."""
    delta = _f64(delta)
    cand = np.empty(n_cand, dtype=np.int32)
    rc = _load().so_sample_part(C.c_int64(delta.shape[0]), _p(delta), C.c_double(eta), C.c_uint64(seed), C.c_uint64(t),
                                C.c_int32(n_sched), C.c_int32(sched), C.c_int32(n_cand), _p(cand))
    if rc:
        raise ValueError(f"so_sample_part failed: {rc}")
    return cand


def colnorm2(X: Matrix):
    n2 = np.empty(X.n_cols, dtype=np.float64)
    _load().so_colnorm2(X.ref, _p(n2))
    return n2


def corr(X: Matrix, n2, j, k):
    return float(_load().so_corr(X.ref, _p(_f64(n2)), C.c_int64(j), C.c_int64(k)))


def filter(X: Matrix, n2, cand, n_keep, rho, follow=None, tol=0.0):
    """Greedy first-fit filter. Returns (kept, n_examined, min_margin)."""
    lib = _load()
    n2 = _f64(n2)
    cand = np.ascontiguousarray(cand, dtype=np.int32)
    kept = np.full(n_keep, -1, dtype=np.int32)
    nk, ne, mm = C.c_int32(0), C.c_int32(0), C.c_double(0)
    fol = None if follow is None else np.ascontiguousarray(follow, dtype=np.int32)
    lib.so_filter(X.ref, _p(n2), _p(cand), C.c_int32(len(cand)), C.c_int32(n_keep), C.c_double(rho),
                  _p(fol), C.c_int32(0 if fol is None else len(fol)), C.c_double(tol),
                  _p(kept), C.byref(nk), C.byref(ne), C.byref(mm))
    return kept[: nk.value].copy(), ne.value, mm.value


def filter_dynamic(X: Matrix, n2, cand, n_keep, rho, beta, delta):
    """The filter with dependencies dropped at run time (a coefficient that is zero and whose last update left it
    there couples with nobody).  Returns (kept, n_examined)."""
    n2, beta, delta = _f64(n2), _f64(beta), _f64(delta)
    cand = np.ascontiguousarray(cand, dtype=np.int32)
    kept = np.full(n_keep, -1, dtype=np.int32)
    nk, ne = C.c_int32(0), C.c_int32(0)
    _load().so_filter_dynamic(X.ref, _p(n2), _p(cand), C.c_int32(len(cand)), C.c_int32(n_keep), C.c_double(rho),
                              _p(beta), _p(delta), _p(kept), C.byref(nk), C.byref(ne))
    return kept[: nk.value].copy(), ne.value


def update(X: Matrix, n2, lam, kept, beta, resid, delta):
    """In-place Jacobi update of the kept coefficients; returns dbeta (float64)."""
    for a in (beta, resid, delta):
        assert a.dtype == np.float64 and a.flags.c_contiguous
    n2 = _f64(n2)
    kept = np.ascontiguousarray(kept, dtype=np.int32)
    dbeta = np.zeros(len(kept), dtype=np.float64)
    _load().so_update(X.ref, _p(n2), C.c_double(lam), _p(kept), C.c_int32(len(kept)),
                      _p(beta), _p(resid), _p(delta), _p(dbeta))
    return dbeta


def init(X: Matrix, y, c_init):
    """Returns (n2, beta, resid, delta) as float64 arrays."""
    y = np.ascontiguousarray(y, dtype=np.float32)
    n2 = np.empty(X.n_cols)
    beta = np.empty(X.n_cols)
    delta = np.empty(X.n_cols)
    resid = np.empty(X.n_rows)
    _load().so_init(X.ref, _p(y), C.c_double(c_init), _p(n2), _p(beta), _p(resid), _p(delta))
    return n2, beta, resid, delta


def round(X: Matrix, n2, lam, eta, rho, n_cand, n_keep, seed, t, beta, resid, delta, n_sched=1, weight="square",
          filter="rho"):
    """One round in place (round t is dispatched by scheduler thread t mod n_sched).
    weight / filter: another schedule (WEIGHT_MODES, FILTER_MODES), one scheduler thread only.
    Returns dict(cand, kept, dbeta, counts)."""
    for a in (beta, resid, delta):
        assert a.dtype == np.float64 and a.flags.c_contiguous
    n2 = _f64(n2)
    cand = np.empty(n_cand, dtype=np.int32)
    kept = np.full(n_keep, -1, dtype=np.int32)
    dbeta = np.zeros(n_keep, dtype=np.float64)
    counts = np.zeros(4, dtype=np.int32)
    if weight != "square" or filter != "rho":
        assert n_sched == 1
        rc = _load().so_round_mode(X.ref, _p(n2), C.c_double(lam), C.c_double(eta), C.c_double(rho),
                                   C.c_int32(n_cand), C.c_int32(n_keep), C.c_uint64(seed), C.c_uint64(t),
                                   C.c_int32(WEIGHT_MODES[weight]), C.c_int32(FILTER_MODES[filter]),
                                   _p(beta), _p(resid), _p(delta), _p(cand), _p(kept), _p(dbeta), _p(counts))
    elif n_sched == 1:
        rc = _load().so_round(X.ref, _p(n2), C.c_double(lam), C.c_double(eta), C.c_double(rho),
                              C.c_int32(n_cand), C.c_int32(n_keep), C.c_uint64(seed), C.c_uint64(t),
                              _p(beta), _p(resid), _p(delta), _p(cand), _p(kept), _p(dbeta), _p(counts))
    else:
        rc = _load().so_round_part(X.ref, _p(n2), C.c_double(lam), C.c_double(eta), C.c_double(rho),
                                   C.c_int32(n_cand), C.c_int32(n_keep), C.c_uint64(seed), C.c_uint64(t),
                                   C.c_int32(n_sched), _p(beta), _p(resid), _p(delta), _p(cand), _p(kept),
                                   _p(dbeta), _p(counts))
    if rc:
        raise ValueError(f"so_round failed: {rc}")
    nk = int(counts[2])
    return {"cand": cand, "kept": kept[:nk].copy(), "dbeta": dbeta[:nk].copy(), "counts": counts}


def objective(resid, beta, lam):
    resid, beta = _f64(resid), _f64(beta)
    return float(_load().so_objective(C.c_int64(len(resid)), C.c_int64(len(beta)), _p(resid), _p(beta),
                                      C.c_double(lam)))


def objective_from_scratch(X: Matrix, y, beta, lam):
    """Returns (F, r) with r = y - X beta recomputed from beta alone."""
    y = np.ascontiguousarray(y, dtype=np.float32)
    beta = _f64(beta)
    r = np.empty(X.n_rows)
    f = _load().so_objective_from_scratch(X.ref, _p(y), _p(beta), C.c_double(lam), _p(r))
    return float(f), r


def gradient(X: Matrix, resid):
    g = np.empty(X.n_cols)
    _load().so_gradient(X.ref, _p(_f64(resid)), _p(g))
    return g


# ---- logistic loss (labels y in {0, 1}; state: beta, the margin X beta, r = y - sigma(margin), delta) ----
def init_logistic(X: Matrix, y, c_init):
    """Returns (n2, beta, margin, resid, delta) as float64 arrays."""
    y = np.ascontiguousarray(y, dtype=np.float32)
    n2, beta, delta = np.empty(X.n_cols), np.empty(X.n_cols), np.empty(X.n_cols)
    margin, resid = np.empty(X.n_rows), np.empty(X.n_rows)
    _load().so_init_logistic(X.ref, _p(y), C.c_double(c_init), _p(n2), _p(beta), _p(margin), _p(resid), _p(delta))
    return n2, beta, margin, resid, delta


def update_logistic(X: Matrix, y, n2, lam, kept, beta, margin, resid, delta):
    y = np.ascontiguousarray(y, dtype=np.float32)
    for a in (beta, margin, resid, delta):
        assert a.dtype == np.float64 and a.flags.c_contiguous
    kept = np.ascontiguousarray(kept, dtype=np.int32)
    dbeta = np.zeros(len(kept), dtype=np.float64)
    _load().so_update_logistic(X.ref, _p(y), _p(_f64(n2)), C.c_double(lam), _p(kept), C.c_int32(len(kept)),
                               _p(beta), _p(margin), _p(resid), _p(delta), _p(dbeta))
    return dbeta


def objective_logistic(y, margin, beta, lam):
    y = np.ascontiguousarray(y, dtype=np.float32)
    margin, beta = _f64(margin), _f64(beta)
    return float(_load().so_objective_logistic(C.c_int64(len(margin)), C.c_int64(len(beta)), _p(y), _p(margin), _p(beta),
                                               C.c_double(lam)))


def round_logistic(X: Matrix, y, n2, lam, eta, rho, n_cand, n_keep, seed, t, beta, margin, resid, delta, weight="square",
                   filter="rho"):
    """One round in place with the logistic loss.  Returns dict(cand, kept, dbeta, counts)."""
    y = np.ascontiguousarray(y, dtype=np.float32)
    for a in (beta, margin, resid, delta):
        assert a.dtype == np.float64 and a.flags.c_contiguous
    n2 = _f64(n2)
    cand = np.empty(n_cand, dtype=np.int32)
    kept = np.full(n_keep, -1, dtype=np.int32)
    dbeta = np.zeros(n_keep, dtype=np.float64)
    counts = np.zeros(4, dtype=np.int32)
    rc = _load().so_round_logistic(X.ref, _p(y), _p(n2), C.c_double(lam), C.c_double(eta), C.c_double(rho),
                                   C.c_int32(n_cand), C.c_int32(n_keep), C.c_uint64(seed), C.c_uint64(t),
                                   C.c_int32(WEIGHT_MODES[weight]), C.c_int32(FILTER_MODES[filter]),
                                   _p(beta), _p(margin), _p(resid), _p(delta), _p(cand), _p(kept), _p(dbeta), _p(counts))
    if rc:
        raise ValueError(f"so_round_logistic failed: {rc}")
    nk = int(counts[2])
    return {"cand": cand, "kept": kept[:nk].copy(), "dbeta": dbeta[:nk].copy(), "counts": counts}
