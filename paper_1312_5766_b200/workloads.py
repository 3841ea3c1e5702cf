"""Seeded synthetic Lasso problems shaped like the paper's workloads.

The paper's Lasso experiments use few samples and very many covariates with a
sparse true coefficient vector (Section 5, "Datasets": 463 x 508,999 real SNP
data and 450 x 1,000,000 synthetic with 10,000 true non-zeros).  The real data
is not available, so every problem here is generated from a seed.

This module is the one piece shared by the CUDA tests, the CPU oracle tests and
the benchmark.  It holds data preparation only (random draws, column
standardisation, y = X beta* + noise, the choice of lambda); none of the
scheduled-round arithmetic lives here.  Everything is plain torch, so the same
function runs on the CPU (small cases) or on a CUDA device (large cases); the
arrays are then handed to both implementations unchanged.
"""
from __future__ import annotations

import dataclasses
import math

import torch

DENSE, CSC = 0, 1


@dataclasses.dataclass
class LassoProblem:
    layout: int
    n_rows: int
    n_cols: int
    # dense: x_cols [J, ld] float32, row j of the tensor is column j of X.  CSC: values [nnz]
    values: torch.Tensor
    row_idx: torch.Tensor | None   # int32 [nnz], ascending inside each column
    col_ptr: torch.Tensor | None   # int64 [J+1]
    y: torch.Tensor                # float32 [N]
    beta_star: torch.Tensor        # float32 [J]
    lam: float
    eta: float
    rho: float
    n_candidates: int
    n_keep: int
    rounds: int
    seed: int
    name: str = ""

    @property
    def ld(self) -> int:
        return int(self.values.shape[1]) if self.layout == DENSE else 0

    @property
    def nnz(self) -> int:
        return int(self.values.numel()) if self.layout == CSC else self.n_rows * self.n_cols


# name -> generator kwargs.  c1..c5 are the five benchmark configurations.
CONFIGS = {
    "c1": dict(kind="dense_iid", n_rows=1_000, n_cols=10_000, n_true=100, lam_frac=0.05,
               n_candidates=200, n_keep=32, rho=0.1, rounds=1_000),
    "c2": dict(kind="dense_iid", n_rows=10_000, n_cols=100_000, n_true=1_000, lam_frac=0.02,
               n_candidates=2_048, n_keep=256, rho=0.1, rounds=2_000),
    "c3": dict(kind="dense_grouped", n_rows=20_000, n_cols=200_000, n_true=2_000, lam_frac=0.02,
               n_candidates=4_096, n_keep=512, rho=0.1, rounds=2_000, group=20),
    "c4": dict(kind="csc_uniform", n_rows=50_000, n_cols=1_000_000, n_true=5_000, lam_frac=0.01,
               n_candidates=8_192, n_keep=1_024, rho=0.1, rounds=5_000, nnz_col=50),
    "c5": dict(kind="csc_zipf", n_rows=1_000_000, n_cols=10_000_000, n_true=20_000, lam_frac=0.01,
               n_candidates=16_384, n_keep=4_096, rho=0.05, rounds=5_000, nnz_col=20, zipf_a=1.1),
}


def scaled(name: str, div: int) -> dict:
    """The named configuration with N, J, the true support and U', U divided by `div`."""
    c = dict(CONFIGS[name])
    for k in ("n_rows", "n_cols", "n_true", "n_candidates", "n_keep"):
        c[k] = max(1, c[k] // div)
    if "group" in c:
        c["n_cols"] = (c["n_cols"] // c["group"]) * c["group"]
    if "nnz_col" in c:
        c["n_rows"] = max(c["n_rows"], 4 * c["nnz_col"])
    return c


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _standardise_(block: torch.Tensor, centre: bool) -> None:
    """In place: every row of `block` (a column of X) to mean 0 (optional) and unit 2-norm."""
    b64 = block.double()
    if centre:
        b64 -= b64.mean(dim=1, keepdim=True)
    nrm = b64.norm(dim=1, keepdim=True).clamp_min(1e-300)
    block.copy_((b64 / nrm).float())


def _beta_star(n_cols: int, support: torch.Tensor, g: torch.Generator, device) -> torch.Tensor:
    k = support.numel()
    mag = 0.5 + torch.rand(k, generator=g, device=device)
    sign = torch.where(torch.rand(k, generator=g, device=device) < 0.5, -1.0, 1.0)
    b = torch.zeros(n_cols, dtype=torch.float32, device=device)
    b[support] = (mag * sign).float()
    return b


def _dense(kind, n_rows, n_cols, n_true, lam_frac, sigma, seed, device, group=20, chunk=4096):
    gx, gb, gn = _gen(seed, device), _gen(seed + 1, device), _gen(seed + 2, device)
    x = torch.empty((n_cols, n_rows), dtype=torch.float32, device=device)
    if kind == "dense_grouped":
        chunk = max(group, (chunk // group) * group)
    for j0 in range(0, n_cols, chunk):
        j1 = min(n_cols, j0 + chunk)
        blk = torch.randn((j1 - j0, n_rows), generator=gx, device=device, dtype=torch.float32)
        if kind == "dense_grouped":
            # column j in group j // group: x = sqrt(0.8) z_g + sqrt(0.2) e
            ng = (j1 - j0 + group - 1) // group
            z = torch.randn((ng, n_rows), generator=gx, device=device, dtype=torch.float32)
            z = z.repeat_interleave(group, dim=0)[: j1 - j0]
            blk = math.sqrt(0.8) * z + math.sqrt(0.2) * blk
        _standardise_(blk, centre=True)
        x[j0:j1] = blk
    if kind == "dense_grouped":
        n_groups = n_cols // group
        grp = torch.randperm(n_groups, generator=gb, device=device)[:n_true]
        support = grp * group + torch.randint(0, group, (n_true,), generator=gb, device=device)
    else:
        support = torch.randperm(n_cols, generator=gb, device=device)[:n_true]
    beta_star = _beta_star(n_cols, support, gb, device)
    y64 = (x[support].double() * beta_star[support].double()[:, None]).sum(dim=0)
    y64 += sigma * torch.randn(n_rows, generator=gn, device=device, dtype=torch.float64)
    y = y64.float()
    xty_max = 0.0
    for j0 in range(0, n_cols, chunk):
        xty_max = max(xty_max, float((x[j0:j0 + chunk].double() @ y.double()).abs().max()))
    return x, y, beta_star, lam_frac * xty_max


def _distinct_rows(n_cols, nnz_col, draw, device, max_iter=200):
    """[J, nnz_col] sorted row indices, distinct inside each column.  `draw(k)` returns k fresh
    row draws; only entries that duplicate another entry of their column are redrawn."""
    rows = draw(n_cols * nnz_col).view(n_cols, nnz_col)
    for _ in range(max_iter):
        rows, _ = rows.sort(dim=1)
        dup = torch.zeros_like(rows, dtype=torch.bool)
        dup[:, 1:] = rows[:, 1:] == rows[:, :-1]
        n_dup = int(dup.sum())
        if n_dup == 0:
            return rows
        rows[dup] = draw(n_dup)
    raise RuntimeError("could not draw distinct rows")


def _csc(kind, n_rows, n_cols, n_true, lam_frac, sigma, seed, device, nnz_col, zipf_a=1.1):
    gx, gb, gn = _gen(seed, device), _gen(seed + 1, device), _gen(seed + 2, device)
    if kind == "csc_uniform":
        def draw(k):
            return torch.randint(0, n_rows, (k,), generator=gx, device=device, dtype=torch.int64)
    else:
        # Zipf(a) truncated to 1..N, P(i) proportional to i^-a, by inverse CDF
        w = torch.arange(1, n_rows + 1, device=device, dtype=torch.float64).pow_(-zipf_a)
        cdf = torch.cumsum(w, 0)
        cdf /= cdf[-1].clone()

        def draw(k):
            u = torch.rand(k, generator=gx, device=device, dtype=torch.float64)
            return torch.searchsorted(cdf, u).clamp_(max=n_rows - 1)
    rows = _distinct_rows(n_cols, nnz_col, draw, device)
    vals = torch.randn((n_cols, nnz_col), generator=gx, device=device, dtype=torch.float32)
    _standardise_(vals, centre=False)
    support = torch.randperm(n_cols, generator=gb, device=device)[:n_true]
    beta_star = _beta_star(n_cols, support, gb, device)
    y64 = sigma * torch.randn(n_rows, generator=gn, device=device, dtype=torch.float64)
    contrib = vals[support].double() * beta_star[support].double()[:, None]
    y64.index_add_(0, rows[support].reshape(-1), contrib.reshape(-1))
    y = y64.float()
    xty_max = 0.0
    step = max(1, (1 << 24) // nnz_col)
    for j0 in range(0, n_cols, step):
        r = rows[j0:j0 + step]
        xty = (vals[j0:j0 + step].double() * y.double()[r]).sum(dim=1)
        xty_max = max(xty_max, float(xty.abs().max()))
    col_ptr = torch.arange(0, n_cols + 1, device=device, dtype=torch.int64) * nnz_col
    return vals.reshape(-1), rows.reshape(-1).to(torch.int32), col_ptr, y, beta_star, lam_frac * xty_max


def make_problem(cfg: dict | str, seed: int = 0, device="cpu", eta: float = 1e-6,
                 sigma: float = 0.1) -> LassoProblem:
    """Generate one problem.  `cfg` is a name from CONFIGS or a dict of the same keys."""
    name = cfg if isinstance(cfg, str) else cfg.get("name", "custom")
    c = dict(CONFIGS[cfg]) if isinstance(cfg, str) else dict(cfg)
    kind = c["kind"]
    common = dict(eta=eta, rho=c["rho"], n_candidates=c["n_candidates"], n_keep=c["n_keep"],
                  rounds=c.get("rounds", 100), seed=seed, name=name)
    if kind in ("dense_iid", "dense_grouped"):
        x, y, bs, lam = _dense(kind, c["n_rows"], c["n_cols"], c["n_true"], c["lam_frac"], sigma, seed,
                               device, group=c.get("group", 20))
        return LassoProblem(DENSE, c["n_rows"], c["n_cols"], x, None, None, y, bs, lam, **common)
    if kind in ("csc_uniform", "csc_zipf"):
        v, r, p, y, bs, lam = _csc(kind, c["n_rows"], c["n_cols"], c["n_true"], c["lam_frac"], sigma, seed,
                                   device, c["nnz_col"], c.get("zipf_a", 1.1))
        return LassoProblem(CSC, c["n_rows"], c["n_cols"], v, r, p, y, bs, lam, **common)
    raise ValueError(f"unknown kind {kind!r}")


def to_logistic(p: LassoProblem, lam_frac: float = 0.1) -> LassoProblem:
    """The same design with binary labels for the logistic loss: y_i = 1 where the linear response
    x_i^T beta* + noise is positive, else 0; lambda = lam_frac * ||X^T (y - 1/2)||_inf (the smallest lambda
    for which beta = 0 is optimal, times lam_frac)."""
    y = (p.y > 0).to(torch.float32)
    c = (y.double() - 0.5)
    if p.layout == DENSE:
        xty_max = 0.0
        for j0 in range(0, p.n_cols, 4096):
            xty_max = max(xty_max, float((p.values[j0:j0 + 4096, : p.n_rows].double() @ c).abs().max()))
    else:
        contrib = p.values.double() * c[p.row_idx.long()]
        seg = torch.repeat_interleave(torch.arange(p.n_cols, device=p.values.device), p.col_ptr[1:] - p.col_ptr[:-1])
        xty = torch.zeros(p.n_cols, dtype=torch.float64, device=p.values.device).index_add_(0, seg, contrib)
        xty_max = float(xty.abs().max())
    return dataclasses.replace(p, y=y, lam=lam_frac * xty_max, name=p.name + "+logistic")
