"""Objective against cumulative coefficient updates under the three schedules the paper compares
(Section 5.1 and its convergence figure for the Lasso): the dynamic schedule of Algorithm 1 (priority draw +
rho filter), "static" (uniform draw + rho filter) and "random" (uniform draw, no dependency check).

    python -m paper_1312_5766_b200.compare_schedules [--workload c1] [--rounds N] [--every K] [--scale D]

Runs on a CUDA device through the library; prints one line per schedule and checkpoint.  The curves of the
paper's figure came from data that is not available; this regenerates their shape on the synthetic workloads.
"""
from __future__ import annotations

import argparse

import torch

from . import binding, workloads as wl

SCHEDULES = {                      # name -> flags
    "priority": 0,
    "static": binding.FLAG_UNIFORM_DRAW,
    "random": binding.FLAG_UNIFORM_DRAW | binding.FLAG_NO_FILTER,
}


def trace(p: wl.LassoProblem, schedule: str, rounds: int, every: int, device="cuda", extra_flags: int = 0):
    """[(rounds done, cumulative updates, objective)] at round 0 and after every `every` rounds."""
    s = binding.StradsLasso.from_problem(p, device=device, flags=SCHEDULES[schedule] | extra_flags)
    out = [(0, 0, s.objective())]
    done = 0
    while done < rounds:
        n = min(every, rounds - done)
        s.run(n)
        done += n
        out.append((done, s.totals()["kept"], s.objective()))
    rc, bits = s.status()
    if rc != 0:
        raise binding.StradsError(rc, "strads_status")
    s.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c1")
    ap.add_argument("--scale", type=int, default=1, help="divide N, J, the true support, P' and P by this")
    ap.add_argument("--rounds", type=int, default=0, help="0: the workload's own round count (divided by --scale)")
    ap.add_argument("--every", type=int, default=0)
    args = ap.parse_args()
    cfg = dict(wl.scaled(args.workload, args.scale) if args.scale > 1 else wl.CONFIGS[args.workload], name=args.workload)
    p = wl.make_problem(cfg, seed=0, device="cuda" if torch.cuda.is_available() else "cpu")
    rounds = args.rounds or max(1, cfg["rounds"] // args.scale)
    every = args.every or max(1, rounds // 10)
    print(f"# {args.workload}/{args.scale}: N={p.n_rows} J={p.n_cols} P'={p.n_candidates} P={p.n_keep} rho={p.rho} lambda={p.lam:.6g}")
    print("schedule rounds updates objective")
    for name in SCHEDULES:
        for r, u, f in trace(p, name, rounds, every):
            print(f"{name} {r} {u} {f:.9g}")


if __name__ == "__main__":
    main()
