#!/usr/bin/env python
"""Benchmark of the scheduled-Lasso round on B200: coordinate updates per second.

A step is one whole round (sample -> Gram -> greedy filter -> update) on synthetic data generated on the
device from a seed.  The headline workload is the largest dense configuration ("c3": 20,000 x 200,000 with
correlated groups, P' = 4,096, P = 512); the largest sparse one ("c5": CSC 1,000,000 x 10,000,000 with Zipf
rows) is timed the same way in the same run and reported under the key "c5" of the same JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3] [--sparse-leg c5|none]
                    [--impl ours|reference]

Prints ONE JSON line.  The K-step region is timed REPEATS times back to back (CUDA events on the launching
stream) and the median is reported.  `--impl reference` times the FP64 CPU oracle instead (rank 0 only).
With N > 1 (under torchrun) every rank runs an independent replica: the round has no inter-GPU step.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_1312_5766_b200 import workloads as wl  # noqa: E402

METRIC = "coordinate updates/sec and % of HBM roofline per STRADS round (1xB200)"
UNIT = "coordinate updates/s"
REPEATS = 7              # timed regions of K steps each; the median is reported
GRAPH_ROUNDS = 16        # untimed rounds that make sure the captured launch sequences have been replayed before timing
# DRAM bytes (read + write) per launch of the dominant kernel from ncu (dram__bytes_read.sum + dram__bytes_write.sum),
# keyed by (workload, kernel); None where the kernel has changed since its counters were taken.  Sources: the summaries
# under profiles/ named for the kernel and workload.
NCU_TRAFFIC = {
    # profiles/ncu_k_gram_dense_tc_window_c3_J20000.md: 25.75 MB read + 0 written per launch (captured with J cut to 20,000;
    # the kernel reads the window's BF16 copies only, so its traffic does not depend on J) = the algorithmic 2 N W
    ("c3", "k_gram_dense_tc<screen>"): 25.75e6,
    # profiles/ncu_full_round_kernels_c4.md: 6.82 MB read per launch (the buckets of the window candidates' rows)
    ("c4", "k_csc_bucket_dots"): 6.82e6,
    # k_walk_csc spins on a grid barrier: no multi-pass capture of it is made (one-pass launch list only)
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]),
                "sm_max_mhz": d.get("sm_max_mhz", 1965.0), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "sm_max_mhz": 1965.0,
            "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "100", "-i", str(gpu_index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self) -> dict:
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1])); mx.append(float(c[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        self.f.close()
        os.unlink(self.f.name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def l2_note(p: wl.LassoProblem) -> str:
    gb = (4.0 * p.n_rows * p.n_cols if p.layout == wl.DENSE else 8.0 * p.nnz) / 1e9
    return (f"inputs larger than L2: the design matrix ({gb:.1f} GB for {p.name}) far exceeds the 126 MB L2 and every round "
            "draws a fresh candidate set from all of it")


def config_of(p: wl.LassoProblem, workload: str, world: int, n_candidates=None, n_keep=None) -> dict:
    """The `config` object, the same keys from both arms."""
    return {"workload": workload, "layout": "dense" if p.layout == wl.DENSE else "csc", "n_rows": p.n_rows,
            "n_cols": p.n_cols, "n_candidates": n_candidates or p.n_candidates, "n_keep": n_keep or p.n_keep,
            "rho": p.rho, "eta": p.eta, "lambda": p.lam, "parallelism": f"replicas x{world}", "l2": l2_note(p)}


def oracle_inputs(p: wl.LassoProblem):
    """Host copies of the device arrays for the CPU oracle (the same FP32 bits)."""
    import oracle
    if p.layout == wl.DENSE:
        return oracle.Matrix.dense(p.values.cpu().numpy(), n_rows=p.n_rows)
    return oracle.Matrix.csc(p.n_rows, p.n_cols, p.values.cpu().numpy(), p.row_idx.cpu().numpy(),
                             p.col_ptr.cpu().numpy())


def host_has_room_for(p: wl.LassoProblem) -> bool:
    try:
        import psutil
        need = p.values.numel() * 4 * 1.5 + (p.row_idx.numel() * 4 if p.row_idx is not None else 0)
        return psutil.virtual_memory().available > need + (8 << 30)
    except Exception:
        return True


def time_oracle_rounds(p, X, n2, state, t0, n_cand, n_keep, budget_s, min_rounds=3, max_rounds=10**9):
    """Runs oracle rounds from `state` until the time budget is used; returns (updates, seconds, rounds)."""
    import oracle
    beta, resid, delta = state
    lam, eta, rho = float(np.float32(p.lam)), float(np.float32(p.eta)), float(np.float32(p.rho))
    kept_total, rounds = 0, 0
    start = time.perf_counter()
    while rounds < max_rounds and (rounds < min_rounds or time.perf_counter() - start < budget_s):
        out = oracle.round(X, n2, lam, eta, rho, n_cand, n_keep, p.seed, t0 + rounds, beta, resid, delta)
        kept_total += int(out["counts"][2])
        rounds += 1
    return kept_total, time.perf_counter() - start, rounds


def run_reference(args, device):
    """The reference arm: the FP64 oracle, as it stands, on the host cores (single thread)."""
    import oracle
    p = wl.make_problem(args.workload, seed=0, device=device)
    X = oracle_inputs(p)
    n2, beta, resid, delta = oracle.init(X, p.y.cpu().numpy(), 1e4)
    # size the per-step sample so that the whole run ends within a few minutes
    n_cand, n_keep = p.n_candidates, p.n_keep
    budget = 150.0
    probe = (beta.copy(), resid.copy(), delta.copy())
    while True:
        _, sec, _ = time_oracle_rounds(p, X, n2, tuple(a.copy() for a in probe), 0, n_cand, n_keep, 0.0, min_rounds=1,
                                       max_rounds=1)
        if sec * (args.steps + args.warmup) <= budget or n_keep == 1:
            break
        n_keep = max(1, n_keep // 2)
        n_cand = max(n_keep, n_cand // 2)
    time_oracle_rounds(p, X, n2, (beta, resid, delta), 0, n_cand, n_keep, 0.0, min_rounds=args.warmup,
                       max_rounds=args.warmup)
    kept, sec, rounds = time_oracle_rounds(p, X, n2, (beta, resid, delta), args.warmup, n_cand, n_keep, 0.0,
                                           min_rounds=args.steps, max_rounds=args.steps)
    value = kept / sec
    sample = (f"{rounds} oracle rounds of {args.workload} with P'={n_cand}, P={n_keep} per step "
              f"(full round is P'={p.n_candidates}, P={p.n_keep})")
    return {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * sec / rounds, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(p, args.workload, args.gpus, n_cand, n_keep),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


def aggregate(units_local: float, ms_local: float, dist_ok: bool, device):
    """Whole-job numbers: units summed over ranks, time = max over ranks."""
    if not dist_ok:
        return units_local, ms_local
    import torch.distributed as dist
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    m = torch.tensor([ms_local], dtype=torch.float64, device=device)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    dist.all_reduce(m, op=dist.ReduceOp.MAX)
    return float(u.item()), float(m.item())


def window_of(p: wl.LassoProblem) -> int:
    """The library's rule for the leading window of candidates whose Gram is formed first."""
    slack = max(p.n_keep // 4, 64) if p.layout == wl.DENSE else p.n_keep // 2 + 128
    w = (p.n_keep + slack + 127) // 128 * 128
    return w if 2 * w <= p.n_candidates else p.n_candidates


def rooflines(p: wl.LassoProblem, workload: str, step_ms: dict, kept_per_round: float, examined_per_round: float,
              moving_per_round: float, ms_per_step: float, peaks: dict) -> dict:
    """Roofline of the dominant kernel plus the streaming kernels against the measured HBM bandwidth."""
    window = window_of(p)
    out = {}
    if p.layout == wl.DENSE:
        # dominant: the tensor-core Gram of the window (screen on BF16 operands, split K combined inside thread-block
        # clusters, exact recheck and the greedy walk by the last CTA).  Algorithmic flops W(W-1)N.
        kernel = "k_gram_dense_tc<screen>"
        flops = float(window) * (window - 1) * p.n_rows
        achieved = flops / (step_ms["gram_ms"] * 1e-3) / 1e12
        peak = peaks["bf16_tflops"]
        out["roofline"] = {
            "kernel": kernel, "bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
            "frac": achieved / peak, "traffic": NCU_TRAFFIC.get((workload, kernel)), "window": window,
            "launch_ms": step_ms["gram_ms"], "algorithmic_flops_per_launch": flops,
            "peak_source": f"{peaks['source']} BF16 burst (the screen's operands are BF16; pairs it cannot call are decided "
                           "exactly in FP64); the kernel is timed alone between events"}
        # the update reads the columns of the kept coefficients that move (a null change needs no column) and r twice
        upd_bytes = 4.0 * p.n_rows * moving_per_round + 8.0 * p.n_rows + 16.0 * kept_per_round
        pack_bytes = 6.0 * p.n_rows * window              # FP32 columns read, BF16 copies written
        ns_bytes = 4.0 * p.n_rows * (p.n_candidates + kept_per_round) + 8.0 * p.n_rows
        moved_bytes = 4.0 * p.n_rows * window + 8.0 * p.n_rows
    else:
        nnz_col = p.nnz / p.n_cols
        if step_ms["walk_ms"] >= step_ms["gram_ms"]:
            # dominant: the cooperative on-demand walk; every kept candidate's column is merged with every later
            # candidate not yet blocked (at most all examined ones): <= 2 nnz_col - 1 compare steps per merge
            kernel = "k_walk_csc"
            ops = kept_per_round * examined_per_round * (2.0 * nnz_col - 1.0)
            ms = step_ms["walk_ms"]
        else:
            # dominant: the inner products of the window's pairs that share a row
            kernel = "k_csc_bucket_dots"
            ops = 0.5 * window * (window - 1) * (nnz_col * nnz_col / p.n_rows) * (2.0 * nnz_col - 1.0)
            ms = step_ms["gram_ms"]
        peak = 148 * 128 * peaks["sm_max_mhz"] * 1e6 / 1e12        # integer / FP32 lanes x clock, T op/s
        achieved = ops / (ms * 1e-3) / 1e12
        out["roofline"] = {
            "kernel": kernel, "bound": "alu", "achieved": achieved, "peak": peak, "unit": "Tcompare/s",
            "frac": achieved / peak, "traffic": NCU_TRAFFIC.get((workload, kernel)), "window": window, "launch_ms": ms,
            "algorithmic_ops_per_launch": ops,
            "peak_source": "148 SMs x 128 lanes x max SM clock: one merge step (compare + advance) per lane per cycle",
            "note": "inner products of sparse columns counted as sorted-list merge steps, over a few MB of columns: bound by "
                    "dependent loads and barriers, not by HBM"}
        upd_bytes = 8.0 * nnz_col * kept_per_round + 8.0 * p.n_rows
        pack_bytes = 0.0
        ns_bytes = 8.0 * nnz_col * (p.n_candidates + kept_per_round) + 8.0 * p.n_rows
        moved_bytes = 8.0 * nnz_col * examined_per_round + 8.0 * p.n_rows
    hbm = peaks["hbm_gbs"]
    upd_gbs = upd_bytes / (step_ms["update_ms"] * 1e-3) / 1e9
    out["update_hbm"] = {"achieved": upd_gbs, "peak": hbm, "unit": "GB/s", "frac": upd_gbs / hbm, "bytes_per_round": upd_bytes}
    if pack_bytes:
        g = pack_bytes / (step_ms["pack_ms"] * 1e-3) / 1e9
        out["pack_hbm"] = {"achieved": g, "peak": hbm, "unit": "GB/s", "frac": g / hbm, "bytes_per_round": pack_bytes}
    g = ns_bytes / (ms_per_step * 1e-3) / 1e9
    out["round_hbm"] = {"achieved": g, "peak": hbm, "unit": "GB/s", "frac": g / hbm, "bytes_per_round": ns_bytes,
                        "note": "bytes by the metric's count 4N(P'+P)+8N (CSC: 8 nnz_col (P'+P)+8N) / round time; the "
                                "candidate window reads only a fraction of them"}
    g = moved_bytes / (ms_per_step * 1e-3) / 1e9
    out["round_hbm_moved"] = {"achieved": g, "peak": hbm, "unit": "GB/s", "frac": g / hbm, "bytes_per_round": moved_bytes,
                              "note": "bytes a round has to bring from HBM as built (window or examined columns once, r "
                                      "read and written) / round time"}
    return out


def launches_per_round(p: wl.LassoProblem) -> int:
    """Kernels of the library launched per round of strads_run (its fixed sequence; launches of the whole-list retry
    return at once when the window sufficed)."""
    window = window_of(p)
    if p.layout == wl.DENSE:
        n = 3              # the early draw of the next round: histogram pass, collect pass, ordering
        n += 1             # correction of the early list
        n += 2             # pack, window Gram (screen + cluster split-K + recheck + walk)
        n += 1             # update
        if window < p.n_candidates:
            # retry branch: walk kernel on the window (if the Gram's last CTA left it the job), pack, screen, recheck, 3xTF32,
            # walk of the whole list, gated correction of the early list, gated update
            n += 8
        else:
            n += 3         # no window: recheck, 3xTF32 fallback, walk kernel
        return n
    n = 3 + 3 + 1 + 3      # draw; bucket fill, bucket dots, all-pairs fallback; walk; dot, scatter, apply
    if window < p.n_candidates:
        n += 1             # cooperative on-demand walk
    return n


def measure(workload: str, args, device, rank: int, world: int, dist_ok: bool, peaks: dict, with_cpu: float,
            with_round_robin: bool) -> dict:
    from paper_1312_5766_b200 import binding
    cfg = dict(wl.CONFIGS[workload], name=workload)
    if args.n_cols:
        cfg["n_cols"] = args.n_cols
        cfg["n_true"] = max(1, cfg["n_true"] * args.n_cols // wl.CONFIGS[workload]["n_cols"])
    p = wl.make_problem(cfg, seed=0, device=device)                # every rank: the same problem, own replica
    p.seed = rank                                                   # ... with its own random stream
    s = binding.StradsLasso.from_problem(p, device=device)
    torch.cuda.synchronize()

    def barrier():
        if dist_ok:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing: REPEATS regions of K rounds after the warm-up ------------------------------
    s.run(args.warmup)
    s.run(GRAPH_ROUNDS + 7)                # whatever W is: every captured launch sequence (8 rounds, and 4, 2, 1 for what is
                                           # left over: 8 + 8 + 4 + 2 + 1 here) has run before the clock starts
    tot0 = s.totals()
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(REPEATS + 1)]
    barrier()
    clocks = ClockSampler(torch.cuda.current_device())
    evs[0].record()
    for r in range(REPEATS):
        s.run(args.steps)                  # strads_run: captured launch sequences replayed, no host synchronisation
        evs[r + 1].record()
    barrier()
    region_ms = [evs[r].elapsed_time(evs[r + 1]) for r in range(REPEATS)]
    clk = clocks.stop()
    ms_local = statistics.median(region_ms)
    tot1 = s.totals()
    n_timed = REPEATS * args.steps
    kept_per_round = (tot1["kept"] - tot0["kept"]) / n_timed
    examined_per_round = (tot1["examined"] - tot0["examined"]) / n_timed
    moving_per_round = (tot1["nonzero"] - tot0["nonzero"]) / n_timed
    # per-step device times: the next rounds of the same run, launched kernel by kernel with events between the steps
    prof_rounds = min(max(args.steps, 100), 500)
    s.profile_begin(prof_rounds)
    s.run(prof_rounds)
    prof = s.profile_end()
    kept_all, ms = aggregate(kept_per_round * args.steps, ms_local, dist_ok, device)
    value = kept_all / (ms * 1e-3)
    objective = s.objective()
    rc, status_bits = s.status()
    step_ms = {k: prof[k] / max(prof["rounds"], 1) for k in ("sample_ms", "pack_ms", "gram_ms", "walk_ms", "update_ms")}
    rec = {
        "value": value, "unit": UNIT, "ms_per_step": ms / args.steps, "steps": args.steps, "repeats": REPEATS,
        "ms_per_step_repeats": [m / args.steps for m in region_ms],
        "config": config_of(p, workload + (f" with J={args.n_cols}" if args.n_cols else ""), world),
        "rounds_per_s": world * args.steps / (ms * 1e-3), "kept_per_round": kept_per_round,
        "examined_per_round": examined_per_round, "moving_per_round": moving_per_round, "objective": objective, "status_bits": status_bits,
        "step_ms": step_ms, "step_ms_rounds": prof["rounds"],
        "step_ms_note": "device time per step over the rounds right after the timed regions, launched kernel by kernel "
                        "with CUDA events between steps and a plain draw; the timed regions replay captured launch "
                        "sequences, in which (dense) the draw of the next round runs beside the Gram on a second stream",
        "sampling_ahead": p.layout == wl.DENSE and p.n_keep <= 4096,
        "clocks": clk,
    }
    rec.update(rooflines(p, workload, step_ms, kept_per_round, examined_per_round, moving_per_round, ms_local / args.steps,
                         peaks))

    # ---- the same workload with S round-robin scheduler threads (blocks of later rounds prepared during updates) ----
    if with_round_robin and args.schedulers > 1 and p.n_candidates * args.schedulers <= p.n_cols:
        S = args.schedulers
        s2 = binding.StradsLasso.from_problem(p, device=device, n_schedulers=S)
        s2.run(max(args.warmup, 2 * 16 * S))           # includes building the captured sequence
        kept0 = s2.totals()["kept"]
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        s2.run(args.steps)
        e1.record()
        barrier()
        rr_kept_all, rr_ms = aggregate(s2.totals()["kept"] - kept0, e0.elapsed_time(e1), dist_ok, device)
        rec["round_robin"] = {"schedulers": S, "value": rr_kept_all / (rr_ms * 1e-3), "unit": UNIT,
                              "ms_per_step": rr_ms / args.steps, "steps": args.steps, "objective": s2.objective(),
                              "status_bits": s2.status()[1],
                              "note": "scheduler s owns the coefficients j mod S == s and dispatches the rounds t mod S == s; "
                                      "results are those of the same rounds run one after another"}
        s2.close()
        del s2
        torch.cuda.empty_cache()

    # ---- end to end: state in pinned host memory, copied in and out every step ---------------------
    e2e_steps = min(args.e2e_steps, args.steps)
    beta_h = s.beta.cpu().pin_memory(); resid_h = s.resid.cpu().pin_memory(); delta_h = s.delta.cpu().pin_memory()
    kept_h = torch.zeros(p.n_keep, dtype=torch.int32).pin_memory()
    dbeta_h = torch.zeros(p.n_keep).pin_memory(); counts_h = torch.zeros(4, dtype=torch.int32).pin_memory()
    for _ in range(3):
        s.round_host(beta_h, resid_h, delta_h, kept_h, dbeta_h, counts_h)
    barrier()
    e2e_kept = 0
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        s.round_host(beta_h, resid_h, delta_h, kept_h, dbeta_h, counts_h)
        e2e_kept += int(counts_h[2])
    torch.cuda.synchronize()
    e2e_kept_all, e2e_ms = aggregate(e2e_kept, (time.perf_counter() - t0) * 1e3, dist_ok, device)
    h2d = 4 * (2 * p.n_cols + p.n_rows)
    rec["e2e"] = {"value": e2e_kept_all / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                  "d2h_bytes_per_step": h2d + 4 * (2 * p.n_keep + 4), "steps": e2e_steps}

    # ---- CPU baseline: the oracle on a bounded sample of the same workload (rank 0, N = 1 only) ----
    rec["cpu_baseline"] = None
    if rank == 0 and world == 1 and with_cpu > 0:
        if host_has_room_for(p):
            X = oracle_inputs(p)
            n2 = s.colnorm2().cpu().numpy().copy()
            state = (s.beta.cpu().numpy().astype(np.float64), s.resid.cpu().numpy().astype(np.float64),
                     s.delta.cpu().numpy().astype(np.float64))
            k, sec, rounds = time_oracle_rounds(p, X, n2, state, s.get_round(), p.n_candidates, p.n_keep, with_cpu)
            rec["cpu_baseline"] = {"value": k / sec, "unit": UNIT, "cores": 1, "kind": "oracle",
                                   "sample": f"{rounds} full oracle rounds of {workload} from the state after the timed "
                                             f"regions ({sec:.1f} s, single thread; host has {os.cpu_count()} cores)"}
            del X
        else:
            rec["cpu_baseline"] = {"value": None, "unit": UNIT, "cores": 1, "kind": "oracle",
                                   "sample": "not run: the host has too little free memory for a copy of the design matrix"}
    rec["gpu_launches"] = launches_per_round(p) * args.steps * REPEATS
    s.close()
    del s, p
    torch.cuda.empty_cache()
    return rec


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="c3")
    ap.add_argument("--sparse-leg", default="c5", help="second workload timed in the same run and reported under its own key "
                                                       "(none: skip)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=200)
    ap.add_argument("--cpu-baseline-seconds", type=float, default=15.0)
    ap.add_argument("--schedulers", type=int, default=4,
                    help="also time the same workload with this many round-robin scheduler threads (0: skip)")
    ap.add_argument("--n-cols", type=int, default=0,
                    help="profiling aid: same workload with fewer columns J (keeps N, P', P), so that a "
                         "multi-pass ncu capture holds less device memory")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank != 0:
            return
        device = f"cuda:{local_rank}" if torch.cuda.is_available() else "cpu"
        print(json.dumps(run_reference(args, device)), flush=True)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (the library has no CPU path)")
    torch.cuda.set_device(local_rank)
    device = f"cuda:{local_rank}"
    dist_ok = world > 1
    if dist_ok:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(device))

    peaks = measured_peaks()
    main_rec = measure(args.workload, args, device, rank, world, dist_ok, peaks, args.cpu_baseline_seconds, True)
    leg = None
    if args.sparse_leg != "none" and args.sparse_leg != args.workload and not args.n_cols:
        leg = measure(args.sparse_leg, args, device, rank, world, dist_ok, peaks, min(args.cpu_baseline_seconds, 6.0), False)
    if rank == 0:
        line = {"metric": METRIC, "value": main_rec.pop("value"), "unit": main_rec.pop("unit"), "n_gpus": world,
                "steps": main_rec.pop("steps"), "warmup": args.warmup, "ms_per_step": main_rec.pop("ms_per_step"),
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": main_rec.pop("config")}
        line.update(main_rec)
        if leg is not None:
            line[args.sparse_leg] = leg
            line["gpu_launches"] += leg["gpu_launches"]
        print(json.dumps(line), flush=True)
    if dist_ok:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
