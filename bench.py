#!/usr/bin/env python
"""Benchmark of the scheduled-Lasso round on B200: coordinate updates per second.

A step is one whole round (sample -> Gram -> greedy filter -> update) of the dense 10,000 x 100,000
configuration ("c2"), on synthetic data generated on the device from a seed.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--impl ours|reference]

Prints ONE JSON line.  `--impl reference` times the FP64 CPU oracle instead (rank 0 only).
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
# DRAM bytes (read + write) per launch of the window-Gram kernels from ncu (dram__bytes_read.sum +
# dram__bytes_write.sum; profiles/ncu_full_round_kernels_c2_J20000.md), keyed by (workload, window).  The capture was made
# with J cut to 20,000; the window kernels read the packed window only, so their traffic does not depend on J.
GRAM_WINDOW_TRAFFIC = {("c2", 512): 10.3e6}


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


def oracle_inputs(p: wl.LassoProblem):
    """Host copies of the device arrays for the CPU oracle (the same FP32 bits)."""
    import oracle
    if p.layout == wl.DENSE:
        X = oracle.Matrix.dense(p.values.cpu().numpy(), n_rows=p.n_rows)
    else:
        X = oracle.Matrix.csc(p.n_rows, p.n_cols, p.values.cpu().numpy(), p.row_idx.cpu().numpy(),
                              p.col_ptr.cpu().numpy())
    return X


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
        "config": {"workload": args.workload, "n_rows": p.n_rows, "n_cols": p.n_cols, "n_candidates": n_cand,
                   "n_keep": n_keep},
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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="c2")
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

    from paper_1312_5766_b200 import binding
    cfg = dict(wl.CONFIGS[args.workload], name=args.workload)
    if args.n_cols:
        cfg["n_cols"] = args.n_cols
        cfg["n_true"] = max(1, cfg["n_true"] * args.n_cols // wl.CONFIGS[args.workload]["n_cols"])
    p = wl.make_problem(cfg, seed=0, device=device)                # every rank: the same problem, own replica
    p.seed = rank                                                   # ... with its own random stream
    s = binding.StradsLasso.from_problem(p, device=device)
    torch.cuda.synchronize()

    def barrier():
        if dist_ok:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing: K rounds after W warm-up rounds -------------------------------------
    s.run(args.warmup)
    kept_before = s.totals()["kept"]
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    clocks = ClockSampler(local_rank)
    ev0.record()
    s.run(args.steps)                      # strads_run: one captured round replayed K times
    ev1.record()
    barrier()
    ms_local = ev0.elapsed_time(ev1)
    tot = s.totals()
    kept_local = tot["kept"] - kept_before
    # per-step device times: the next rounds of the same run, launched kernel by kernel with events between the steps
    prof_rounds = min(args.steps, 500)
    s.profile_begin(prof_rounds)
    s.run(prof_rounds)
    prof = s.profile_end()
    clk = clocks.stop()
    kept_all, ms = aggregate(kept_local, ms_local, dist_ok, device)
    value = kept_all / (ms * 1e-3)
    objective = s.objective()
    rc, status_bits = s.status()

    # ---- roofline -----------------------------------------------------------------------------------------
    peaks = measured_peaks()
    step_ms = {k: prof[k] / max(prof["rounds"], 1) for k in ("sample_ms", "pack_ms", "gram_ms", "walk_ms", "update_ms")}
    kept_per_round = kept_local / args.steps
    # the Gram is formed on a leading window of the candidates (the library's rule: 1.5 P + 128 rounded up to 128,
    # used when at most half the list)
    window = (p.n_keep + p.n_keep // 2 + 128 + 127) // 128 * 128
    if 2 * window > p.n_candidates:
        window = p.n_candidates
    if p.layout == wl.DENSE:
        # dominant kernel: the tensor-core Gram of the window (k_gram_dense_tc screen + its split-K reduce and the
        # exact recheck, timed together).  Algorithmic flops W(W-1)N: upper triangle, 2 flop per multiply-add.
        flops = float(window) * (window - 1) * p.n_rows
        achieved = flops / (step_ms["gram_ms"] * 1e-3) / 1e12
        peak = peaks["bf16_tflops"]                          # the screen multiplies BF16 roundings of the columns
        roofline = {"kernel": "k_gram_dense_tc<screen> (+ k_gram_reduce, whose last CTA rechecks the open pairs)", "bound": "tensor",
                    "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                    "traffic": GRAM_WINDOW_TRAFFIC.get((args.workload, window)),
                    "window": window, "launch_ms": step_ms["gram_ms"],
                    "peak_source": f"{peaks['source']} BF16 burst (the screen's operands are BF16; pairs it cannot call "
                                   "are decided exactly in FP64); the kernel is timed alone between events"}
    else:
        # dominant kernel: the pair merges of the window (k_gram_csc); bytes: each window column once
        nnz_col = p.nnz / p.n_cols
        byts = 8.0 * nnz_col * window
        achieved = byts / (step_ms["gram_ms"] * 1e-3) / 1e9
        roofline = {"kernel": "k_gram_csc", "bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"],
                    "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "traffic": None, "window": window,
                    "launch_ms": step_ms["gram_ms"], "peak_source": peaks["source"],
                    "note": "a few MB of columns against ~1e6 sorted-list merges: bound by ALU/latency, not by HBM"}
    # streaming kernels against the HBM roofline: pack (window columns read + written) and update (kept columns once
    # + r read and written)
    if p.layout == wl.DENSE:
        upd_bytes = 4.0 * p.n_rows * kept_per_round + 8.0 * p.n_rows + 16.0 * kept_per_round
        pack_bytes = 6.0 * p.n_rows * window              # FP32 columns read, BF16 copies written
    else:
        upd_bytes = 8.0 * (p.nnz / p.n_cols) * kept_per_round + 8.0 * p.n_rows
        pack_bytes = 0.0
    upd_gbs = upd_bytes / (step_ms["update_ms"] * 1e-3) / 1e9
    pack_gbs = pack_bytes / (step_ms["pack_ms"] * 1e-3) / 1e9 if pack_bytes else None
    # the metric's own byte count per round (all P' candidate columns + kept columns + r twice) over the round time:
    # what a round would have to stream if it formed the whole Gram; the window avoids most of it
    if p.layout == wl.DENSE:
        ns_bytes = 4.0 * p.n_rows * (p.n_candidates + kept_per_round) + 8.0 * p.n_rows
    else:
        ns_bytes = 8.0 * (p.nnz / p.n_cols) * (p.n_candidates + kept_per_round) + 8.0 * p.n_rows
    round_gbs = ns_bytes / (ms_local / args.steps * 1e-3) / 1e9

    # ---- the same workload with S round-robin scheduler threads (blocks of later rounds prepared during updates) ----
    round_robin = None
    if args.schedulers > 1 and p.n_candidates * args.schedulers <= p.n_cols:
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
        rr_ms_local = e0.elapsed_time(e1)
        rr_kept_all, rr_ms = aggregate(s2.totals()["kept"] - kept0, rr_ms_local, dist_ok, device)
        round_robin = {"schedulers": S, "value": rr_kept_all / (rr_ms * 1e-3), "unit": UNIT, "ms_per_step": rr_ms / args.steps,
                       "steps": args.steps, "objective": s2.objective(), "status_bits": s2.status()[1],
                       "note": "scheduler s owns the coefficients j mod S == s and dispatches the rounds t mod S == s; "
                               "results are those of the same rounds run one after another"}
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
    e2e_ms_local = (time.perf_counter() - t0) * 1e3
    e2e_kept_all, e2e_ms = aggregate(e2e_kept, e2e_ms_local, dist_ok, device)
    h2d = 4 * (2 * p.n_cols + p.n_rows)
    d2h = h2d + 4 * (2 * p.n_keep + 4)

    # ---- CPU baseline: the oracle on a bounded sample of the same workload (rank 0, N = 1 only) ----
    cpu_baseline = None
    if rank == 0 and world == 1 and args.cpu_baseline_seconds > 0:
        import oracle
        X = oracle_inputs(p)
        n2 = s.colnorm2().cpu().numpy().copy()
        state = (s.beta.cpu().numpy().astype(np.float64), s.resid.cpu().numpy().astype(np.float64),
                 s.delta.cpu().numpy().astype(np.float64))
        k, sec, rounds = time_oracle_rounds(p, X, n2, state, s.get_round(), p.n_candidates, p.n_keep,
                                            args.cpu_baseline_seconds)
        cpu_baseline = {"value": k / sec, "unit": UNIT, "cores": 1, "kind": "oracle",
                        "sample": f"{rounds} full oracle rounds of {args.workload} from the state after the timed "
                                  f"region ({sec:.1f} s, single thread; host has {os.cpu_count()} cores)"}

    # kernels launched per round (the library's fixed sequence; launches of the whole-list retry return at once when
    # the window sufficed): sampler hist + collect (winners grouped by histogram bin) + ordering (ranks inside the groups);
    # dense Gram of n candidates: pack, screen, split-K reduce (few tiles only), recheck, and a 3xTF32 launch unless a
    # retry follows; CSC Gram: bucket fill, bucket pairs, pair bits, all-pairs fallback; walk 1; update: dense 1 (the
    # pack kernel has formed the changes), CSC 3
    def gram_launches(n, retry_follows):
        if p.layout != wl.DENSE:
            return 4
        nt = (n + 127) // 128
        tiles = nt * (nt + 1) // 2
        split = tiles * 2 <= 148
        if retry_follows and split:
            return 3                   # pack, screen, reduce (whose last CTA also rechecks the open pairs)
        return 3 + (1 if split else 0) + (0 if retry_follows else 1)
    launches_per_round = 2 + 1 + (1 if p.layout == wl.DENSE else 3)
    sampling_ahead = p.layout == wl.DENSE and p.n_keep <= 4096
    if sampling_ahead:
        launches_per_round += 1        # the early list's correction; the early draw itself launches what a plain draw does
    if window < p.n_candidates:
        if sampling_ahead:
            launches_per_round += 1    # the update's gated copy at the end of the retry branch
        launches_per_round += gram_launches(window, True) + 1
        launches_per_round += (gram_launches(p.n_candidates, False) + 1) if p.layout == wl.DENSE else 1
    else:
        launches_per_round += gram_launches(p.n_candidates, False) + 1
    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": args.workload + (f" with J={args.n_cols}" if args.n_cols else ""), "layout": "dense" if p.layout == wl.DENSE else "csc",
                       "n_rows": p.n_rows, "n_cols": p.n_cols, "n_candidates": p.n_candidates, "n_keep": p.n_keep,
                       "rho": p.rho, "eta": p.eta, "lambda": p.lam, "parallelism": f"replicas x{world}",
                       "l2": "design matrix (4 GB for c2) far exceeds L2; every round draws a fresh candidate set"},
            "rounds_per_s": world * args.steps / (ms * 1e-3),
            "kept_per_round": kept_per_round,
            "objective": objective, "status_bits": status_bits,
            "step_ms": step_ms, "step_ms_rounds": prof["rounds"],
            "step_ms_note": "device time per step over the rounds right after the timed region, launched kernel by "
                            "kernel with CUDA events between steps (the timed region itself replays a CUDA graph"
                            + (", in which the draw of the next round runs beside the Gram and walk on a second "
                               "stream, so sample_ms is not on its critical path)" if sampling_ahead else ")"),
            "sampling_ahead": sampling_ahead,
            "roofline": roofline,
            "update_hbm": {"achieved": upd_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                           "frac": upd_gbs / peaks["hbm_gbs"], "bytes_per_round": upd_bytes},
            "pack_hbm": None if pack_gbs is None else {"achieved": pack_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                                      "frac": pack_gbs / peaks["hbm_gbs"], "bytes_per_round": pack_bytes},
            "round_hbm": {"achieved": round_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                          "frac": round_gbs / peaks["hbm_gbs"], "bytes_per_round": ns_bytes,
                          "note": "bytes by the metric's count 4N(P'+P)+8N (CSC: 8 nnz_col (P'+P)+8N) / round time; the "
                                  "candidate window reads only a fraction of them"},
            "cpu_baseline": cpu_baseline,
            "round_robin": round_robin,
            "e2e": {"value": e2e_kept_all / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "steps": e2e_steps},
            "gpu_launches": launches_per_round * args.steps,
            "clocks": clk,
        }
        print(json.dumps(line), flush=True)
    if dist_ok:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
