#!/usr/bin/env python
"""Benchmark of the CAT hot path: one step = cat_fit (all Lloyd rounds, final pass,
gamma/beta solve) + cat_apply over one synthetic workload.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]

Prints ONE JSON line (rank 0).  `value` is rows through the hot path per second:
(fit rows x (iters + 1) assignment passes + apply rows) / step time, summed over
ranks; `apply_rows_per_s` and `fit_s_per_lloyd_iter` give the two quantities
separately (a Lloyd iteration = (fit time - time of the same fit with 0 rounds) / rounds).  Inputs are resident in HBM before the timed region; `e2e` repeats the
step through the host-buffer entry points with the copies inside the timed region.
With --impl reference the CPU oracle is timed on a bounded sample of the same
workload (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2509_26277_b200 import workloads as W

# dram__bytes_read.sum + dram__bytes_write.sum of the fused inference kernel per row at D = 1024, K = 256
# (the ncu capture summarised in profiles/; None while no capture of the current kernel exists)
APPLY_DRAM_BYTES_PER_ROW = 10658.0

METRIC = "CAT rows/s through the hot path (fit row-passes + apply rows); see apply_rows_per_s, fit_s_per_lloyd_iter"
UNIT = "rows/s"


def measured_peaks():
    """(HBM GB/s, dense bf16 TFLOP/s of a kernel timed alone, source)."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return float(p["hbm_gbs"]), float(p["bf16_tflops"]), "measured"
    return 6650.0, 1590.0, "fallback"


def cpu_model():
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("model name"):
                return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


class ClockSampler:
    """nvidia-smi clock and throttle-reason samples while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100", "-i", str(self.index)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def row_passes(n_fit, iters, n_apply):
    return n_fit * (iters + 1) + n_apply


# ---------------------------------------------------------------------------------------
# reference arm: the CPU oracle on a bounded sample
# ---------------------------------------------------------------------------------------

def oracle_sample(config: int):
    """A bounded sample of workload `config` for the CPU oracle: same D, K and value
    recipe, fewer rows and ONE Lloyd round (+ final pass) so a step takes seconds."""
    sp = W.spec(config)
    terms_budget = 2.0e11                     # (row, centroid, column) distance terms per step
    per_row = sp["K"] * sp["D"]
    n_fit = int(min(sp["N_fit"], max(sp["K"], terms_budget / 3 / per_row)))
    n_apply = int(min(sp["N_apply"], max(1, terms_budget / 3 / per_row)))
    if config == 4:
        # fit and apply samples come from the head of one generated matrix
        w = W.gaussian_mixture(sp["name"], 4, sp["seed"], max(n_fit, n_apply), sp["D"], 256, n_fit,
                               sp["K"], sp["iters"], "cpu")
    else:
        scale = max(n_fit / sp["N_fit"], n_apply / sp["N_apply"])
        w = W.make(config, device="cpu", rows_scale=min(1.0, scale * 1.0001))
    n_fit = min(n_fit, w.N_fit)
    n_apply = min(n_apply, w.N_apply)
    return w, n_fit, n_apply, 1


def oracle_step(O, w, n_fit, n_apply, iters):
    res = O.fit(w.Yq_fit[:n_fit].numpy(), w.Yfp_fit[:n_fit].numpy(), w.K, iters)
    O.apply(w.Yq_apply[:n_apply].numpy(), res.centroids, res.gamma, res.beta)


def time_oracle(config: int, steps: int, warmup: int, threads: int = 0, shrink: float = 1.0):
    """threads = 0: all cores; shrink < 1 cuts the sample (the single-thread figure)."""
    from oracle import cat_oracle as O
    w, n_fit, n_apply, iters = oracle_sample(config)
    all_threads = O.num_threads()
    if threads:
        O.set_num_threads(threads)
    n_fit = max(w.K, int(n_fit * shrink))
    n_apply = max(1, int(n_apply * shrink))
    for _ in range(warmup):
        oracle_step(O, w, n_fit, n_apply, iters)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle_step(O, w, n_fit, n_apply, iters)
    dt = (time.perf_counter() - t0) / steps
    rows = row_passes(n_fit, iters, n_apply)
    sample = (f"config {config} recipe, D={w.D} K={w.K}: fit on {n_fit} rows with {iters} Lloyd round "
              f"+ final pass, apply on {n_apply} rows")
    used = O.num_threads()
    if threads:
        O.set_num_threads(all_threads)
    return rows / dt, dt, used, sample


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    value, dt, cores, sample = time_oracle(args.config, args.steps, args.warmup)
    sp = W.spec(args.config)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"config {args.config} ({sp['name']}), bounded sample", "D": sp["D"], "K": sp["K"]},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                         "cpu_model": cpu_model()},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------
# CUDA arm
# ---------------------------------------------------------------------------------------

def run_cuda(args):
    import torch.distributed as dist
    from paper_2509_26277_b200 import binding as B
    from paper_2509_26277_b200 import sharded

    if args.tc_min_k is not None:
        B.cat_set_tensor_core_min_k(args.tc_min_k)
    if args.small_kernels is not None:
        B.cat_set_small_problem_kernels(args.small_kernels)
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    B.lib()

    # cpu baseline first (before the big device allocations), rank 0 at N=1 only
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import cat_oracle as _O
        _O.assign(np.zeros((4, 4), np.float32), np.zeros((2, 4), np.float32))   # load the checker
        v, dt, cores, sample = time_oracle(args.config, 1, 0)
        v1, dt1, _, _ = time_oracle(args.config, 1, 0, threads=1, shrink=1.0 / 16)
        cpu_baseline = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                        "seconds": dt, "cpu_model": cpu_model(),
                        "single_thread": {"value": v1, "unit": UNIT, "seconds": dt1, "sample": "1/16 of the rows above"}}

    # each rank holds its own shard of the same recipe (weak scaling): seed offset per rank
    sp = W.spec(args.config)
    w = W.make(args.config, device=device, rows_scale=args.rows_scale, seed_offset=100 * rank)
    N_fit, N_apply, D, K, iters = w.N_fit, w.N_apply, w.D, w.K, w.iters
    Yq_fit, Yfp_fit, Yq_apply = w.Yq_fit, w.Yfp_fit, w.Yq_apply

    C = torch.empty((K, D), dtype=torch.float32, device=device)
    G = torch.empty_like(C)
    Bt = torch.empty_like(C)
    labels = torch.empty((N_fit,), dtype=torch.int32, device=device)
    out = torch.empty((N_apply, D), dtype=torch.float32, device=device)
    ws_fit = B.workspace("fit", N_fit, D, K, device)
    ws_apply = B.workspace("apply", N_apply, D, K, device)

    shard_backend = sharded.CudaBackend() if world > 1 else None

    def fit(rounds):
        """cat_fit on one GPU; on several, the row-sharded fit (same kernels, one all-reduce per round)."""
        if world == 1:
            B.cat_fit_into(Yq_fit, Yfp_fit, K, rounds, C, G, Bt, labels, ws_fit)
            return C, G, Bt
        c, g, b, _ = sharded.fit_sharded(Yq_fit, Yfp_fit, K, rounds, backend=shard_backend)
        return c, g, b

    def step():
        c, g, b = fit(iters)
        B.cat_apply(Yq_apply, c, g, b, out=out, ws=ws_apply)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()

    stream = torch.cuda.current_stream()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    launches0 = B.cat_kernel_launches()
    barrier()
    t_wall0 = time.perf_counter()
    for i in range(args.steps):
        ev[i][0].record(stream)
        c, g, b = fit(iters)
        ev[i][1].record(stream)
        B.cat_apply(Yq_apply, c, g, b, out=out, ws=ws_apply)
        ev[i][2].record(stream)
    barrier()
    t_wall = time.perf_counter() - t_wall0
    launches = B.cat_kernel_launches() - launches0
    # A Lloyd round = (fit with `iters` rounds - fit with 1 round) / (iters - 1), the same way at every
    # number of GPUs: the fp16 copy, the first round (every row enters the sums), the final assignment,
    # the moments and the solve drop out of the difference.
    fit1_ms = None
    if iters > 1:
        e0 = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        fit(1)
        barrier()
        e0[0].record(stream)
        for _ in range(args.steps):
            fit(1)
        e0[1].record(stream)
        barrier()
        fit1_ms = e0[0].elapsed_time(e0[1]) / args.steps
        fit(iters)   # leave the fitted model in place
    rep_fit = B.cat_workspace_report(ws_fit) if world == 1 else None
    rep_apply = B.cat_workspace_report(ws_apply)
    clocks = sampler.stop() if rank == 0 else None

    fit_ms = [ev[i][0].elapsed_time(ev[i][1]) for i in range(args.steps)]
    apply_ms = [ev[i][1].elapsed_time(ev[i][2]) for i in range(args.steps)]
    total_ms = ev[0][0].elapsed_time(ev[-1][2])
    t = torch.tensor([total_ms, sum(fit_ms), sum(apply_ms), fit1_ms or 0.0], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    total_ms, fit_total_ms, apply_total_ms, fit1_max = t.tolist()
    if fit1_ms is not None:
        fit1_ms = fit1_max
    ms_per_step = total_ms / args.steps
    fit_ms_step = fit_total_ms / args.steps
    apply_ms_step = apply_total_ms / args.steps

    rows_step = row_passes(N_fit, iters, N_apply) * world
    value = rows_step / (ms_per_step * 1e-3)
    peak, peak_tf, peak_src = measured_peaks()

    # dominant kernel: the fused assign+affine kernel of cat_apply (one launch per step).
    # algorithmic bytes per launch = read N*D fp32 + write N*D fp32.
    # DRAM counter traffic of that kernel (ncu capture at 262 144 rows of this recipe, scaled by
    # the rows: see profiles/): only meaningful for the shape it was taken on.
    traffic = APPLY_DRAM_BYTES_PER_ROW * N_apply if (args.config == 4 and APPLY_DRAM_BYTES_PER_ROW) else None
    apply_bytes = 2.0 * N_apply * D * 4
    apply_gbs = apply_bytes / (apply_ms_step * 1e-3) / 1e9
    if fit1_ms is not None:
        lloyd_ms = max(fit_ms_step - fit1_ms, 0.0) / (iters - 1)
    else:
        lloyd_ms = fit_ms_step / (iters + 1)
    # What a round moves and computes.  With K at or above the tensor threshold and D % 8 == 0 the assignment reads the fp16 copy of
    # the rows (N D 2 bytes, plus labels) and is paced by the tensor cores (2 N K D flop); otherwise it
    # reads the fp32 rows.  The algorithmic figure (one fp32 read of Yq per round) is reported beside it.
    fp16_rounds = (K >= B.cat_get_tensor_core_min_k() and D % 8 == 0 and K <= 256 and B.cat_tensor_path_available())
    lloyd_alg_gbs = 1.0 * N_fit * D * 4 / (lloyd_ms * 1e-3) / 1e9
    lloyd_moved_gbs = (N_fit * D * (2.0 if fp16_rounds else 4.0) + 8.0 * N_fit) / (lloyd_ms * 1e-3) / 1e9
    lloyd_tflops = 2.0 * N_fit * K * D / (lloyd_ms * 1e-3) / 1e12
    # ---- end to end through the host-buffer entry points (copies inside the timed region)
    e2e = None
    if not args.no_e2e:
        try:
            e2e = run_e2e(B, w, device, world, args, barrier)
        except Exception as exc:  # report, do not hide
            e2e = {"value": None, "unit": UNIT, "error": repr(exc)}
        if world > 1 and e2e.get("value") is not None:
            tt = torch.tensor([e2e["seconds_per_step"]], dtype=torch.float64, device=device)
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
            e2e["seconds_per_step"] = float(tt.item())
            e2e["value"] = rows_step / e2e["seconds_per_step"]

    parity = None
    if args.check and rank == 0 and world == 1:
        parity = run_check(B, w, C, G, Bt, labels, out)
        # the library's own per-assignment record (extra passes over Yq: outside the timed region)
        d = B.cat_fit(Yq_fit, Yfp_fit, K, iters, want_labels=False, want_diag=True, ws=ws_fit)[4]
        parity["library_fit_record"] = {"near_tie_rows_per_assignment": d["near_tie_rows"],
                                        "undecided_rows_per_assignment": d["undecided_rows"],
                                        "objective_first": d["objective"][0], "objective_last": d["objective"][-1],
                                        "objective_never_rises": bool(all(b <= a * (1 + 1e-12) for a, b in
                                                                          zip(d["objective"], d["objective"][1:])))}
    form = B.lib().cat_get_apply_column_split()
    apply_kernel = ("apply_h64_kernel (64-row tiles, fp16 operands made in the kernel)"
                    if (form in (0, 64) and K >= B.cat_get_tensor_core_min_k() and K <= 256 and 640 <= D <= 2048
                        and D % 8 == 0 and N_apply >= 4096) else "assign_tc_kernel<affine> / assign_kernel<affine>")
    if ((B.cat_get_small_problem_kernels() & 1) and D in (32, 64, 128) and B.cat_get_tensor_core_min_k() <= K <= 128
            and N_apply >= 128):
        apply_kernel = "small_kernel<inference> (one persistent launch: TF32 scores, in-kernel exact pass, affine from the staged tile)"
    small_fit = ((B.cat_get_small_problem_kernels() & 2) and D in (32, 64, 128) and K * D <= 4096
                 and B.cat_get_tensor_core_min_k() <= K <= 128 and N_fit >= 128)
    if small_fit:
        # all rounds in one persistent launch: a round reads the fp32 rows once (TF32 scores from the staged tile)
        roofline_fit = {"bound": "hbm", "kernel": "one Lloyd round inside small_kernel<fit> (one cooperative launch for the "
                        "whole fit: TF32 scores, in-kernel exact pass, fp64 sums in shared memory, ordered grid-wide combine)",
                        "achieved": lloyd_alg_gbs, "peak": peak, "unit": "GB/s", "frac": lloyd_alg_gbs / peak,
                        "peak_source": peak_src, "tflops": lloyd_tflops}
    elif fp16_rounds:
        # paced by the tensor cores: flop of the distance contraction against the measured dense peak
        roofline_fit = {"bound": "tensor", "kernel": "one Lloyd round of cat_fit (assign_tc_kernel<labels, pair, fp16> + exact "
                        "pass + changed-row sums + centroid update)", "achieved": lloyd_tflops, "peak": peak_tf,
                        "unit": "TFLOP/s", "frac": lloyd_tflops / peak_tf, "peak_source": peak_src,
                        "hbm_moved_gbs": lloyd_moved_gbs, "hbm_moved_frac": lloyd_moved_gbs / peak,
                        "hbm_algorithmic_fp32_gbs": lloyd_alg_gbs, "hbm_algorithmic_fp32_frac": lloyd_alg_gbs / peak}
    else:
        roofline_fit = {"bound": "hbm", "kernel": "one Lloyd round of cat_fit (assign_kernel, fp32 pipes + exact pass + "
                        "changed-row sums + centroid update)", "achieved": lloyd_alg_gbs, "peak": peak, "unit": "GB/s",
                        "frac": lloyd_alg_gbs / peak, "peak_source": peak_src, "tflops": lloyd_tflops}
    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"config {args.config} ({sp['name']})", "N_fit": N_fit, "N_apply": N_apply,
                       "D": D, "K": K, "iters": iters, "rows_scale": args.rows_scale,
                       "l2": "inputs larger than L2" if N_apply * D * 4 > 126e6 else "L2-resident inputs",
                       "parallelism": f"rows x{world}", "tensor_core_min_k": B.cat_get_tensor_core_min_k(),
                       "small_kernels": B.cat_get_small_problem_kernels()},
            "apply_rows_per_s": N_apply * world / (apply_ms_step * 1e-3),
            "fit_s_per_lloyd_iter": lloyd_ms * 1e-3,
            "fit_ms": fit_ms_step, "fit_one_round_ms": fit1_ms, "apply_ms": apply_ms_step,
            "wall_s": t_wall,
            "roofline": {"bound": "hbm", "kernel": apply_kernel + ("" if apply_kernel.startswith("small_kernel") else " (the one kernel of cat_apply besides the exact pass)"),
                         "achieved": apply_gbs, "peak": peak, "unit": "GB/s", "frac": apply_gbs / peak,
                         "peak_source": peak_src, "traffic": traffic},
            "roofline_fit": roofline_fit,
            "exact_pass_rows": {"apply": rep_apply["refined_rows_last"],
                                "fit_all_assignments": rep_fit["refined_rows_total"] if rep_fit else None},
            "parity": parity,
            "cpu_baseline": cpu_baseline,
            "e2e": e2e,
            "gpu_launches": int(launches),
            "clocks": clocks,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_check(B, w, C, G, Bt, labels, out):
    """The model bench just fitted and the outputs it just wrote, against the CPU oracle (outside every
    timed region).  Labels must match except inside the 1e-6 near-tie band; gamma/beta are compared with
    the oracle's closed form for the library's labels; outputs with the oracle's affine map."""
    from oracle import cat_oracle as O
    rng = np.random.default_rng(0)
    N_fit, N_apply, D, K = w.N_fit, w.N_apply, w.D, w.K
    budget = 4.0e10                                  # (row, centroid, column) terms the oracle may spend per part
    n_s = int(min(N_fit, max(256, budget / (K * D))))
    idx = np.arange(N_fit) if n_s == N_fit else np.sort(rng.choice(N_fit, n_s, replace=False))
    hC, hG, hB = C.cpu().numpy(), G.cpu().numpy(), Bt.cpu().numpy()
    t_idx = torch.from_numpy(idx).to(C.device)
    lab, best, second = O.assign(w.Yq_fit[t_idx].cpu().numpy(), hC)
    near = (second - best) <= 1e-6 * second
    glab = labels[t_idx].cpu().numpy()
    res = {"fit_rows_checked": int(len(idx)), "fit_near_tie_rows": int(near.sum()),
           "fit_label_mismatches_outside_band": int(((glab != lab) & ~near).sum())}
    if n_s == N_fit:
        g_want, b_want = O.solve_gamma_beta(w.Yq_fit.cpu().numpy(), w.Yfp_fit.cpu().numpy(), labels.cpu().numpy(), K)
        tol = lambda a, b: float(np.max(np.abs(a - b) / (1e-6 + 1e-5 * np.abs(b))))
        res["gamma_worst_over_tolerance"] = tol(hG.astype(np.float64), g_want)
        res["beta_worst_over_tolerance"] = tol(hB.astype(np.float64), b_want)
    n_a = int(min(N_apply, max(256, budget / (K * D))))
    aidx = np.arange(N_apply) if n_a == N_apply else np.sort(rng.choice(N_apply, n_a, replace=False))
    ta = torch.from_numpy(aidx).to(C.device)
    want, alab, best, second = O.apply(w.Yq_apply[ta].cpu().numpy(), hC, hG, hB)
    near = (second - best) <= 1e-6 * second
    got = out[ta].cpu().numpy().astype(np.float64)
    ok_rows = ~near
    err = np.abs(got[ok_rows] - want[ok_rows]) / (1e-6 + 1e-5 * np.abs(want[ok_rows]))
    res.update({"apply_rows_checked": int(len(aidx)), "apply_near_tie_rows": int(near.sum()),
                "apply_worst_over_tolerance": float(err.max()) if err.size else 0.0,
                "apply_max_abs_err": float(np.abs(got[ok_rows] - want[ok_rows]).max()) if err.size else 0.0})
    res["ok"] = bool(res["fit_label_mismatches_outside_band"] == 0 and res["apply_worst_over_tolerance"] <= 1.0
                     and res.get("gamma_worst_over_tolerance", 0.0) <= 1.0 and res.get("beta_worst_over_tolerance", 0.0) <= 1.0)
    return res


def run_e2e(B, w, device, world, args, barrier):
    """Same step through cat_fit_host + cat_apply_host: pinned host inputs/outputs,
    H2D and D2H inside the timed region."""
    N_fit, N_apply, D, K, iters = w.N_fit, w.N_apply, w.D, w.K, w.iters
    need = (2 * N_fit + 2 * N_apply) * D * 4
    avail = os.sysconf("SC_AVPHYS_PAGES") * os.sysconf("SC_PAGE_SIZE")
    if need > 0.5 * avail:
        return {"value": None, "unit": UNIT, "error": f"host buffers need {need >> 30} GiB, {avail >> 30} GiB free"}
    hq_fit = torch.empty((N_fit, D), dtype=torch.float32, pin_memory=True)
    hf_fit = torch.empty((N_fit, D), dtype=torch.float32, pin_memory=True)
    hq_apply = torch.empty((N_apply, D), dtype=torch.float32, pin_memory=True)
    h_out = torch.empty((N_apply, D), dtype=torch.float32, pin_memory=True)
    hq_fit.copy_(w.Yq_fit)
    hf_fit.copy_(w.Yfp_fit)
    hq_apply.copy_(w.Yq_apply)
    hC, hG, hB = (torch.empty((K, D), dtype=torch.float32, pin_memory=True) for _ in range(3))
    ws_f = B.workspace("fit_host", N_fit, D, K, device)
    ws_a = B.workspace("apply_host", N_apply, D, K, device)

    def step():
        B.cat_fit_host(hq_fit, hf_fit, K, iters, hC, hG, hB, None, device=device, ws=ws_f)
        B.cat_apply_host(hq_apply, hC, hG, hB, h_out, None, device=device, ws=ws_a)

    step()  # warm-up (page-locks, side streams)
    barrier()
    steps = max(1, min(args.steps, 3))
    s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s.record()
    for _ in range(steps):
        step()
    e.record()
    barrier()
    sec = s.elapsed_time(e) * 1e-3 / steps
    rows = row_passes(N_fit, iters, N_apply) * world
    h2d = (2 * N_fit + N_apply) * D * 4 + 3 * K * D * 4
    d2h = N_apply * D * 4 + 3 * K * D * 4
    return {"value": rows / sec, "unit": UNIT, "seconds_per_step": sec, "steps": steps,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "apply_rows_per_s": None}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=4)
    ap.add_argument("--rows-scale", type=float, default=1.0, dest="rows_scale")
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--tensor-core-min-k", type=int, default=None, dest="tc_min_k",
                    help="kernel selection: tensor-core scores for K >= this (library default 32)")
    ap.add_argument("--small-kernels", type=int, default=None, dest="small_kernels",
                    help="kernel selection: mask of the persistent small-shape kernels (library default 3)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--check", action="store_true",
                    help="after timing, compare the fitted model and the apply outputs with the CPU oracle "
                         "(all rows where it finishes in seconds, a seeded row sample otherwise) and report "
                         "near-tie counts and the largest deviations")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "cuda":
        print(f"note: --warmup {args.warmup} < 3", file=sys.stderr)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
