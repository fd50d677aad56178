#!/usr/bin/env python
"""Benchmark of the PolluxSched optimizer core on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one whole scheduling round of the "large" workload (256 nodes x 8 GPUs, 1024
jobs, 128 x 32 (m, s) grid, population 512, 200 generations): speedup tables, initial
population, and per generation ranking / selection + crossover + perturbation / repair /
fitness, then the best allocation.  The headline value is candidate fitness evaluations
per second over the round.  With N > 1 (torchrun) every rank schedules its own cluster
(independent problems, no data-path collective): weak scaling.

Rank 0 prints ONE JSON line.  Besides the contract keys it carries the per-kernel device
times of the timed region, the roofline of the dominant kernel, and - at N = 1 - two
single-kernel measurements: the goodput sweep (ALU-bound) and the dense fitness kernel on
a chunk of the stress workload (HBM-bound), plus the CPU oracle timed on a bounded sample.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2008_12260_b200 import dist as pdist  # noqa: E402
from paper_2008_12260_b200 import synth  # noqa: E402

METRIC = "ga_candidate_fitness_evals_per_sec"
UNIT = "candidates/s"
FP32_LANES_PER_SM = 128          # CUDA cores per SM (compute capability 10.0)
OPS_PER_POINT = 10               # fp32 lane-ops counted as useful per (job, K, class, m, s) point
HBM_FALLBACK_GBS = 6650.0

# the workload both arms (the CUDA path and the oracle as the reference) are quoted on
CONFIG = {
    "workload": "large: 256 nodes x 8 GPUs, 1024 jobs, grid 128x32, population 512, 200 generations, p=-1, "
                "random current allocation, one scheduling round per step",
    "per_rank": "one independent cluster per rank",
    "arithmetic": "int16 matrices, fp32 tables and fitness on the GPU (the oracle computes in fp64)",
    "l2": "every round rebuilds its 17 MB tables and a fresh population; inside a round the generations work on "
          "the row store (records + indices, about 40 MB), L2-resident by design; the single-kernel sections flush "
          "L2 or stream more than L2 per pass",
}

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the committed ncu
# summaries under profiles/ (not measured in this run); None = the kernel has changed since its
# counters were taken.
# "rows": one dense large-workload generation of the streaming row kernel (227.7 MB read + 233.7 MB
# written: some parent rows are shared by several children and come from L2).
# "fitness_stress": 16 dense stress candidates moved 544.8 + 3.5 MB; every candidate is streamed
# once, so the figure is scaled by candidates / 16 to the chunk that is timed.
# "generation_store": one row-store generation of the large workload (3.4 - 3.6 MB read in
# generations 6 to 8 of a 12-generation round).
NCU_TRAFFIC_BYTES = {"rows": 461.4e6, "fitness_stress_per_candidate": 548.3e6 / 16, "generation_store": 3.5e6}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return float(d["hbm_gbs"]), "measured", float(d.get("sm_max_mhz", 1965.0))
        except Exception:
            pass
    return HBM_FALLBACK_GBS, "fallback", 1965.0


class ClockSampler:
    """nvidia-smi clocks / throttle reasons sampled every 20 ms while the timed region runs (the region
    is about 0.1 s long; the sampler is stopped right after it)."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.proc = None
        self.tmp = None

    def start(self):
        try:
            self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.idx), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "20"], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def lines(self):
        try:
            with open(self.tmp.name) as f:
                return [ln for ln in f.read().splitlines() if ln.count(",") >= 8]
        except Exception:
            return []

    def wait_ready(self, seconds=2.0):
        """Blocks until the sampler has printed its first line (it takes a while to start)."""
        t0 = time.time()
        while self.proc is not None and not self.lines() and time.time() - t0 < seconds:
            time.sleep(0.01)

    def mark(self):
        """Number of samples taken so far: the timed region's samples lie between two marks."""
        return len(self.lines())

    def stop(self, first=0, last=None):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.05)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        all_lines = [ln for ln in self.tmp.read().splitlines() if ln.count(",") >= 8]
        # the samples between the two marks, and the one right after (a region shorter than the
        # sampling interval would otherwise have none)
        chosen = all_lines[first:(None if last is None else max(last, first) + 1)]
        if not chosen or not last:          # (nothing was visible in the file while the region ran: keep all)
            chosen = all_lines
        for line in chosen:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        self.tmp.close()
        os.unlink(self.tmp.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


def large_inputs(rank: int, fair_share):
    """Inputs of the large workload; `fair_share` is the arm's own (K_f, N_f) routine: the
    library's for the CUDA arm, the oracle's for the reference arm."""
    cfg = synth.LARGE
    cl = cfg.cluster()
    jobs = synth.draw_jobs(cfg.num_jobs, cfg.seed + 1000 * rank, cfg.grid_m, cfg.grid_s, cl.k_max,
                           phi_hi=cfg.phi_hi, with_history=True)
    fk, fn = fair_share(cl.node_capacity, cfg.num_jobs, cl.k_max)
    jobs.fair_k = np.full(cfg.num_jobs, fk, np.int32)
    jobs.fair_n = np.full(cfg.num_jobs, fn, np.int32)
    cur = synth.random_feasible_allocation(cl, cfg.num_jobs, cfg.seed + 1000 + rank)
    return cfg, cl, jobs, cur


def distinct_classes(cl) -> int:
    """(K, class) pairs the sweep evaluates per job: K that fit one node, and K >= 2 that
    fit on min(K, n_max) nodes."""
    cap = np.sort(np.maximum(cl.node_capacity.astype(np.int64), 0))[::-1]
    kfit = np.concatenate([[0], np.cumsum(cap)])
    n = 0
    for K in range(1, cl.k_max + 1):
        n += int(K <= kfit[1])
        n += int(cl.n_max >= 2 and K >= 2 and K <= kfit[min(K, cl.n_max, len(cap))])
    return n


def allocation_summary(best, jobs, cl):
    """What the returned allocation looks like (to read best_fitness by): with p = -1 and a floor of
    1e-3 every active job left without GPUs contributes 1000 to the harmonic sum."""
    act = jobs.active.astype(bool)
    K = best.astype(np.int64).sum(1)
    return {"active_jobs": int(act.sum()), "gpus_allocated": int(K[act].sum()), "gpus_in_cluster": int(cl.node_capacity.sum()),
            "share_of_active_jobs_without_gpus": float((K[act] == 0).mean()) if act.any() else 0.0,
            "mean_gpus_of_served_jobs": float(K[act & (K > 0)].mean()) if (act & (K > 0)).any() else 0.0}


def bench_ga_quality(api, torch, dev, stream):
    """Best fitness of the search against the brute-force optimum of Eq. 14 over every feasible
    matrix, on clusters small enough to enumerate (report only: the search is a heuristic)."""
    import itertools

    import oracle

    out = []
    for name, nodes, gpn, J in (("2 nodes x 2 GPUs, 3 jobs", 2, 2, 3), ("2 nodes x 4 GPUs, 2 jobs", 2, 4, 2)):
        cfg = synth.Config("quality", nodes, gpn, J, 40 + J, 16, 8, 32, 100, num_elite=2, mutate_prob=0.2)
        cl = cfg.cluster()
        jobs = cfg.jobs()
        fk, fn = api.fair_share(cl.node_capacity, J, cl.k_max)
        jobs.fair_k = np.full(J, fk, np.int32)
        jobs.fair_n = np.full(J, fn, np.int32)
        _, sp, _ = oracle.build_speedup_table(jobs, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s, want_argmax=False)
        mats = np.array(list(itertools.product(range(gpn + 1), repeat=J * nodes)), np.int16).reshape(-1, J, nodes)
        A = mats.astype(np.int64)
        dist = (A > 0).sum(2) >= 2
        ok = (A.sum(1) <= gpn).all(1) & (((A > 0) & dist[:, :, None]).sum(1) <= 1).all(1)
        fit = oracle.eval_fitness(mats[ok], sp, cl.k_max, cl.n_max, cfg.p, cfg.speedup_floor)
        optimum = float(fit.max())
        sched = api.scheduler_for(cfg, stream=stream.cuda_stream)
        dj = api.DeviceJobs(jobs, dev, torch)
        best = torch.empty((J, nodes), dtype=torch.int16, device=dev)
        bf = torch.zeros(1, dtype=torch.float32, device=dev)
        row = {"cluster": name, "feasible_matrices": int(ok.sum()), "optimum": optimum}
        for gens in (10, 100):
            sched.schedule_round(dj, None, best, bf, round=0, generations=gens)
            sched.sync_status()
            row["best_after_%d_generations" % gens] = float(bf.item())
            row["gap_after_%d_generations" % gens] = 1.0 - float(bf.item()) / optimum
        sched.close()
        out.append(row)
    return out


# ------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    from paper_2008_12260_b200 import api

    rank, local_rank, world = pdist.init("nccl")
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    stream = torch.cuda.Stream(device=dev)      # not the NULL stream: rounds may replay as CUDA graphs
    torch.cuda.set_stream(stream)
    hbm_peak, peak_src, sm_max_mhz = measured_peaks()

    cfg, cl, jobs, cur = large_inputs(rank, api.fair_share)
    G, P, J, NN = cfg.generations, cfg.population, cfg.num_jobs, cfg.num_nodes
    sched = api.scheduler_for(cfg, stream=stream.cuda_stream)
    dj = api.DeviceJobs(jobs, dev, torch)
    d_cur = torch.from_numpy(cur).to(dev)
    d_best = torch.empty((J, NN), dtype=torch.int16, device=dev)
    d_bf = torch.zeros(1, dtype=torch.float32, device=dev)

    def step(rnd):
        sched.schedule_round(dj, d_cur, d_best, d_bf, round=rnd, generations=G)

    for w in range(args.warmup):
        step(w)
    sched.sync_status()
    torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    sampler.start()
    sampler.wait_ready()
    launches0 = sched.launch_count()
    pdist.barrier()
    torch.cuda.synchronize()
    mark0 = sampler.mark()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for k in range(args.steps):
        step(100 + k)
    e1.record(stream)
    torch.cuda.synchronize()
    mark1 = sampler.mark()
    pdist.barrier()
    clocks = sampler.stop(mark0, mark1)
    elapsed_ms = e0.elapsed_time(e1)
    launches = sched.launch_count() - launches0
    sched.sync_status()
    # the same K steps once more with every kernel bracketed by CUDA events (this pass is not
    # the headline: event pairs add a little time and rounds are not replayed as graphs)
    sched.set_kernel_timing(True)
    sched.read_kernel_timing()
    e0.record(stream)
    for k in range(args.steps):
        step(100 + k)
    e1.record(stream)
    torch.cuda.synchronize()
    profiled_ms = e0.elapsed_time(e1)
    kernel_ms = sched.read_kernel_timing()
    sched.set_kernel_timing(False)
    units = float(P) * (G + 1) * args.steps
    value, t_max, u_sum = pdist.throughput(elapsed_ms, units, device=dev)
    # The generation kernel inside the clean region: rounds of G and of G / 2 generations, both
    # replayed as graphs, differ by G / 2 generations (kernel, launch gap and the compaction
    # checks that fall among them) and by nothing else.
    def clean_round_ms(gens):
        for k in range(3):                                  # plain, capture, first replay
            sched.schedule_round(dj, d_cur, d_best, d_bf, round=200 + k, generations=gens)
        torch.cuda.synchronize()
        e0.record(stream)
        for k in range(args.steps):
            sched.schedule_round(dj, d_cur, d_best, d_bf, round=100 + k, generations=gens)
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / args.steps
    half_ms = clean_round_ms(G // 2)
    full_ms = clean_round_ms(G)
    gen_us_clean = 1e3 * (full_ms - half_ms) / (G - G // 2)
    moves = sched.store_moves()

    # ---- end to end through the host-buffer entry point (pinned host memory) -------------
    hj = api.HostJobs(jobs, torch)
    h_cur = torch.from_numpy(cur.copy()).pin_memory()
    h_best = torch.empty((J, NN), dtype=torch.int16).pin_memory()
    h_bf = torch.zeros(1, dtype=torch.float32).pin_memory()
    sched.schedule_round_host(hj, h_cur, h_best, h_bf, round=0, generations=G)
    pdist.barrier()
    t0 = time.perf_counter()
    e0.record(stream)
    for k in range(args.steps):
        sched.schedule_round_host(hj, h_cur, h_best, h_bf, round=100 + k, generations=G)
    e1.record(stream)
    torch.cuda.synchronize()
    e2e_ms = max(e0.elapsed_time(e1), (time.perf_counter() - t0) * 1e3)
    e2e_value, _, _ = pdist.throughput(e2e_ms, units, device=dev)
    h2d = hj.nbytes + h_cur.numel() * 2
    d2h = h_best.numel() * 2 + 4
    assert np.array_equal(h_best.numpy(), d_best.cpu().numpy()), "host and device rounds disagree"

    # ---- per-kernel accounting and the roofline of the dominant kernel --------------------
    pop_bytes = float(P) * J * NN * 2
    algo_bytes = {
        # dense row pass (initial population here): parent rows in, child rows out, per-row flag
        # and summary out; the current allocation (J * NN * 2 bytes) stays in L2, counted once
        "rows": 2 * pop_bytes + P * J * 5 + J * NN * 2,
        # row-store generation: per (candidate, job) a row index in, its 32-byte record, a row
        # index out; fitness out.  Rows that change (about 2 % per generation here: read, written,
        # new record) are data-dependent and NOT counted, so the figure errs low.
        "generation_store": float(P) * J * (4 + 32 + 4) + 4 * P,
    }
    kernels = []
    for name, (ms, n) in sorted(kernel_ms.items(), key=lambda kv: -kv[1][0]):
        if n == 0:
            continue
        k = {"kernel": name, "launches": n, "total_ms": round(ms, 3), "avg_us": round(1e3 * ms / n, 2),
             "share": round(ms / max(sum(v[0] for v in kernel_ms.values()), 1e-9), 4)}
        if name in algo_bytes:
            k["algorithmic_bytes"] = algo_bytes[name]
            k["achieved_gbs"] = round(algo_bytes[name] / (ms / n * 1e-3) / 1e9, 1)
            k["frac_of_hbm_peak"] = round(k["achieved_gbs"] / hbm_peak, 4)
        kernels.append(k)
    dom = next((k for k in kernels if "achieved_gbs" in k), None)
    roofline = None
    if dom and dom["kernel"] == "generation_store":
        # the dominant kernel, timed inside the clean region (see clean_round_ms above); the
        # per-kernel pass only gives the shares
        gbs = dom["algorithmic_bytes"] / (gen_us_clean * 1e-6) / 1e9
        roofline = {"kernel": "generation_store", "bound": "hbm", "achieved": round(gbs, 1), "peak": hbm_peak,
                    "peak_source": "MEASURED_PEAKS.json hbm_gbs" if peak_src == "measured" else "recipe fallback",
                    "unit": "GB/s", "frac": round(gbs / hbm_peak, 4),
                    "traffic": NCU_TRAFFIC_BYTES.get("generation_store"),
                    "algorithmic_bytes_per_launch": dom["algorithmic_bytes"],
                    "avg_launch_us": round(gen_us_clean, 2),
                    "avg_launch_us_how": "(round of %d generations - round of %d) / %d, both replayed as graphs in a "
                                         "clean region: kernel + launch gap + the compaction checks among them"
                                         % (G, G // 2, G - G // 2),
                    "avg_launch_us_with_event_pairs": dom["avg_us"],
                    "launches_per_step": G + 1, "share_of_step": round(gen_us_clean * (G + 1) / (1e3 * t_max / args.steps), 3),
                    "note": "one block evolves one candidate per launch on L2-resident 32-byte records: bound by "
                            "latency and by the L2's rate of 32-byte requests, not by DRAM (the dense operator "
                            "kernel, which is, is reported under dense_generation)",
                    # what the same generation costs on dense matrices (parents read, children written, the
                    # repair's row and column passes: about four population sweeps): the bytes this kernel
                    # exists to avoid.  Reported for scale only; it is NOT the kernel's traffic.
                    "dense_equivalent": {"bytes_per_launch": 4 * pop_bytes,
                                         "floor_us_at_hbm_peak": round(4 * pop_bytes / (hbm_peak * 1e9) * 1e6, 1),
                                         "this_kernel_us": round(gen_us_clean, 2)}}
    elif dom:
        roofline = {"kernel": dom["kernel"], "bound": "hbm", "achieved": dom["achieved_gbs"], "peak": hbm_peak,
                    "peak_source": "MEASURED_PEAKS.json hbm_gbs" if peak_src == "measured" else "recipe fallback",
                    "unit": "GB/s", "frac": dom["frac_of_hbm_peak"], "traffic": NCU_TRAFFIC_BYTES.get(dom["kernel"]),
                    "algorithmic_bytes_per_launch": dom["algorithmic_bytes"], "avg_launch_us": dom["avg_us"]}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": t_max / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": CONFIG,
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                "ms_per_step": e2e_ms / args.steps, "api": "schedule_round_host (pinned host buffers)"},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "kernels": kernels,
        "kernel_timing": {"how": "second pass over the same steps with a CUDA-event pair around every kernel (no "
                                 "graph replay, no overlap between consecutive kernels): shares only",
                          "ms_per_step": profiled_ms / args.steps},
        "row_store": {"pool_moves_so_far": moves, "clean_round_ms": full_ms, "clean_half_round_ms": half_ms},
        "best_fitness": float(h_bf.item()),
        "best_allocation": allocation_summary(h_best.numpy(), jobs, cl),
    }
    sched.close()

    if world == 1 and not args.skip_extras:
        line["dense_generation"] = bench_dense_generation(api, torch, dev, stream, cfg, cl, jobs, cur, hbm_peak, peak_src)
        line["goodput_model"] = bench_table(api, torch, dev, stream, cfg, cl, jobs, sm_max_mhz, clocks)
        line["stress_fitness"] = bench_stress(api, torch, dev, stream, hbm_peak, peak_src, args)
        line["testbed_round"] = bench_testbed(api, torch, dev, stream)
        line["trace_replay"] = bench_trace(api, torch, stream)
        line["theta_fit"] = bench_fit(api, torch, dev, stream)
        line["ga_quality"] = bench_ga_quality(api, torch, dev, stream)
        line["cpu_baseline"] = oracle_sample(cfg, cl, jobs, cur, table_jobs=256, gens=20)
        line["cpu_baseline_single_thread"] = oracle_sample(cfg, cl, jobs, cur, table_jobs=8, gens=3, threads=1)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def bench_dense_generation(api, torch, dev, stream, cfg, cl, jobs, cur, hbm_peak, peak_src):
    """ga_generation on dense matrices (the entry point; a round of this size uses the row store
    instead): the row pass streams 268 MB of parents in and 268 MB of children out."""
    P, J, NN = cfg.population, cfg.num_jobs, cfg.num_nodes
    sched = api.scheduler_for(cfg, stream=stream.cuda_stream)
    dj = api.DeviceJobs(jobs, dev, torch)
    a = torch.empty((P, J, NN), dtype=torch.int16, device=dev)
    b = torch.empty_like(a)
    fit = torch.rand(P, dtype=torch.float32, device=dev)
    sched.init_population(dj, torch.from_numpy(cur).to(dev), a, round=0)
    for g in range(3):
        sched.ga_generation(dj, a, fit, b, round=0, generation=g)
        a, b = b, a
    sched.set_kernel_timing(True)
    sched.read_kernel_timing()
    reps = 20
    for g in range(reps):
        sched.ga_generation(dj, a, fit, b, round=0, generation=3 + g)     # 536 MB per pass: larger than L2
        a, b = b, a
    t = sched.read_kernel_timing()
    sched.close()
    # a device-to-device copy of one population (the runtime's own copy, same 268 MB in and out,
    # same stream): what a plain copy of this size reaches on this GPU, beside the row pass
    copy_us = []
    for _ in range(9):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        b.copy_(a)
        e1.record(stream)
        e1.synchronize()
        copy_us.append(e0.elapsed_time(e1) * 1e3)
    copy_us = sorted(copy_us)[len(copy_us) // 2]
    rows_ms = t["rows"][0] / reps
    cols_ms = t["cols"][0] / reps
    algo = 2.0 * P * J * NN * 2 + P * J * 5
    gbs = algo / (rows_ms * 1e-3) / 1e9
    return {"workload": "large shape, dense int16 [512][1024][256] in and out", "rows_us": round(rows_ms * 1e3, 2),
            "column_repair_us": round(cols_ms * 1e3, 2), "generations_per_sec": 1e3 / (rows_ms + cols_ms),
            "plain_copy_same_size_us": round(copy_us, 2),
            "plain_copy_note": "runtime device-to-device copy of one population, for context: the measured peak "
                               "below was taken on buffers several times larger",
            "roofline": {"kernel": "rows", "bound": "hbm", "achieved": round(gbs, 1), "peak": hbm_peak,
                         "peak_source": "MEASURED_PEAKS.json hbm_gbs" if peak_src == "measured" else "recipe fallback",
                         "unit": "GB/s", "frac": round(gbs / hbm_peak, 4), "traffic": NCU_TRAFFIC_BYTES["rows"],
                         "algorithmic_bytes_per_launch": algo}}


def bench_table(api, torch, dev, stream, cfg, cl, jobs, sm_max_mhz, clocks):
    """build_speedup_table alone on the large workload: distinct (job, K, class, m, s) points
    per second, and the share of the fp32 lane-op peak (ALU-bound kernel) - the nominal one and
    the one an FMA-chain microbenchmark reaches in this very process; the special-function
    unit's share of the sweep time against a lg2/ex2-chain microbenchmark."""
    import oracle

    sched = api.scheduler_for(cfg, stream=stream.cuda_stream)
    dj = api.DeviceJobs(jobs, dev, torch)
    sp = torch.empty(sched.table_shape, dtype=torch.float32, device=dev)
    gp = torch.empty_like(sp)
    am = torch.empty(sched.table_shape, dtype=torch.uint16, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    for _ in range(3):
        sched.build_speedup_table(dj, gp, sp, am)
    sched.set_kernel_timing(True)
    sched.read_kernel_timing()
    reps = 20
    for _ in range(reps):
        flush.fill_(1)                      # L2 flush between iterations
        sched.build_speedup_table(dj, gp, sp, am)
    t = sched.read_kernel_timing()
    # the total-batch sampling search of Sec. 4.3 on the same jobs (128 candidates per job)
    ms = torch.from_numpy(synth.make_m_samples(jobs.m0, jobs.m_max_total, 128)).to(dev)
    mm = torch.from_numpy(jobs.m_max_gpu).to(dev)
    for _ in range(3):
        sched.build_speedup_table_msample(dj, ms, mm, gp, sp, am)
    sched.read_kernel_timing()
    for _ in range(reps):
        flush.fill_(1)
        sched.build_speedup_table_msample(dj, ms, mm, gp, sp, am)
    t2 = sched.read_kernel_timing()
    msample_ms = t2["goodput_sweep"][0] / reps
    sched.set_kernel_timing(False)
    fma_peak, mufu_peak, _ = sched.measure_peaks(None, reps=5)
    sched.close()
    sweep_ms = t["goodput_sweep"][0] / reps
    expand_ms = t["speedup_expand"][0] / reps
    classes = distinct_classes(cl)
    points = float(cfg.num_jobs) * classes * cfg.grid_m * cfg.grid_s
    num_sms = torch.cuda.get_device_properties(dev).multi_processor_count
    peak = num_sms * FP32_LANES_PER_SM * sm_max_mhz * 1e6          # lane-ops/s (an FMA counts once)
    achieved = OPS_PER_POINT * points / (sweep_ms * 1e-3)
    mufu_ops = 3.0 * cfg.num_jobs * classes * cfg.grid_m            # per (job, K, class, m): ex2, lg2, ex2
    # the oracle's table build on a sample of jobs, all threads and one
    sub = jobs.take(slice(0, 8))
    t0 = time.perf_counter()
    oracle.build_speedup_table(sub, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s, want_argmax=False)
    cpu_all = 8 * classes * cfg.grid_m * cfg.grid_s / (time.perf_counter() - t0)
    oracle.set_threads(1)
    try:
        t0 = time.perf_counter()
        oracle.build_speedup_table(jobs.take(slice(0, 1)), cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s, want_argmax=False)
        cpu_one = classes * cfg.grid_m * cfg.grid_s / (time.perf_counter() - t0)
    finally:
        oracle.set_threads(0)
    return {
        "workload": "large", "distinct_points": points, "sweep_us": round(sweep_ms * 1e3, 2),
        "expand_us": round(expand_ms * 1e3, 2),
        "evals_per_sec": points / ((sweep_ms + expand_ms) * 1e-3),
        "evals_per_sec_sweep_only": points / (sweep_ms * 1e-3),
        "msample_search": {"candidates_per_job": 128, "sweep_us": round(msample_ms * 1e3, 2),
                           "evals_per_sec": float(cfg.num_jobs) * classes * 128 / (msample_ms * 1e-3),
                           "note": "integer (m, s) derivation + 3 MUFU per candidate; latency-sized at this size"},
        "roofline": {"kernel": "goodput_sweep", "bound": "alu", "achieved": achieved / 1e12, "peak": peak / 1e12,
                     "unit": "T lane-op/s", "frac": achieved / peak,
                     "peak_source": "%d SMs x %d fp32 lanes x %.0f MHz (max SM clock)" % (num_sms, FP32_LANES_PER_SM, sm_max_mhz),
                     "peak_measured": fma_peak / 1e12, "frac_of_measured": achieved / fma_peak,
                     "peak_measured_how": "eight independent FMA chains per thread, %d x 8 blocks of 256 threads, same process"
                                          % num_sms,
                     "mufu": {"ops_per_launch": mufu_ops, "peak_measured_ops_per_sec": mufu_peak,
                              "peak_nominal_ops_per_sec": num_sms * 16 * sm_max_mhz * 1e6,
                              "share_of_sweep_time": (mufu_ops / mufu_peak) / (sweep_ms * 1e-3),
                              "note": "three special-function operations per (job, K, class, m), amortised over the s loop"},
                     "ops_per_point": OPS_PER_POINT, "traffic": None, "l2": "flushed between iterations"},
        "cpu_baseline": {"value": cpu_all, "unit": "distinct points/s", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": "tables of 8 of %d jobs" % cfg.num_jobs, "single_thread_value": cpu_one,
                         "single_thread_sample": "table of 1 job"},
    }


def bench_stress(api, torch, dev, stream, hbm_peak, peak_src, args):
    """eval_fitness on the stress workload (2048 x 8 cluster, 8192 jobs, fp32 [8192][65][65] tables,
    4096 dense int16 candidates of 33.5 MB each = 137 GB): evaluated in chunks that are generated on
    the device one after another (generation untimed), kernel times summed over the whole
    population; candidates are independent, so the chunking does not change the metric."""
    import oracle

    st = synth.STRESS
    chunk = args.stress_chunk
    total = args.stress_population
    J, NN = st["num_jobs"], st["num_nodes"]
    cap = synth.uniform_cluster(NN, st["gpus_per_node"]).node_capacity
    sched = api.Scheduler(node_capacity=cap, num_jobs=J, grid_m=1, grid_s=1, population=chunk,
                          stream=stream.cuda_stream)
    h_table = synth.stress_speedup_table(J, 64, 64, st["gpus_per_node"], st["seed"])
    table = torch.from_numpy(h_table).to(dev)
    fit = torch.empty(chunk, dtype=torch.float32, device=dev)
    bytes_per_cand = J * NN * 2 + J * 4 + 4
    out = {"workload": "stress: %d candidates in chunks of %d, 8192 jobs x 2048 nodes, int16 dense" % (total, chunk),
           "chunk_bytes": int(chunk) * J * NN * 2, "p": {}}
    sched.set_kernel_timing(True)
    ms_sum = {p: 0.0 for p in st["p_values"]}
    pop = None
    for first in range(0, total, chunk):
        del pop
        pop = torch.cat([synth.stress_population(32, J, NN, st["gpus_per_node"], st["seed"], device=dev, first_candidate=c)
                         for c in range(first, first + chunk, 32)])
        for p in st["p_values"]:
            if first == 0:
                for _ in range(3):
                    sched.eval_fitness(pop, table, fit, p=p)
            sched.read_kernel_timing()
            sched.eval_fitness(pop, table, fit, p=p)          # 8.6 GB per pass: far larger than L2
            ms_sum[p] += sched.read_kernel_timing()["fitness"][0]
    sched.set_kernel_timing(False)
    _, _, read_peak = sched.measure_peaks(pop, reps=3)       # read-only stream over the last chunk, same process
    worst = None
    for p in st["p_values"]:
        gbs = total * bytes_per_cand / (ms_sum[p] * 1e-3) / 1e9
        out["p"][str(p)] = {"ms_whole_population": round(ms_sum[p], 3), "candidates_per_sec": total / (ms_sum[p] * 1e-3),
                            "achieved_gbs": round(gbs, 1), "frac_of_hbm_peak": round(gbs / hbm_peak, 4)}
        if worst is None or gbs < worst[0]:
            worst = (gbs, ms_sum[p])
    per_launch_ms = worst[1] * chunk / total
    out["roofline"] = {"kernel": "fitness", "bound": "hbm", "achieved": round(worst[0], 1), "peak": hbm_peak,
                       "peak_source": "MEASURED_PEAKS.json hbm_gbs (a copy: read + write)" if peak_src == "measured" else "recipe fallback",
                       "unit": "GB/s", "frac": round(worst[0] / hbm_peak, 4), "frac_of_8tbs_nominal": round(worst[0] / 8000.0, 4),
                       "read_only_peak_measured_gbs": round(read_peak / 1e9, 1),
                       "frac_of_read_only_peak": round(worst[0] * 1e9 / read_peak, 4) if read_peak > 0 else None,
                       "read_only_peak_how": "16-byte loads, four in flight per thread, over the %.1f GB chunk, same process"
                                             % (chunk * J * NN * 2 / 1e9),
                       "traffic": NCU_TRAFFIC_BYTES["fitness_stress_per_candidate"] * chunk,
                       "traffic_note": "ncu capture of 16 candidates scaled by candidates / 16 (committed summary, not this run)",
                       "algorithmic_bytes_per_launch": chunk * bytes_per_cand, "avg_launch_us": round(per_launch_ms * 1e3, 1),
                       "note": "slowest of the three exponents; one launch = one chunk"}
    # the oracle on 64 candidates of the last chunk, scaled to candidates per second
    sample = pop[:64].cpu().numpy()
    t64 = h_table.astype(np.float64)
    t0 = time.perf_counter()
    oracle.eval_fitness(sample, t64, 64, 64, -1.0, 1e-3)
    cpu_all = 64 / (time.perf_counter() - t0)
    oracle.set_threads(1)
    try:
        t0 = time.perf_counter()
        oracle.eval_fitness(sample[:8], t64, 64, 64, -1.0, 1e-3)
        cpu_one = 8 / (time.perf_counter() - t0)
    finally:
        oracle.set_threads(0)
    out["cpu_baseline"] = {"value": cpu_all, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                           "sample": "64 candidates of one chunk (scaled linearly to the population)",
                           "single_thread_value": cpu_one, "single_thread_sample": "8 candidates"}
    sched.close()
    del pop, table
    torch.cuda.empty_cache()
    return out


def bench_fit(api, torch, dev, stream):
    """fit_throughput_model: 1024 jobs x 64 profiled iteration times each (2 % noise), from a
    generic start; jobs fitted per second, with scipy's L-BFGS-B (the oracle) timed on 8 jobs."""
    from oracle import fit as ofit

    J, per_job = 1024, 64
    jobs = synth.draw_jobs(J, 7, 8, 8, 16)
    offset, K, N, m, s, factor = synth.draw_observations(jobs, per_job, 8)
    true = np.stack([jobs.alpha_grad, jobs.beta_grad, jobs.alpha_local, jobs.beta_local, jobs.alpha_node,
                     jobs.beta_node, jobs.gamma], axis=1).astype(np.float64)
    T = np.empty(offset[-1], np.float32)
    for j in range(J):
        sl = slice(offset[j], offset[j + 1])
        T[sl] = (ofit.t_iter(true[j], K[sl], N[sl], m[sl], s[sl]) * factor[sl]).astype(np.float32)
    theta0 = np.tile(np.array([0.1, 0.01, 0.01, 0.01, 0.01, 0.01, 1.0], np.float32), (J, 1))
    sched = api.Scheduler(node_capacity=np.full(4, 4, np.int16), num_jobs=1, grid_m=1, grid_s=1, population=1,
                          stream=stream.cuda_stream)
    d = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    bufs = [d(x) for x in (offset, K, N, m, s, T, theta0)]
    th = torch.empty((J, 7), dtype=torch.float32, device=dev)
    loss = torch.empty(J, dtype=torch.float32, device=dev)
    for _ in range(2):
        sched.fit_throughput_model(*bufs, th, loss, max_iters=100)
    sched.set_kernel_timing(True)
    sched.read_kernel_timing()
    reps = 5
    for _ in range(reps):
        sched.fit_throughput_model(*bufs, th, loss, max_iters=100)
    ms = sched.read_kernel_timing()["fit_theta"][0] / reps
    sched.close()
    t0 = time.perf_counter()
    ref = [ofit.fit(K[offset[j]:offset[j + 1]], N[offset[j]:offset[j + 1]], m[offset[j]:offset[j + 1]],
                    s[offset[j]:offset[j + 1]], T[offset[j]:offset[j + 1]], theta0[j])[1] for j in range(8)]
    cpu_s = (time.perf_counter() - t0) / 8
    lg = loss.cpu().numpy()
    return {"workload": "1024 jobs x 64 observations, 2% noise", "ms": round(ms, 3), "jobs_per_sec": J / (ms * 1e-3),
            "median_rmsle": float(np.median(lg)), "oracle_lbfgsb_sec_per_job": cpu_s,
            "oracle_median_rmsle_8_jobs": float(np.median(ref)),
            "note": "fp64 damped Gauss-Newton, one warp per job; the paper reports 0.2 s per fit on a CPU core"}


def bench_testbed(api, torch, dev, stream):
    """schedule_round on the testbed-scale workload (16 nodes x 4 GPUs, 48 jobs, grid 64 x 16,
    population 100, 100 generations, re-allocation penalty against a random current allocation):
    the size of the paper's own cluster.  Launch- and latency-bound; rounds replay as graphs."""
    cfg = synth.TESTBED
    cl = cfg.cluster()
    jobs = cfg.jobs()
    fk, fn = api.fair_share(cl.node_capacity, cfg.num_jobs, cl.k_max)
    jobs.fair_k = np.full(cfg.num_jobs, fk, np.int32)
    jobs.fair_n = np.full(cfg.num_jobs, fn, np.int32)
    sched = api.scheduler_for(cfg, stream=stream.cuda_stream)
    dj = api.DeviceJobs(jobs, dev, torch)
    d_cur = torch.from_numpy(cfg.cur()).to(dev)
    best = torch.empty((cfg.num_jobs, cfg.num_nodes), dtype=torch.int16, device=dev)
    bf = torch.zeros(1, dtype=torch.float32, device=dev)
    for r in range(5):
        sched.schedule_round(dj, d_cur, best, bf, round=r, generations=cfg.generations)
    sched.sync_status()
    n = 200
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for r in range(n):
        sched.schedule_round(dj, d_cur, best, bf, round=10 + r, generations=cfg.generations)
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / n
    sched.close()
    return {"workload": "testbed: 16 nodes x 4 GPUs, 48 jobs, grid 64x16, population 100, 100 generations, p=-1",
            "ms_per_round": ms, "rounds_per_sec": 1e3 / ms,
            "candidates_per_sec": cfg.population * (cfg.generations + 1) / (ms * 1e-3),
            "us_per_generation": 1e3 * ms / cfg.generations,
            "note": "one 100-block kernel per generation (thread per row): latency-bound, no roofline; "
                    "the paper reports about 1 s per round on one CPU core at this cluster size"}


def bench_trace(api, torch, stream):
    """Trace replay: 480 scheduling rounds (one per 60 s of an 8-hour, 160-job trace on 16 x 4
    GPUs), each a table rebuild + 100 generations at population 100, through the host-buffer
    entry point; wall-clock rounds per second including the host driver."""
    from paper_2008_12260_b200 import trace

    tr = trace.TraceReplay()
    sched = api.scheduler_for(tr.cfg, stream=stream.cuda_stream)
    trace.replay(sched, tr, torch, rounds=20)          # warm-up, graph capture
    tr.reset()
    torch.cuda.synchronize()
    l0 = sched.launch_count()
    t0 = time.perf_counter()
    fits, used = trace.replay(sched, tr, torch)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    out = {"workload": "160 jobs, Poisson arrivals over 8 h, 16 nodes x 4 GPUs, round every 60 s, "
                       "table rebuild + 100 generations, population 100",
           "rounds": len(fits), "seconds": dt, "rounds_per_sec": len(fits) / dt,
           "kernel_launches_per_round": (sched.launch_count() - l0) / len(fits),
           "mean_best_fitness": float(np.mean(fits[10:])), "mean_gpus_allocated": float(np.mean(used[10:])),
           "note": "launch- and latency-bound (population 150 KB): a roofline fraction is not meaningful here"}
    # the same trace with training progress coupled to the allocations (jobs advance at the goodput
    # the round's own tables predict, 30 s restart delay): completion times depend on the scheduler
    pr = trace.ProgressReplay()
    t0 = time.perf_counter()
    pfits = trace.replay_progress(sched, pr, torch)
    torch.cuda.synchronize()
    pdt = time.perf_counter() - t0
    jct = pr.completion_times()
    out["progress_coupled"] = {"rounds_per_sec": len(pfits) / pdt, "jobs_finished": int(jct.size),
                               "avg_jct_hours": float(jct.mean() / 3600.0) if jct.size else None,
                               "p99_jct_hours": float(np.percentile(jct, 99) / 3600.0) if jct.size else None}
    sched.close()
    return out


# ------------------------------------------------------------------------------------------
def oracle_sample(cfg, cl, jobs, cur, table_jobs: int = 8, gens: int = 2, threads: int = 0):
    """The CPU oracle on a bounded sample of the large round: tables of `table_jobs` jobs, the
    initial population, and `gens` x (generation + fitness) at the full population; the
    time of a whole round is extrapolated linearly (tables x J / table_jobs, generations x
    G / gens).  threads = 1: one core, the figure the paper's scheduler is quoted on
    (Sec. 5.2, system overheads)."""
    import oracle

    oracle.set_threads(threads)
    try:
        return _oracle_sample(oracle, cfg, cl, jobs, cur, table_jobs, gens)
    finally:
        oracle.set_threads(0)


def _oracle_sample(oracle, cfg, cl, jobs, cur, table_jobs, gens):
    P, J, G = cfg.population, cfg.num_jobs, cfg.generations
    sub = jobs.take(slice(0, table_jobs))
    t0 = time.perf_counter()
    oracle.build_speedup_table(sub, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s, want_argmax=False)
    t_table = (time.perf_counter() - t0) * (J / table_jobs)
    rng = np.random.default_rng(0)
    speedup = rng.uniform(0.1, 3.0, (J, cl.k_max + 1, cl.n_max + 1))
    rf = oracle.realloc_factor(jobs.age_sec, jobs.num_restarts, cfg.delta_sec)
    thr_m, thr_i = synth.prob_to_threshold(cfg.mutate_prob), synth.prob_to_threshold(cfg.init_prob)
    t0 = time.perf_counter()
    pop = oracle.init_population(P, cur, J, cl.node_capacity, jobs.k_cap, cl.k_max, cl.n_max, thr_i, cfg.seed, 0)
    fit = oracle.eval_fitness(pop, speedup, cl.k_max, cl.n_max, cfg.p, cfg.speedup_floor, cur=cur, realloc=rf)
    t_init = time.perf_counter() - t0
    t0 = time.perf_counter()
    for g in range(gens):
        pop = oracle.ga_generation(pop, fit.astype(np.float32), cl.node_capacity, jobs.k_cap, cl.k_max, cl.n_max,
                                   cfg.num_elite, thr_m, cfg.seed, 0, g)
        fit = oracle.eval_fitness(pop, speedup, cl.k_max, cl.n_max, cfg.p, cfg.speedup_floor, cur=cur, realloc=rf)
    t_gen = (time.perf_counter() - t0) / gens
    round_s = t_table + t_init + G * t_gen
    return {"value": P * (G + 1) / round_s, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": "tables of %d of %d jobs, initial population, %d of %d generations at population %d; "
                      "round time extrapolated linearly" % (table_jobs, J, gens, G, P),
            "round_seconds_extrapolated": round_s, "table_seconds_extrapolated": t_table,
            "generation_seconds": t_gen}


def run_reference(args):
    """The oracle as the reference arm: CPU only, rank 0 only."""
    rank, _, world = pdist.env_world()
    if rank != 0:
        return
    import oracle

    cfg, cl, jobs, cur = large_inputs(0, oracle.fair_share)
    samples = []
    for i in range(args.warmup + args.steps):
        s = oracle_sample(cfg, cl, jobs, cur, table_jobs=16, gens=2)
        if i >= args.warmup:
            samples.append(s)
    round_s = statistics.mean(s["round_seconds_extrapolated"] for s in samples)
    value = cfg.population * (cfg.generations + 1) / round_s
    base = dict(samples[-1], value=value)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round_s * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": CONFIG,
        "reference_note": "CPU oracle (fp64); each step times a bounded sample and extrapolates the round",
        "cpu_baseline": base,
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--skip-extras", action="store_true", help="only the timed rounds (no single-kernel sections, no oracle)")
    ap.add_argument("--stress-chunk", type=int, default=256, help="candidates in the stress fitness chunk (multiple of 32)")
    ap.add_argument("--stress-population", type=int, default=4096, help="candidates of the stress population (multiple of the chunk)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
