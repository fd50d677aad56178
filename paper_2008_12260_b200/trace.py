"""Trace replay: a scheduling round every 60 s over an 8-hour synthetic job trace.

160 jobs arrive as a Poisson process on a 16 x 4-GPU cluster; each has a fixed lifetime
(so every round's inputs can be generated without simulating training progress) and a
gradient noise scale that grows linearly from phi0 to 10 phi0 over its life (Sec. 3.1 of
the paper: phi grows about tenfold during training).  Each round rebuilds the speedup
tables for the jobs present, and searches from the previous round's allocation.  The age
T_j and the re-allocation count R_j that enter the re-allocation penalty are tracked on
the host from the allocations the rounds return.

Input generation and bookkeeping only: every step of a round runs in the CUDA library.
"""
from __future__ import annotations

import numpy as np

from . import synth

ROUND_SEC = 60.0


class TraceReplay:
    def __init__(self, num_jobs: int = 160, seed: int = 4, horizon_sec: float = 8 * 3600.0,
                 num_nodes: int = 16, gpus_per_node: int = 4, grid_m: int = 64, grid_s: int = 16,
                 population: int = 100, generations: int = 100):
        self.cfg = synth.Config("trace", num_nodes, gpus_per_node, num_jobs, seed, grid_m, grid_s, population,
                                generations, num_elite=4, mutate_prob=0.08, init_prob=0.25)
        self.cluster = self.cfg.cluster()
        self.base = synth.draw_jobs(num_jobs, seed, grid_m, grid_s, self.cluster.k_max)
        tr = synth.trace_arrivals(num_jobs, seed, horizon_sec)
        self.arrive = np.array([t.arrive_sec for t in tr])
        self.life = np.array([t.life_sec for t in tr])
        self.phi0 = self.base.phi.astype(np.float64).copy()
        self.num_rounds = int(horizon_sec // ROUND_SEC)
        self.restarts = np.zeros(num_jobs, dtype=np.int32)
        self.cur = np.zeros((num_jobs, num_nodes), dtype=np.int16)

    def reset(self):
        self.restarts[:] = 0
        self.cur[:] = 0

    def round_inputs(self, k: int):
        """Job arrays and current allocation of round k (time t = 60 k seconds)."""
        from .api import fair_share

        t = k * ROUND_SEC
        age = t - self.arrive
        active = (age >= 0.0) & (age < self.life)
        jobs = self.base.take(slice(None))
        frac = np.clip(age / self.life, 0.0, 1.0)
        jobs.phi = (self.phi0 * (1.0 + 9.0 * frac)).astype(np.float32)
        jobs.age_sec = np.maximum(age, 1.0).astype(np.float32)
        jobs.num_restarts = self.restarts.copy()
        jobs.active = active.astype(np.uint8)
        fk, fn = fair_share(self.cluster.node_capacity, int(active.sum()), self.cluster.k_max)
        jobs.fair_k = np.full(jobs.num_jobs, fk, np.int32)
        jobs.fair_n = np.full(jobs.num_jobs, fn, np.int32)
        cur = self.cur.copy()
        cur[~active] = 0
        return jobs, cur

    def commit(self, k: int, jobs, cur, best: np.ndarray):
        """Book-keeping after round k returned `best`: a running job whose row changed was
        re-allocated once more."""
        running = cur.sum(axis=1) > 0
        moved = running & (best != cur).any(axis=1) & (jobs.active > 0)
        self.restarts[moved] += 1
        self.cur = best.astype(np.int16).copy()


def replay(sched, trace: TraceReplay, torch, rounds=None, first_round: int = 0, on_round=None):
    """Runs `rounds` scheduling rounds through schedule_round_host with pinned buffers.
    Returns (best fitness per round, GPUs allocated per round)."""
    from .api import HostJobs

    cfg = trace.cfg
    rounds = trace.num_rounds if rounds is None else rounds
    h_best = torch.empty((cfg.num_jobs, cfg.num_nodes), dtype=torch.int16).pin_memory()
    h_bf = torch.zeros(1, dtype=torch.float32).pin_memory()
    h_cur = torch.empty((cfg.num_jobs, cfg.num_nodes), dtype=torch.int16).pin_memory()
    fits, used = [], []
    for k in range(first_round, first_round + rounds):
        jobs, cur = trace.round_inputs(k)
        hj = HostJobs(jobs, torch, pin=False)
        h_cur.copy_(torch.from_numpy(cur))
        sched.schedule_round_host(hj, h_cur, h_best, h_bf, round=k, generations=cfg.generations)
        best = h_best.numpy().copy()
        trace.commit(k, jobs, cur, best)
        fits.append(float(h_bf.item()))
        used.append(int(best.sum()))
        if on_round is not None:
            on_round(k, jobs, cur, best, fits[-1])
    return fits, used


class ProgressReplay(TraceReplay):
    """Trace replay in which jobs make training progress at the goodput the scheduler's own
    tables predict for their allocation, in the manner of the paper's discrete-time simulator
    (Sec. 5.3) but without its measured profiles.

    A job's total work is what one GPU at its initial noise scale would process during its
    nominal lifetime.  Every 60 s round a job advances by goodput x (60 s minus a 30 s restart
    delay if its allocation changed); phi grows from phi0 to 10 phi0 with the fraction of
    work done; a job leaves when its work is done.  Completion times therefore depend on the
    allocations the rounds return.
    """

    RESTART_DELAY_SEC = 30.0

    def __init__(self, **kw):
        super().__init__(**kw)
        self.work = None          # set on first use (needs the 1-GPU goodput of every job)
        self.reset()

    def reset(self):
        super().reset()
        n = self.cfg.num_jobs
        self.done = np.zeros(n)
        self.finish = np.full(n, np.nan)

    def round_inputs(self, k: int):
        from .api import fair_share

        t = k * ROUND_SEC
        age = t - self.arrive
        total = self.work if self.work is not None else np.full(self.cfg.num_jobs, np.inf)
        active = (age >= 0.0) & np.isnan(self.finish)
        jobs = self.base.take(slice(None))
        frac = np.clip(self.done / total, 0.0, 1.0)
        jobs.phi = (self.phi0 * (1.0 + 9.0 * frac)).astype(np.float32)
        jobs.age_sec = np.maximum(age, 1.0).astype(np.float32)
        jobs.num_restarts = self.restarts.copy()
        jobs.active = active.astype(np.uint8)
        fk, fn = fair_share(self.cluster.node_capacity, int(active.sum()), self.cluster.k_max)
        jobs.fair_k = np.full(jobs.num_jobs, fk, np.int32)
        jobs.fair_n = np.full(jobs.num_jobs, fn, np.int32)
        cur = self.cur.copy()
        cur[~active] = 0
        return jobs, cur

    def advance(self, k: int, jobs, cur, best: np.ndarray, goodput_kn: np.ndarray, goodput_1gpu: np.ndarray):
        """After round k: goodput_kn[j] is the table's goodput of job j at its new allocation,
        goodput_1gpu[j] at one GPU (used once, to fix the job's total work)."""
        if self.work is None:
            self.work = np.full(self.cfg.num_jobs, np.inf)
        fresh = np.isinf(self.work) & (jobs.active > 0)
        self.work[fresh] = self.life[fresh] * goodput_1gpu[fresh]
        moved = (best != cur).any(axis=1)
        run = ROUND_SEC - np.where(moved, self.RESTART_DELAY_SEC, 0.0)
        gain = np.where((jobs.active > 0) & (best.sum(axis=1) > 0), goodput_kn * run, 0.0)
        before = self.done.copy()
        self.done = self.done + gain
        fin = (jobs.active > 0) & (self.done >= self.work) & np.isnan(self.finish)
        # finish time interpolated inside the interval
        part = np.where(gain > 0, (self.work - before) / np.maximum(gain, 1e-30), 1.0)
        self.finish[fin] = (k * ROUND_SEC + (ROUND_SEC - run[fin]) + part[fin] * run[fin])
        self.commit(k, jobs, cur, best)
        self.cur[fin] = 0

    def completion_times(self):
        ok = ~np.isnan(self.finish)
        return (self.finish - self.arrive)[ok]


def replay_progress(sched, trace: ProgressReplay, torch, rounds=None, on_round=None):
    """Like replay(), but jobs advance at the goodput of the round's own tables."""
    from .api import HostJobs

    cfg = trace.cfg
    rounds = trace.num_rounds if rounds is None else rounds
    dev = "cuda"
    h_best = torch.empty((cfg.num_jobs, cfg.num_nodes), dtype=torch.int16).pin_memory()
    h_bf = torch.zeros(1, dtype=torch.float32).pin_memory()
    h_cur = torch.empty((cfg.num_jobs, cfg.num_nodes), dtype=torch.int16).pin_memory()
    d_gp = torch.empty(sched.table_shape, dtype=torch.float32, device=dev)
    jidx = torch.arange(cfg.num_jobs, device=dev)
    fits = []
    for k in range(rounds):
        jobs, cur = trace.round_inputs(k)
        hj = HostJobs(jobs, torch, pin=False)
        h_cur.copy_(torch.from_numpy(cur))
        sched.schedule_round_host(hj, h_cur, h_best, h_bf, round=k, generations=cfg.generations)
        best = h_best.numpy().copy()
        sched.get_round_tables(d_gp, None)
        sched.sync_status()
        K = torch.from_numpy(np.minimum(best.sum(axis=1), sched.cfg.k_max).astype(np.int64)).to(dev)
        N = torch.from_numpy(np.minimum((best > 0).sum(axis=1), sched.cfg.n_max).astype(np.int64)).to(dev)
        g_kn = d_gp[jidx, K, N].double().cpu().numpy()
        g_1 = d_gp[:, 1, 1].double().cpu().numpy()
        trace.advance(k, jobs, cur, best, g_kn, g_1)
        fits.append(float(h_bf.item()))
        if on_round is not None:
            on_round(k, jobs, cur, best, fits[-1], g_kn)
    return fits
