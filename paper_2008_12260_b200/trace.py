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
