"""Small, self-terminating cases of each hot kernel for profiler captures.

    python -m paper_2008_12260_b200.profile_cases fitness_stress   # 16 stress candidates (537 MB)
    python -m paper_2008_12260_b200.profile_cases table_large      # 1024-job speedup table
    python -m paper_2008_12260_b200.profile_cases round_large [G]  # large round, G generations (default 2)
    python -m paper_2008_12260_b200.profile_cases generation_large # dense ga_generation, large shape
    python -m paper_2008_12260_b200.profile_cases round_testbed [G] # testbed-scale round, G generations

Each case holds well under a few GB on the device, launches its kernel a handful of
times and exits; inputs are larger than L2 wherever DRAM traffic is the point.
"""
from __future__ import annotations

import sys

import numpy as np


def _large(api, synth, torch):
    cfg = synth.LARGE
    cl = cfg.cluster()
    jobs = cfg.jobs()
    fk, fn = api.fair_share(cl.node_capacity, cfg.num_jobs, cl.k_max)
    jobs.fair_k = np.full(cfg.num_jobs, fk, np.int32)
    jobs.fair_n = np.full(cfg.num_jobs, fn, np.int32)
    s = api.scheduler_for(cfg, stream=torch.cuda.current_stream().cuda_stream)
    return cfg, cl, jobs, s, api.DeviceJobs(jobs, "cuda", torch)


def main(case: str, reps: int = 3, generations: int = 2):
    import torch
    from . import api, synth

    if case == "fitness_stress":
        st = synth.STRESS
        n = 16
        cap = synth.uniform_cluster(st["num_nodes"], 8).node_capacity
        s = api.Scheduler(node_capacity=cap, num_jobs=st["num_jobs"], grid_m=1, grid_s=1, population=n,
                          stream=torch.cuda.current_stream().cuda_stream)
        table = torch.from_numpy(synth.stress_speedup_table(st["num_jobs"], 64, 64, 8, st["seed"])).cuda()
        pop = synth.stress_population(n, st["num_jobs"], st["num_nodes"], 8, st["seed"], device="cuda")
        fit = torch.empty(n, dtype=torch.float32, device="cuda")
        for _ in range(reps):
            s.eval_fitness(pop, table, fit, p=-1.0)
        s.sync_status()
        print("fitness_stress", fit[:3].tolist())
    elif case == "table_large":
        cfg, cl, jobs, s, dj = _large(api, synth, torch)
        sp = torch.empty(s.table_shape, dtype=torch.float32, device="cuda")
        for _ in range(reps):
            s.build_speedup_table(dj, None, sp, None)
        s.sync_status()
        print("table_large", float(sp[0, 2, 1]))
    elif case == "round_large":
        cfg, cl, jobs, s, dj = _large(api, synth, torch)
        s.set_store_budget(2 << 30)        # a small row pool: a profiler saves and restores device memory per pass
        cur = torch.from_numpy(cfg.cur()).cuda()
        best = torch.empty((cfg.num_jobs, cfg.num_nodes), dtype=torch.int16, device="cuda")
        bf = torch.zeros(1, dtype=torch.float32, device="cuda")
        s.schedule_round(dj, cur, best, bf, round=0, generations=generations)
        s.sync_status()
        print("round_large", float(bf.item()))
    elif case == "round_testbed":
        cfg = synth.TESTBED
        cl = cfg.cluster()
        jobs = cfg.jobs()
        fk, fn = api.fair_share(cl.node_capacity, cfg.num_jobs, cl.k_max)
        jobs.fair_k = np.full(cfg.num_jobs, fk, np.int32)
        jobs.fair_n = np.full(cfg.num_jobs, fn, np.int32)
        s = api.scheduler_for(cfg, stream=torch.cuda.current_stream().cuda_stream)
        dj = api.DeviceJobs(jobs, "cuda", torch)
        cur = torch.from_numpy(cfg.cur()).cuda()
        best = torch.empty((cfg.num_jobs, cfg.num_nodes), dtype=torch.int16, device="cuda")
        bf = torch.zeros(1, dtype=torch.float32, device="cuda")
        s.schedule_round(dj, cur, best, bf, round=0, generations=generations)
        s.sync_status()
        print("round_testbed", float(bf.item()))
    elif case == "generation_large":
        cfg, cl, jobs, s, dj = _large(api, synth, torch)
        shape = (cfg.population, cfg.num_jobs, cfg.num_nodes)
        a = torch.empty(shape, dtype=torch.int16, device="cuda")
        b = torch.empty_like(a)
        fit = torch.rand(cfg.population, dtype=torch.float32, device="cuda")
        s.init_population(dj, torch.from_numpy(cfg.cur()).cuda(), a, round=0)
        for g in range(reps):
            s.ga_generation(dj, a, fit, b, round=0, generation=g)
            a, b = b, a
        s.sync_status()
        print("generation_large", int(a.sum().item()))
    else:
        raise SystemExit("unknown case %r" % case)
    s.close()


if __name__ == "__main__":
    main(sys.argv[1] if len(sys.argv) > 1 else "fitness_stress",
         generations=int(sys.argv[2]) if len(sys.argv) > 2 else 2)
