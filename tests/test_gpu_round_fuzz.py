"""Randomly drawn problem shapes through a whole round: the round's specialised kernels (row store,
thread-per-row kernel, fused batched kernel) against the same round made of the dense entry points
called one by one - populations and fitness bit for bit - and the last generation against the
oracle.  Shapes, probabilities, the current allocation (none / feasible / breaking every rule),
inactive jobs and small replica caps all vary with the seed.  POLLUX_FUZZ_CASES raises the number
of seeds for a longer sweep."""
import os

import numpy as np
import pytest

from helpers import assert_close, feasible, with_fair_share
from paper_2008_12260_b200 import synth
from test_gpu_round_kernels import _stepwise

pytestmark = pytest.mark.gpu

N_CASES = int(os.environ.get("POLLUX_FUZZ_CASES", "16"))


def draw_case(seed):
    g = np.random.default_rng(1000 + seed)
    nodes = int(g.choice([8, 16, 24, 32, 40, 64, 128, 256]))
    gpn = int(g.choice([1, 2, 4, 8, 16, 96]))
    if g.uniform() < 0.35 and nodes <= 32:
        jobs = int(g.integers(3, 257))            # thread-per-row kernel
    else:
        jobs = int(g.integers(257, 900))          # row store
    cfg = synth.Config("fuzz-%d" % seed, nodes, gpn, jobs, 5000 + seed, 16, 8, int(g.integers(6, 40)),
                       int(g.integers(2, 12)), p=float(g.choice([-1.0, -1.0, 0.5, 1.0, 0.0])),
                       num_elite=int(g.integers(0, 4)), mutate_prob=float(g.choice([0.02, 0.1, 0.3, 0.7, 1.0])),
                       init_prob=float(g.choice([0.0, 0.1, 0.5, 1.0])), with_history=bool(g.integers(0, 2)),
                       random_cur=True)
    kind = int(g.integers(0, 3))                  # current allocation: none / feasible / infeasible
    return cfg, kind, g


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2008_12260_b200 import api
    assert torch.cuda.is_available()
    return torch, api


@pytest.mark.parametrize("seed", range(N_CASES))
def test_random_round_equals_dense_stepwise_round(gpu, oracle, seed):
    torch, api = gpu
    cfg, kind, g = draw_case(seed)
    cl = cfg.cluster()
    jobs = cfg.jobs()
    if g.uniform() < 0.5:
        jobs.active[g.uniform(size=cfg.num_jobs) < 0.15] = 0
        if jobs.active.sum() == 0:
            jobs.active[0] = 1
    if g.uniform() < 0.5:
        small = g.uniform(size=cfg.num_jobs) < 0.3
        jobs.k_cap[small] = g.integers(0, 4, int(small.sum()))
    jobs = with_fair_share(jobs, cl)
    cur = None
    if kind == 1:
        cur = cfg.cur(jobs)
    elif kind == 2:
        cur = synth.random_raw_population(1, cfg.num_jobs, cl, 9000 + seed, density=float(g.uniform(0.02, 0.6)),
                                          v_hi=int(g.choice([3, 9, 200, 3000])))[0]
    penalise = cur is not None
    rnd = int(g.integers(0, 5))
    s = api.scheduler_for(cfg, stream=torch.cuda.current_stream().cuda_stream)
    dj = api.DeviceJobs(jobs, "cuda:0", torch)
    d_cur = None if cur is None else torch.from_numpy(cur).cuda()
    best = torch.full((cfg.num_jobs, cfg.num_nodes), -1, dtype=torch.int16, device="cuda:0")
    bf = torch.zeros(1, dtype=torch.float32, device="cuda:0")
    s.schedule_round(dj, d_cur, best, bf, round=rnd, generations=cfg.generations)
    s.sync_status()
    pop = torch.empty((cfg.population, cfg.num_jobs, cfg.num_nodes), dtype=torch.int16, device="cuda:0")
    fit = torch.empty(cfg.population, dtype=torch.float32, device="cuda:0")
    s.get_population(pop, fit)
    pop, fit = pop.cpu().numpy(), fit.cpu().numpy()

    ref_pop, ref_fit, sp, prev = _stepwise(torch, s, dj, cfg, d_cur, rnd, cfg.generations, penalise)
    what = "%s: %d nodes x %d, %d jobs, cur kind %d" % (cfg.name, cfg.num_nodes, cfg.gpus_per_node, cfg.num_jobs, kind)
    assert np.array_equal(pop, ref_pop), what
    assert np.array_equal(fit.view(np.uint32), ref_fit.view(np.uint32)), what
    i = int(np.argmax(fit))
    assert np.array_equal(best.cpu().numpy(), pop[i]) and float(bf.item()) == fit[i], what
    k_cap = np.minimum(np.maximum(jobs.k_cap, 0), cl.k_max)
    for c in range(cfg.population):
        assert feasible(pop[c], cl.node_capacity, k_cap, cl.n_max), what

    want = oracle.ga_generation(prev[0], prev[1], cl.node_capacity, jobs.k_cap, cl.k_max, cl.n_max, cfg.num_elite,
                                synth.prob_to_threshold(cfg.mutate_prob), cfg.seed, rnd, cfg.generations - 1,
                                active=jobs.active)
    assert np.array_equal(pop, want), what
    rf_ref = oracle.realloc_factor(jobs.age_sec, jobs.num_restarts, cfg.delta_sec) if penalise else None
    fit_ref = oracle.eval_fitness(pop, sp.astype(np.float64), cl.k_max, cl.n_max, cfg.p, cfg.speedup_floor,
                                  cur=cur, realloc=rf_ref, active=jobs.active)
    assert_close(fit, fit_ref, what=what)
    s.close()
