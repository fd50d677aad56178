"""Inside a round the generations run on specialised kernels: problems with more than 256 jobs
keep their population as shared rows (indices into a row pool, copy on write), problems with
at most 256 jobs and 32 nodes use a thread-per-row kernel.  Either way the round must equal,
bit for bit, the same round made of the dense entry points called one by one, which the other
tests pin to the oracle; the last generation is also checked against the oracle directly
(teacher-forced)."""
import dataclasses

import numpy as np
import pytest

from helpers import REL_TOL, assert_close, feasible, setup
from paper_2008_12260_b200 import synth

pytestmark = pytest.mark.gpu

# name, nodes, GPUs per node, jobs, seed, grid, population, generations, mutation, what it exercises
CASES = [
    # half of the rows perturbed per generation: the pool's half in use fills up and the live
    # rows move to the other half several times
    synth.Config("store-compaction", 32, 8, 300, 11, 16, 8, 48, 24, num_elite=3, mutate_prob=0.5,
                 init_prob=0.3, with_history=True, random_cur=True),
    # every row perturbed in every generation and a pool with room for two worst-case generations only:
    # a candidate may take its full J + 16 slots per generation without the pool running out
    synth.Config("store-all-perturbed", 16, 4, 280, 21, 16, 8, 20, 10, num_elite=1, mutate_prob=1.0,
                 init_prob=1.0, with_history=True, random_cur=True),
    # a current allocation that breaks every rule (node sizes, replica caps, interference) on large
    # nodes: rows hold more GPUs before the row caps than a summary can say
    synth.Config("store-infeasible-current", 8, 1500, 300, 22, 16, 8, 24, 6, num_elite=2, mutate_prob=0.3,
                 init_prob=0.6, with_history=True, random_cur=False),
    # few large nodes: more jobs on a node than a block lists per node (column scan through the
    # indices), and many GPUs per job
    synth.Config("store-crowded-nodes", 8, 64, 400, 12, 16, 8, 32, 12, num_elite=2, mutate_prob=0.3,
                 init_prob=0.5, with_history=True, random_cur=True),
    # many small nodes and frequent growth: rows that occupy more nodes than a record holds
    synth.Config("store-wide-rows", 64, 4, 260, 13, 16, 8, 32, 60, num_elite=2, mutate_prob=0.9,
                 init_prob=0.9, with_history=True, random_cur=False),
    # no current allocation, inactive jobs, ragged job count
    synth.Config("store-plain", 16, 8, 257, 14, 16, 8, 20, 6, num_elite=1, mutate_prob=0.1),
    # the widest rows the store takes (512 nodes: four 16-byte pieces per lane of a row's group)
    synth.Config("store-512-nodes", 512, 2, 600, 15, 16, 8, 12, 10, num_elite=2, mutate_prob=0.2,
                 init_prob=0.3, with_history=True, random_cur=True),
    # rows whose pieces do not fill the lanes evenly (17 pieces), many jobs per candidate
    synth.Config("store-ragged-pieces", 136, 4, 1100, 16, 16, 8, 10, 8, num_elite=1, mutate_prob=0.15,
                 init_prob=0.3, with_history=True, random_cur=True),
    # the large workload itself (the configuration the benchmark times), ten generations
    dataclasses.replace(synth.LARGE, name="store-large", generations=10),
    # thread-per-row kernel: more jobs on a node than its list holds (column scan in shared memory)
    synth.Config("small-crowded-nodes", 8, 128, 256, 17, 16, 8, 24, 30, num_elite=2, mutate_prob=0.3,
                 init_prob=0.9, with_history=True, random_cur=True),
    # thread-per-row kernel: the widest rows it takes (32 nodes), row caps at work, inactive jobs
    synth.Config("small-32-nodes", 32, 4, 120, 18, 16, 8, 20, 15, num_elite=3, mutate_prob=0.6,
                 init_prob=0.6, with_history=True, random_cur=True),
    # thread-per-row kernel: three 16-byte pieces per row, no current allocation
    synth.Config("small-24-nodes", 24, 2, 90, 19, 16, 8, 16, 10, num_elite=1, mutate_prob=0.4, init_prob=0.4),
]


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2008_12260_b200 import api
    assert torch.cuda.is_available()
    return torch, api


def _stepwise(torch, s, dj, cfg, d_cur, rnd, gens, penalise):
    dev = "cuda:0"
    sp = torch.empty(s.table_shape, dtype=torch.float32, device=dev)
    s.build_speedup_table(dj, None, sp, None)
    rf = None
    if penalise:
        rf = torch.empty(cfg.num_jobs, dtype=torch.float32, device=dev)
        s.compute_realloc_factor(dj, rf)
    a = torch.empty((cfg.population, cfg.num_jobs, cfg.num_nodes), dtype=torch.int16, device=dev)
    b = torch.empty_like(a)
    f = torch.empty(cfg.population, dtype=torch.float32, device=dev)
    kw = dict(p=cfg.p, active=dj.tensors["active"])
    if penalise:
        kw.update(cur=d_cur, realloc_factor=rf)
    s.init_population(dj, d_cur, a, round=rnd)
    s.eval_fitness(a, sp, f, **kw)
    prev = None
    for g in range(gens):
        prev = (a.cpu().numpy().copy(), f.cpu().numpy().copy())
        s.ga_generation(dj, a, f, b, round=rnd, generation=g)
        a, b = b, a
        s.eval_fitness(a, sp, f, **kw)
    return a.cpu().numpy(), f.cpu().numpy(), sp.cpu().numpy(), prev


@pytest.mark.parametrize("cfg", CASES, ids=lambda c: c.name)
def test_store_round_equals_dense_stepwise_round(gpu, oracle, cfg):
    torch, api = gpu
    cl, jobs = setup(cfg)
    if cfg.name in ("store-plain", "small-32-nodes"):
        jobs.active[::7] = 0
        jobs = setup_fair(jobs, cl)
    if cfg.name == "store-wide-rows":      # six jobs share the cluster, so their rows can spread
        jobs.active[6:] = 0
        jobs = setup_fair(jobs, cl)
    cur = cfg.cur(jobs) if cfg.random_cur else None
    if cfg.name == "store-infeasible-current":
        cur = synth.random_raw_population(1, cfg.num_jobs, cl, 77, density=0.5, v_hi=1400)[0]
        jobs.k_cap[::3] = 2
        assert cur.sum(axis=1).max() > 2047
    penalise = cur is not None
    rnd = 3
    s = api.scheduler_for(cfg, stream=torch.cuda.current_stream().cuda_stream)
    if cfg.name in ("store-compaction", "store-all-perturbed"):
        # a pool with room for two worst-case generations per half: the rows have to move every
        # other generation or so
        rows, worst = cfg.population * cfg.num_jobs, cfg.population * (cfg.num_jobs + 16)
        s.set_store_budget(2 * (cfg.num_nodes * 2 + 32) * (rows + 2 * worst + 64))
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
    assert np.array_equal(pop, ref_pop)
    assert np.array_equal(fit.view(np.uint32), ref_fit.view(np.uint32))
    i = int(np.argmax(fit))
    assert np.array_equal(best.cpu().numpy(), pop[i]) and float(bf.item()) == fit[i]
    for c in range(cfg.population):
        assert feasible(pop[c], cl.node_capacity, jobs.k_cap, cl.n_max)
    if cfg.name in ("store-compaction", "store-all-perturbed"):
        assert s.store_moves() >= 3
    elif cfg.name.startswith("store-"):
        assert s.store_moves() == 0
    if cfg.name == "store-crowded-nodes":
        assert (pop > 0).sum(axis=1).max() > 16      # more jobs on a node than a block lists
    if cfg.name == "small-crowded-nodes":
        assert (pop > 0).sum(axis=1).max() > 32
    if cfg.name == "store-wide-rows":
        assert (pop > 0).sum(axis=2).max() > 8       # rows wider than a record

    # the last generation against the oracle, from the population and fitness before it
    want = oracle.ga_generation(prev[0], prev[1], cl.node_capacity, jobs.k_cap, cl.k_max, cl.n_max, cfg.num_elite,
                                synth.prob_to_threshold(cfg.mutate_prob), cfg.seed, rnd, cfg.generations - 1,
                                active=jobs.active)
    assert np.array_equal(pop, want)
    rf_ref = oracle.realloc_factor(jobs.age_sec, jobs.num_restarts, cfg.delta_sec) if penalise else None
    fit_ref = oracle.eval_fitness(pop, sp.astype(np.float64), cl.k_max, cl.n_max, cfg.p, cfg.speedup_floor,
                                  cur=cur, realloc=rf_ref, active=jobs.active)
    assert_close(fit, fit_ref, what="fitness of the final population")
    s.close()


def setup_fair(jobs, cl):
    from helpers import with_fair_share
    return with_fair_share(jobs, cl)


def test_store_round_replays_as_graph_and_is_reproducible(gpu):
    torch, api = gpu
    cfg = CASES[0]
    cl, jobs = setup(cfg)
    cur = cfg.cur(jobs)
    outs = {}
    for graphs in (False, True):
        s = api.scheduler_for(cfg, stream=torch.cuda.Stream().cuda_stream)
        s.set_graphs(graphs)
        dj = api.DeviceJobs(jobs, "cuda:0", torch)
        d_cur = torch.from_numpy(cur).cuda()
        best = torch.empty((cfg.num_jobs, cfg.num_nodes), dtype=torch.int16, device="cuda:0")
        bf = torch.zeros(1, dtype=torch.float32, device="cuda:0")
        torch.cuda.synchronize()
        res = []
        for rnd in range(5):
            s.schedule_round(dj, d_cur, best, bf, round=rnd % 3, generations=10)
            s.sync_status()
            res.append((best.cpu().numpy().copy(), float(bf.item())))
        outs[graphs] = res
        s.close()
    for (b0, f0), (b1, f1) in zip(outs[False], outs[True]):
        assert np.array_equal(b0, b1) and f0 == f1
    assert np.array_equal(outs[True][0][0], outs[True][3][0]) and outs[True][0][1] == outs[True][3][1]
