"""Bit-exact parity of the population-search operators (repair, initial population, one
generation) against the oracle, given the same random stream; teacher-forced: at every
generation the oracle consumes the population and fp32 fitness the CUDA path produced."""
import numpy as np
import pytest

from helpers import REL_TOL, assert_close, feasible, setup, with_fair_share
from paper_2008_12260_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2008_12260_b200 import api
    assert torch.cuda.is_available()
    return torch, api


def _sched(gpu, cl, J, P, seed=5, thr_mutate=0, thr_init=0, num_elite=0, p=-1.0):
    torch, api = gpu
    return api.Scheduler(node_capacity=cl.node_capacity, num_jobs=J, grid_m=1, grid_s=1, population=P,
                         p=p, thr_mutate=thr_mutate, thr_init=thr_init, num_elite=num_elite, seed=seed,
                         stream=torch.cuda.current_stream().cuda_stream)


class _J:   # minimal job view for DeviceJobs: only k_cap / active matter to the operators
    def __init__(self, k_cap=None, active=None):
        self.k_cap = k_cap
        self.active = active


CLUSTERS = {
    "tiny": synth.uniform_cluster(4, 4),
    "testbed": synth.uniform_cluster(16, 4),
    "odd": synth.Cluster(np.array([8, 4, 4, 2, 1, 0, 3], np.int16)),
    "wide": synth.uniform_cluster(72, 8),
    "wide_ragged": synth.uniform_cluster(45, 2),
}


@pytest.mark.parametrize("name", list(CLUSTERS))
def test_repair_bit_exact(gpu, oracle, name):
    torch, api = gpu
    cl = CLUSTERS[name]
    J, P = 23, 37
    raw = synth.random_raw_population(P, J, cl, seed=31, density=0.35, v_hi=9)
    raw[3] = 0
    raw[4, :, :] = 30000                       # saturated garbage
    raw[5, ::2] = -4                           # negative entries are cleared
    rng = np.random.default_rng(2)
    k_cap = rng.integers(0, cl.k_max + 5, J).astype(np.int32)
    active = (rng.uniform(size=J) < 0.8).astype(np.uint8)
    s = _sched(gpu, cl, J, P, seed=0xABCDEF0123)
    dj = api.DeviceJobs(_J(k_cap, active), "cuda:0", torch)
    d = torch.from_numpy(raw).cuda()
    s.repair_population(dj, d, round=3, generation=11, first_candidate=100)
    s.sync_status()
    out = d.cpu().numpy()
    for c in range(P):
        ref = oracle.repair(raw[c], cl.node_capacity, k_cap, cl.k_max, cl.n_max, 0xABCDEF0123, 3, 100 + c, 11,
                            active=active)
        assert np.array_equal(out[c], ref), (name, c)
        assert feasible(out[c], np.maximum(cl.node_capacity, 0), np.clip(k_cap, 0, cl.k_max), cl.n_max)
    # feasible input is a fixed point, whatever the stream; NULL jobs = no caps, all active
    s.repair_population(dj, d, round=9, generation=0)
    assert np.array_equal(d.cpu().numpy(), out)
    d2 = torch.from_numpy(raw).cuda()
    s.repair_population(None, d2, round=3, generation=11, first_candidate=100, count=P - 2)
    out2 = d2.cpu().numpy()
    for c in range(P - 2):
        ref = oracle.repair(raw[c], cl.node_capacity, None, cl.k_max, cl.n_max, 0xABCDEF0123, 3, 100 + c, 11)
        assert np.array_equal(out2[c], ref)
    assert np.array_equal(out2[P - 2:], raw[P - 2:])         # beyond `count`: untouched
    s.close()


def test_repair_n_max_and_k_cap_rows(gpu, oracle):
    torch, api = gpu
    cl = synth.uniform_cluster(80, 2)          # n_max = 64 < 80 nodes, k_max = 64 < 160 GPUs
    J, P = 3, 6
    raw = np.ones((P, J, 80), np.int16)
    raw[1] = 2
    raw[2, 0, 5:] = 0
    s = _sched(gpu, cl, J, P, seed=8)
    d = torch.from_numpy(raw).cuda()
    s.repair_population(None, d, round=0, generation=0)
    out = d.cpu().numpy()
    for c in range(P):
        assert np.array_equal(out[c], oracle.repair(raw[c], cl.node_capacity, None, 64, 64, 8, 0, c, 0))
    s.close()


@pytest.mark.parametrize("cfg", [synth.TINY, synth.TESTBED], ids=lambda c: c.name)
def test_init_population_bit_exact(gpu, oracle, cfg):
    torch, api = gpu
    cl, jobs = setup(cfg)
    cur = synth.random_feasible_allocation(cl, cfg.num_jobs, 77)
    jobs.active[1] = 0
    jobs.k_cap[2] = 1
    thr = synth.prob_to_threshold(0.3)
    s = _sched(gpu, cl, cfg.num_jobs, cfg.population, seed=cfg.seed, thr_init=thr)
    dj = api.DeviceJobs(_J(jobs.k_cap, jobs.active), "cuda:0", torch)
    out = torch.full((cfg.population, cfg.num_jobs, cfg.num_nodes), -1, dtype=torch.int16, device="cuda:0")
    s.init_population(dj, torch.from_numpy(cur).cuda(), out, round=4)
    ref = oracle.init_population(cfg.population, cur, cfg.num_jobs, cl.node_capacity, jobs.k_cap, cl.k_max,
                                 cl.n_max, thr, cfg.seed, 4, active=jobs.active)
    assert np.array_equal(out.cpu().numpy(), ref)
    s.init_population(dj, None, out, round=4)                 # empty cluster
    ref = oracle.init_population(cfg.population, None, cfg.num_jobs, cl.node_capacity, jobs.k_cap, cl.k_max,
                                 cl.n_max, thr, cfg.seed, 4, active=jobs.active)
    assert np.array_equal(out.cpu().numpy(), ref)
    s.close()


def _teacher_forced(gpu, oracle, cl, J, P, gens, seed, mutate_prob, num_elite, k_cap=None, active=None,
                    cur=None, init_prob=0.3, check_fitness=True):
    torch, api = gpu
    thr_m, thr_i = synth.prob_to_threshold(mutate_prob), synth.prob_to_threshold(init_prob)
    s = _sched(gpu, cl, J, P, seed=seed, thr_mutate=thr_m, thr_init=thr_i, num_elite=num_elite)
    dj = api.DeviceJobs(_J(k_cap, active), "cuda:0", torch)
    rng = np.random.default_rng(seed)
    table = rng.uniform(0.1, 3.0, s.table_shape).astype(np.float32)
    table[:, 0, :] = 0; table[:, :, 0] = 0
    d_table = torch.from_numpy(table).cuda()
    d_cur = None if cur is None else torch.from_numpy(cur).cuda()
    rf = rng.uniform(0.3, 1.0, J).astype(np.float32)
    d_rf = torch.from_numpy(rf).cuda()
    d_act = dj.tensors.get("active")
    a = torch.empty((P, J, cl.num_nodes), dtype=torch.int16, device="cuda:0")
    b = torch.empty_like(a)
    fit = torch.empty(P, dtype=torch.float32, device="cuda:0")
    s.init_population(dj, d_cur, a, round=1)
    for g in range(gens):
        s.eval_fitness(a, d_table, fit, p=-1.0, cur=d_cur, realloc_factor=d_rf if cur is not None else None,
                       active=d_act)
        pop_h, fit_h = a.cpu().numpy(), fit.cpu().numpy()
        if check_fitness:
            ref_f = oracle.eval_fitness(pop_h, table.astype(np.float64), cl.k_max, cl.n_max, -1.0, 1e-3,
                                        cur=cur, realloc=rf.astype(np.float64) if cur is not None else None,
                                        active=active)
            assert_close(fit_h, ref_f, what="fitness gen %d" % g)
        s.ga_generation(dj, a, fit, b, round=1, generation=g)
        ref = oracle.ga_generation(pop_h, fit_h, cl.node_capacity, k_cap, cl.k_max, cl.n_max, num_elite,
                                   thr_m, seed, 1, g, active=active)
        got = b.cpu().numpy()
        assert np.array_equal(got, ref), "generation %d differs" % g
        a, b = b, a
    s.sync_status()
    s.close()
    return got


@pytest.mark.parametrize("cfg", [synth.TINY, synth.TESTBED], ids=lambda c: c.name)
def test_generations_teacher_forced(gpu, oracle, cfg):
    cl, jobs = setup(cfg)
    cur = cfg.cur() if cfg.random_cur else None
    last = _teacher_forced(gpu, oracle, cl, cfg.num_jobs, cfg.population, 12, cfg.seed, cfg.mutate_prob,
                           cfg.num_elite, k_cap=jobs.k_cap, cur=cur)
    assert last.any()


def test_generations_with_caps_inactive_and_odd_cluster(gpu, oracle):
    cl = CLUSTERS["odd"]
    J, P = 19, 33
    rng = np.random.default_rng(3)
    k_cap = rng.integers(1, 9, J).astype(np.int32)
    active = (rng.uniform(size=J) < 0.7).astype(np.uint8)
    _teacher_forced(gpu, oracle, cl, J, P, 8, 99, 0.6, 5, k_cap=k_cap, active=active)
    _teacher_forced(gpu, oracle, cl, J, P, 3, 100, 1.0, 0, k_cap=k_cap)            # every row perturbed
    _teacher_forced(gpu, oracle, cl, J, P, 3, 101, 0.0, P, k_cap=k_cap)            # all elites: a sort


def test_large_config_one_generation(gpu, oracle):
    """256 x 8 cluster, 1024 jobs, population 512: the bench's launch configuration."""
    cfg = synth.LARGE
    cl, jobs = setup(cfg)
    _teacher_forced(gpu, oracle, cl, cfg.num_jobs, cfg.population, 2, cfg.seed, cfg.mutate_prob,
                    cfg.num_elite, k_cap=jobs.k_cap, cur=cfg.cur(), init_prob=cfg.init_prob)


def test_fitness_ties_rank_by_index(gpu, oracle):
    torch, api = gpu
    cl = synth.uniform_cluster(4, 4)
    J, P = 6, 16
    s = _sched(gpu, cl, J, P, seed=1, num_elite=4)
    pop = np.zeros((P, J, 4), np.int16)
    for i in range(P):
        pop[i, i % J, i % 4] = 1 + i % 3
    fit = np.array([1, 1, 2, 2, 0.5, 2, 1, -0.0, 0.0, 1, 3, 3, 0.25, 1, 2, 3], np.float32)
    out = torch.empty((P, J, 4), dtype=torch.int16, device="cuda:0")
    s.ga_generation(None, torch.from_numpy(pop).cuda(), torch.from_numpy(fit).cuda(), out, round=0, generation=0)
    ref = oracle.ga_generation(pop, fit, cl.node_capacity, None, cl.k_max, cl.n_max, 4, 0, 1, 0, 0)
    assert np.array_equal(out.cpu().numpy(), ref)
    assert np.array_equal(ref[:4], pop[[10, 11, 15, 2]])
    s.close()
