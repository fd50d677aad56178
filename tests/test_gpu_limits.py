"""The documented maxima and the degenerate sizes, against the oracle:
  * the widest cluster the library takes (SCHED_MAX_NODES = 8192 nodes) with the largest table
    dimensions (k_max = n_max = 1024): table build, fitness, repair, initial population, generation;
  * no jobs at all, a population of one, a single node."""
import numpy as np
import pytest

from helpers import assert_close, feasible, with_fair_share
from paper_2008_12260_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2008_12260_b200 import api
    assert torch.cuda.is_available()
    return torch, api


class _J:
    def __init__(self, k_cap=None, active=None):
        self.k_cap = k_cap
        self.active = active


def test_widest_cluster_operators_and_fitness(gpu, oracle):
    torch, api = gpu
    NN, J, P, k_max, n_max = 8192, 5, 4, 1024, 1024
    rng = np.random.default_rng(3)
    cap = rng.integers(0, 4, NN).astype(np.int16)
    cl = synth.Cluster(cap)
    seed, rnd = 0x1234567, 2
    thr = synth.prob_to_threshold(0.8)
    s = api.Scheduler(node_capacity=cap, num_jobs=J, grid_m=1, grid_s=1, population=P, k_max=k_max, n_max=n_max,
                      thr_mutate=thr, thr_init=thr, num_elite=1, seed=seed, speedup_floor=1e-3,
                      stream=torch.cuda.current_stream().cuda_stream)
    k_cap = np.array([1024, 700, 5000, 3, 0], np.int32)
    dj = api.DeviceJobs(_J(k_cap, None), "cuda:0", torch)

    # repair of raw matrices: rows over k_max GPUs and over n_max nodes, every node over capacity
    raw = synth.random_raw_population(P, J, cl, seed=9, density=0.4, v_hi=5)
    d = torch.from_numpy(raw).cuda()
    s.repair_population(dj, d, round=rnd, generation=7)
    s.sync_status()
    out = d.cpu().numpy()
    for c in range(P):
        want = oracle.repair(raw[c], cap, k_cap, k_max, n_max, seed, rnd, c, 7)
        assert np.array_equal(out[c], want), c
        assert feasible(out[c], cap, np.minimum(k_cap, k_max), n_max)
    assert out.sum(axis=2).max() > 512 and (out > 0).sum(axis=2).max() > 256     # far beyond the usual 64 x 64 tables

    # fitness of the repaired matrices on the largest table
    table = rng.uniform(0.2, 2.0, (J, k_max + 1, n_max + 1)).astype(np.float32)
    table[:, 0, :] = 0.0
    table[:, :, 0] = 0.0
    cur = out[1].copy()
    rf = rng.uniform(0.3, 0.9, J).astype(np.float32)
    d_table, d_cur, d_rf = (torch.from_numpy(a).cuda() for a in (table, cur, rf))
    fit = torch.empty(P, dtype=torch.float32, device="cuda")
    for p in (-1.0, 0.5):
        s.eval_fitness(d, d_table, fit, p=p, cur=d_cur, realloc_factor=d_rf)
        s.sync_status()
        ref = oracle.eval_fitness(out, table.astype(np.float64), k_max, n_max, p, 1e-3, cur=cur, realloc=rf.astype(np.float64))
        assert_close(fit.cpu().numpy(), ref, what="p=%g" % p)

    # initial population and one generation
    init = torch.empty((P, J, NN), dtype=torch.int16, device="cuda")
    s.init_population(dj, d_cur, init, round=rnd)
    want = oracle.init_population(P, cur, J, cap, k_cap, k_max, n_max, thr, seed, rnd)
    assert np.array_equal(init.cpu().numpy(), want)
    s.eval_fitness(init, d_table, fit, p=-1.0, cur=d_cur, realloc_factor=d_rf)
    child = torch.empty_like(init)
    s.ga_generation(dj, init, fit, child, round=rnd, generation=0)
    s.sync_status()
    want = oracle.ga_generation(want, fit.cpu().numpy(), cap, k_cap, k_max, n_max, 1, thr, seed, rnd, 0)
    assert np.array_equal(child.cpu().numpy(), want)
    s.close()


def test_largest_table_dimensions(gpu, oracle):
    """k_max = n_max = 1024 on 8192 nodes of one GPU: every (K, N) pair with N <= K is valid."""
    torch, api = gpu
    cl = synth.uniform_cluster(8192, 1)
    jobs = synth.draw_jobs(2, 41, 16, 8, 1024)
    jobs = with_fair_share(jobs, cl, fair=(3, 3))
    s = api.Scheduler(node_capacity=cl.node_capacity, num_jobs=2, grid_m=16, grid_s=8, population=2, k_max=1024,
                      n_max=1024, stream=torch.cuda.current_stream().cuda_stream)
    dj = api.DeviceJobs(jobs, "cuda:0", torch)
    gp = torch.empty(s.table_shape, dtype=torch.float32, device="cuda")
    sp = torch.empty_like(gp)
    am = torch.empty(s.table_shape, dtype=torch.uint16, device="cuda")
    s.build_speedup_table(dj, gp, sp, am)
    s.sync_status()
    ref_gp, ref_sp, ref_am = oracle.build_speedup_table(jobs, cl.node_capacity, 1024, 1024, 8)
    assert tuple(gp.shape) == (2, 1025, 1025)
    assert_close(gp.cpu().numpy(), ref_gp, what="goodput")
    assert_close(sp.cpu().numpy(), ref_sp, what="speedup")
    assert (ref_gp[:, 1024, 1024] > 0).all() and (ref_gp[:, 5, 6] == 0).all()
    s.close()


def test_no_jobs_population_of_one_single_node(gpu, oracle):
    torch, api = gpu
    stream = torch.cuda.current_stream().cuda_stream
    # no jobs: every call succeeds and a round returns an empty matrix
    s = api.Scheduler(node_capacity=np.array([4, 4], np.int16), num_jobs=0, grid_m=4, grid_s=2, population=3, stream=stream)
    pop = torch.empty((3, 0, 2), dtype=torch.int16, device="cuda")             # (empty tensors: NULL pointers)
    fit = torch.full((3,), -1.0, dtype=torch.float32, device="cuda")
    table = torch.empty(s.table_shape, dtype=torch.float32, device="cuda")
    s.eval_fitness(pop, table, fit, p=-1.0)
    s.repair_population(None, pop, round=0, generation=0)
    s.sync_status()
    ref = oracle.eval_fitness(np.zeros((3, 0, 2), np.int16), np.zeros((0, 9, 3)), 8, 2, -1.0, 1e-3)
    assert np.array_equal(fit.cpu().numpy(), ref.astype(np.float32))
    s.close()

    # one candidate, one node, one job
    cfg = synth.Config("one", 1, 4, 1, 6, 8, 4, 1, 5, num_elite=1, mutate_prob=1.0, init_prob=1.0, with_history=True)
    cl = cfg.cluster()
    jobs = with_fair_share(cfg.jobs(), cl)
    s = api.scheduler_for(cfg, stream=stream)
    dj = api.DeviceJobs(jobs, "cuda:0", torch)
    cur = np.array([[2]], np.int16)
    best = torch.empty((1, 1), dtype=torch.int16, device="cuda")
    bf = torch.zeros(1, dtype=torch.float32, device="cuda")
    s.schedule_round(dj, torch.from_numpy(cur).cuda(), best, bf, round=1, generations=5)
    s.sync_status()
    # the only candidate is the elite of every generation: the current allocation, never penalised
    assert np.array_equal(best.cpu().numpy(), cur)
    ref_best, ref_fit = oracle.schedule_round(jobs, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s, 1, cfg.p, cfg.delta_sec,
                                              cfg.speedup_floor, 1, synth.prob_to_threshold(1.0), synth.prob_to_threshold(1.0),
                                              cfg.seed, 1, 5, cur)
    assert np.array_equal(ref_best, cur)
    assert_close([float(bf.item())], [ref_fit], rel=2e-5, what="one candidate")   # (two table entries' errors compound)
    s.close()
