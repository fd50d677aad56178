"""The scheduling-round driver: equal to the step-by-step entry points, reproducible,
feasible, consistent with the oracle's fitness, and the host-buffer variant."""
import numpy as np
import pytest

from helpers import REL_TOL, assert_close, feasible, setup
from paper_2008_12260_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2008_12260_b200 import api
    assert torch.cuda.is_available()
    return torch, api


def _round(gpu, cfg, jobs, cur, gens, rnd=0):
    torch, api = gpu
    s = api.scheduler_for(cfg, stream=torch.cuda.current_stream().cuda_stream)
    dj = api.DeviceJobs(jobs, "cuda:0", torch)
    best = torch.full((cfg.num_jobs, cfg.num_nodes), -1, dtype=torch.int16, device="cuda:0")
    bf = torch.zeros(1, dtype=torch.float32, device="cuda:0")
    d_cur = None if cur is None else torch.from_numpy(cur).cuda()
    s.schedule_round(dj, d_cur, best, bf, round=rnd, generations=gens)
    s.sync_status()
    pop = torch.empty((cfg.population, cfg.num_jobs, cfg.num_nodes), dtype=torch.int16, device="cuda:0")
    fit = torch.empty(cfg.population, dtype=torch.float32, device="cuda:0")
    s.get_population(pop, fit)
    torch.cuda.synchronize()
    return s, dj, best.cpu().numpy(), float(bf.item()), pop.cpu().numpy(), fit.cpu().numpy()


@pytest.mark.parametrize("cfg", [synth.TINY, synth.TESTBED], ids=lambda c: c.name)
def test_round_equals_stepwise_calls_and_oracle_fitness(gpu, oracle, cfg):
    torch, api = gpu
    cl, jobs = setup(cfg)
    cur = cfg.cur()
    gens = min(cfg.generations, 25)
    s, dj, best, bf, pop, fit = _round(gpu, cfg, jobs, cur, gens, rnd=2)

    # the same round through the individual entry points
    dev = "cuda:0"
    sp = torch.empty(s.table_shape, dtype=torch.float32, device=dev)
    s.build_speedup_table(dj, None, sp, None)
    rf = torch.empty(cfg.num_jobs, dtype=torch.float32, device=dev)
    s.compute_realloc_factor(dj, rf)
    d_cur = torch.from_numpy(cur).cuda()
    a = torch.empty((cfg.population, cfg.num_jobs, cfg.num_nodes), dtype=torch.int16, device=dev)
    b = torch.empty_like(a)
    f = torch.empty(cfg.population, dtype=torch.float32, device=dev)
    s.init_population(dj, d_cur, a, round=2)
    s.eval_fitness(a, sp, f, p=cfg.p, cur=d_cur, realloc_factor=rf, active=dj.tensors["active"])
    f0 = f.cpu().numpy().copy()
    for g in range(gens):
        s.ga_generation(dj, a, f, b, round=2, generation=g)
        a, b = b, a
        s.eval_fitness(a, sp, f, p=cfg.p, cur=d_cur, realloc_factor=rf, active=dj.tensors["active"])
    assert np.array_equal(a.cpu().numpy(), pop)
    assert np.array_equal(f.cpu().numpy().view(np.uint32), fit.view(np.uint32))
    i = int(np.argmax(fit))
    assert np.array_equal(best, pop[i]) and bf == fit[i]
    assert bf >= f0[0]                      # never worse than keeping the current allocation

    # oracle: realloc factors, table, and the fitness of the final population
    rf_ref = oracle.realloc_factor(jobs.age_sec, jobs.num_restarts, cfg.delta_sec)
    assert_close(rf.cpu().numpy(), rf_ref, what="realloc factor")
    _, sp_ref, _ = oracle.build_speedup_table(jobs, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s)
    assert_close(sp.cpu().numpy(), sp_ref, what="speedup")
    # the fitness arithmetic is checked on the inputs the CUDA path itself used (its fp32 table and
    # factors, each within 1e-5 of the oracle's just above), so the stated tolerance applies unchanged
    fit_ref = oracle.eval_fitness(pop, sp.cpu().numpy().astype(np.float64), cl.k_max, cl.n_max, cfg.p,
                                  cfg.speedup_floor, cur=cur, realloc=rf.cpu().numpy().astype(np.float64),
                                  active=jobs.active)
    assert_close(fit, fit_ref, what="fitness of the final population")
    for c in range(cfg.population):
        assert feasible(pop[c], cl.node_capacity, jobs.k_cap, cl.n_max)
    s.close()


def test_large_config_round_equals_stepwise(gpu, oracle):
    """The large configuration (batched row kernel, work-list column repair, fitness from row
    summaries) for three generations: the round must equal the entry points called one by one,
    whose fitness reads the dense matrices; the final fitness is checked against the oracle on a
    sample of candidates."""
    torch, api = gpu
    cfg = synth.LARGE
    cl, jobs = setup(cfg)
    cur = cfg.cur()
    s, dj, best, bf, pop, fit = _round(gpu, cfg, jobs, cur, 3, rnd=7)
    dev = "cuda:0"
    sp = torch.empty(s.table_shape, dtype=torch.float32, device=dev)
    s.build_speedup_table(dj, None, sp, None)
    rf = torch.empty(cfg.num_jobs, dtype=torch.float32, device=dev)
    s.compute_realloc_factor(dj, rf)
    d_cur = torch.from_numpy(cur).cuda()
    a = torch.empty((cfg.population, cfg.num_jobs, cfg.num_nodes), dtype=torch.int16, device=dev)
    b = torch.empty_like(a)
    f = torch.empty(cfg.population, dtype=torch.float32, device=dev)
    s.init_population(dj, d_cur, a, round=7)
    s.eval_fitness(a, sp, f, p=cfg.p, cur=d_cur, realloc_factor=rf, active=dj.tensors["active"])
    for g in range(3):
        s.ga_generation(dj, a, f, b, round=7, generation=g)
        a, b = b, a
        s.eval_fitness(a, sp, f, p=cfg.p, cur=d_cur, realloc_factor=rf, active=dj.tensors["active"])
    assert np.array_equal(a.cpu().numpy(), pop)
    assert np.array_equal(f.cpu().numpy().view(np.uint32), fit.view(np.uint32))
    sample = sorted(set(range(0, 512, 8)) | {1, 100, 511})   # 66 candidates
    ref = oracle.eval_fitness(pop[sample], sp.cpu().numpy().astype(np.float64), cl.k_max, cl.n_max, cfg.p,
                              cfg.speedup_floor, cur=cur, realloc=rf.cpu().numpy().astype(np.float64),
                              active=jobs.active)
    assert_close(fit[sample], ref, what="large round fitness")
    for c in sample:
        assert feasible(pop[c], cl.node_capacity, jobs.k_cap, cl.n_max)
    s.close()


def test_round_is_reproducible_and_round_number_matters(gpu):
    cfg = synth.TESTBED
    cl, jobs = setup(cfg)
    cur = cfg.cur()
    r1 = _round(gpu, cfg, jobs, cur, 10, rnd=5)
    r2 = _round(gpu, cfg, jobs, cur, 10, rnd=5)
    r3 = _round(gpu, cfg, jobs, cur, 10, rnd=6)
    assert np.array_equal(r1[4], r2[4]) and np.array_equal(r1[2], r2[2]) and r1[3] == r2[3]
    assert not np.array_equal(r1[4], r3[4])
    for r in (r1, r2, r3):
        r[0].close()


def test_round_search_quality_against_oracle_round(gpu, oracle):
    """The two rounds may fork at fp32/fp64 near-ties, so only the outcome is compared: the
    CUDA round must reach a fitness close to the oracle's own round on the same inputs."""
    cfg = synth.TINY
    cl, jobs = setup(cfg)
    s, dj, best, bf, pop, fit = _round(gpu, cfg, jobs, None, 40)
    ob, of = oracle.schedule_round(jobs, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s, cfg.population,
                                   cfg.p, cfg.delta_sec, cfg.speedup_floor, cfg.num_elite,
                                   synth.prob_to_threshold(cfg.mutate_prob),
                                   synth.prob_to_threshold(cfg.init_prob), cfg.seed, 0, 40, None)
    assert bf > 0.5 * of and of > 0.5 * bf
    s.close()


def test_zero_generations_and_no_current_allocation(gpu, oracle):
    cfg = synth.TINY
    cl, jobs = setup(cfg)
    s, dj, best, bf, pop, fit = _round(gpu, cfg, jobs, None, 0)
    ref = oracle.init_population(cfg.population, None, cfg.num_jobs, cl.node_capacity, jobs.k_cap, cl.k_max,
                                 cl.n_max, synth.prob_to_threshold(cfg.init_prob), cfg.seed, 0,
                                 active=jobs.active)
    assert np.array_equal(pop, ref)
    assert np.array_equal(best, pop[int(np.argmax(fit))])
    s.close()


def test_host_buffer_round(gpu):
    torch, api = gpu
    cfg = synth.TESTBED
    cl, jobs = setup(cfg)
    cur = cfg.cur()
    s, dj, best, bf, pop, fit = _round(gpu, cfg, jobs, cur, 8, rnd=1)
    hj = api.HostJobs(jobs, torch)
    h_cur = torch.from_numpy(cur).pin_memory()
    h_best = torch.empty((cfg.num_jobs, cfg.num_nodes), dtype=torch.int16).pin_memory()
    h_bf = torch.zeros(1, dtype=torch.float32).pin_memory()
    s.schedule_round_host(hj, h_cur, h_best, h_bf, round=1, generations=8)
    assert np.array_equal(h_best.numpy(), best) and float(h_bf.item()) == bf
    s.close()


def test_graph_replay_gives_the_same_rounds(gpu):
    """Rounds 3+ with unchanged buffers replay a captured CUDA graph; they must equal the same
    rounds run kernel by kernel, for every round number."""
    torch, api = gpu
    cfg = synth.TESTBED
    cl, jobs = setup(cfg)
    cur = cfg.cur()
    outs = {}
    for graphs in (False, True):
        s = api.scheduler_for(cfg, stream=torch.cuda.Stream().cuda_stream if graphs else torch.cuda.current_stream().cuda_stream)
        s.set_graphs(graphs)
        dj = api.DeviceJobs(jobs, "cuda:0", torch)
        d_cur = torch.from_numpy(cur).cuda()
        best = torch.empty((cfg.num_jobs, cfg.num_nodes), dtype=torch.int16, device="cuda:0")
        bf = torch.zeros(1, dtype=torch.float32, device="cuda:0")
        torch.cuda.synchronize()
        res = []
        for rnd in range(6):
            s.schedule_round(dj, d_cur, best, bf, round=rnd, generations=12)
            s.sync_status()
            res.append((best.cpu().numpy().copy(), float(bf.item())))
        outs[graphs] = (res, s.launch_count())
        s.close()
    for (b0, f0), (b1, f1) in zip(outs[False][0], outs[True][0]):
        assert np.array_equal(b0, b1) and f0 == f1
    assert outs[False][1] == outs[True][1]          # launches are accounted for under replay
    assert len({r[1] for r in outs[True][0]}) > 1    # the round number reaches the kernels


def test_graph_survives_scratch_reallocation(gpu):
    """A captured round holds raw scratch pointers; a later call that makes the context grow
    its scratch must not leave a stale graph behind."""
    torch, api = gpu
    cfg = synth.TESTBED
    cl, jobs = setup(cfg)
    s = api.scheduler_for(cfg, stream=torch.cuda.Stream().cuda_stream)
    dj = api.DeviceJobs(jobs, "cuda:0", torch)
    d_cur = torch.from_numpy(cfg.cur()).cuda()
    best = torch.empty((cfg.num_jobs, cfg.num_nodes), dtype=torch.int16, device="cuda:0")
    bf = torch.zeros(1, dtype=torch.float32, device="cuda:0")
    torch.cuda.synchronize()
    ref = []
    for rnd in range(4):
        s.schedule_round(dj, d_cur, best, bf, round=rnd, generations=6)
        s.sync_status()
        ref.append((best.cpu().numpy().copy(), float(bf.item())))
    # a much larger fitness call and a larger repair call reallocate the context's scratch
    big = torch.zeros((cfg.population * 8, cfg.num_jobs, cfg.num_nodes), dtype=torch.int16, device="cuda:0")
    table = torch.ones(s.table_shape, dtype=torch.float32, device="cuda:0")
    fit = torch.empty(big.shape[0], dtype=torch.float32, device="cuda:0")
    s.eval_fitness(big, table, fit, p=1.0)
    s.repair_population(None, big, round=0, generation=0)
    s.sync_status()
    for rnd in range(4):
        s.schedule_round(dj, d_cur, best, bf, round=rnd, generations=6)
        s.sync_status()
        assert np.array_equal(best.cpu().numpy(), ref[rnd][0]) and float(bf.item()) == ref[rnd][1]
    s.close()


def test_argument_errors(gpu):
    torch, api = gpu
    cfg = synth.TINY
    cl, jobs = setup(cfg)
    s = api.scheduler_for(cfg)
    dj = api.DeviceJobs(jobs, "cuda:0", torch)
    best = torch.empty((cfg.num_jobs, cfg.num_nodes), dtype=torch.int16, device="cuda:0")
    bf = torch.zeros(1, dtype=torch.float32, device="cuda:0")
    with pytest.raises(api.SchedError) as e:
        s.schedule_round(dj, None, None, bf, round=0, generations=1)
    assert e.value.code == -1
    with pytest.raises(api.SchedError):
        s.schedule_round(dj, None, best, bf, round=0, generations=-1)
    with pytest.raises(api.SchedError):
        s.ga_generation(None, best, bf, best, round=0, generation=0)          # in == out
    with pytest.raises(api.SchedError):
        s.eval_fitness(best, None, bf, p=-1.0, count=1)
    with pytest.raises(api.SchedError):
        s.get_population(best, bf)                                            # no round yet
    s.schedule_round(dj, None, best, bf, round=0, generations=1)              # still usable afterwards
    s.sync_status()
    s.close()


def test_host_entry_points_validate_their_arrays(gpu):
    """The host-buffer calls can read their inputs, so they reject what Eq. 8-11 and Sec. 4.2
    exclude before anything reaches the GPU."""
    import copy
    torch, api = gpu
    cfg = synth.TINY
    cl, jobs = setup(cfg)
    jobs.age_sec = np.full(cfg.num_jobs, 600.0, np.float32)
    jobs.num_restarts = np.zeros(cfg.num_jobs, np.int32)
    s = api.scheduler_for(cfg)
    J, NN = cfg.num_jobs, cfg.num_nodes
    h_best = torch.empty((J, NN), dtype=torch.int16)
    h_bf = torch.zeros(1, dtype=torch.float32)
    h_cur = torch.zeros((J, NN), dtype=torch.int16)

    def run(j, cur=h_cur):
        s.schedule_round_host(api.HostJobs(j, torch, pin=False), cur, h_best, h_bf, round=0, generations=1)

    run(jobs)                                          # the untouched inputs pass
    cases = [("alpha_grad", np.nan, -5), ("phi", np.inf, -5), ("age_sec", -np.inf, -5), ("beta_node", -1e-3, -1),
             ("gamma", 0.5, -1), ("m0", 0.0, -1), ("phi", -1.0, -1), ("num_restarts", -1, -1)]
    for field, value, code in cases:
        bad = copy.deepcopy(jobs)
        getattr(bad, field)[3] = value
        with pytest.raises(api.SchedError) as e:
            run(bad)
        assert e.value.code == code, (field, value, e.value.code)
        assert field in str(e.value)
    bad = copy.deepcopy(jobs)
    bad.m_max_total[2] = bad.m0[2] - 1                 # M_max below M0
    with pytest.raises(api.SchedError) as e:
        run(bad)
    assert e.value.code == -1
    bad = copy.deepcopy(jobs)
    bad.m_grid[1, 0] = 0
    with pytest.raises(api.SchedError) as e:
        run(bad)
    assert e.value.code == -1
    neg = h_cur.clone()
    neg[0, 0] = -1
    with pytest.raises(api.SchedError) as e:
        run(jobs, neg)
    assert e.value.code == -1

    table = np.ones(s.table_shape, np.float32)
    pop = np.zeros((2, J, NN), np.int16)
    out = np.zeros(2, np.float32)
    s.eval_fitness_host(pop, table, out, p=1.0)
    t2 = table.copy(); t2[1, 2, 1] = np.nan
    with pytest.raises(api.SchedError) as e:
        s.eval_fitness_host(pop, t2, out, p=1.0)
    assert e.value.code == -5
    t2[1, 2, 1] = -0.5
    with pytest.raises(api.SchedError) as e:
        s.eval_fitness_host(pop, t2, out, p=1.0)
    assert e.value.code == -1
    with pytest.raises(api.SchedError) as e:
        s.eval_fitness_host(pop, table, out, p=1.0, cur=np.zeros((J, NN), np.int16),
                            realloc_factor=np.full(J, 1.5, np.float32))
    assert e.value.code == -1
    run(jobs)                                          # the context is still usable
    s.close()


@pytest.mark.parametrize("nodes,gpn,J", [(2, 2, 3), (2, 4, 2)])
def test_search_against_the_brute_force_optimum(gpu, oracle, nodes, gpn, J, record_property):
    """Clusters small enough to enumerate: the best fitness of the search can never exceed the
    maximum of Eq. 14 over every feasible matrix; how close it gets is recorded, not required
    (the method is a heuristic, Sec. 4.3)."""
    import itertools
    torch, api = gpu
    cfg = synth.Config("quality", nodes, gpn, J, 40 + J, 16, 8, 32, 100, num_elite=2, mutate_prob=0.2)
    cl, jobs = setup(cfg)
    _, sp, _ = oracle.build_speedup_table(jobs, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s, want_argmax=False)
    mats = np.array(list(itertools.product(range(gpn + 1), repeat=J * nodes)), np.int16).reshape(-1, J, nodes)
    ok = np.array([feasible(m, cl.node_capacity, jobs.k_cap, cl.n_max) for m in mats])
    fit = oracle.eval_fitness(mats[ok], sp, cl.k_max, cl.n_max, cfg.p, cfg.speedup_floor)
    optimum = float(fit.max())
    for gens in (10, 100):
        s, dj, best, bf, pop, f = _round(gpu, cfg, jobs, None, gens)
        assert feasible(best, cl.node_capacity, jobs.k_cap, cl.n_max)
        assert bf <= optimum * (1 + REL_TOL)
        record_property("gap_after_%d_generations" % gens, 1.0 - bf / optimum)
        if gens == 100:
            assert bf >= 0.5 * optimum          # a search that found nothing would sit at the floor
        s.close()
