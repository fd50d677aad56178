"""Rack-level locality on the GPU (the third synchronisation pair named after Eq. 9): tables of
the rack class, the fitness that reads them for rows that span racks, and whole rounds, against
the oracle."""
import itertools

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


def _tables(gpu, cfg, cl, jobs, ar, br):
    torch, api = gpu
    dev = "cuda:0"
    s = api.scheduler_for(cfg, stream=torch.cuda.current_stream().cuda_stream)
    dj = api.DeviceJobs(jobs, dev, torch)
    d_ar, d_br = torch.from_numpy(ar).cuda(), torch.from_numpy(br).cuda()
    out = []
    for rack in (False, True):
        gp = torch.full(s.table_shape, -1.0, dtype=torch.float32, device=dev)
        sp = torch.full(s.table_shape, -1.0, dtype=torch.float32, device=dev)
        am = torch.full(s.table_shape, 7, dtype=torch.uint16, device=dev)
        if rack:
            s.build_speedup_table_rack(dj, d_ar, d_br, gp, sp, am)
        else:
            s.build_speedup_table(dj, gp, sp, am)
        s.sync_status()
        out.append((gp.cpu().numpy(), sp.cpu().numpy(), am.cpu().numpy()))
    s.close()
    return out


def _check_rack_table(oracle, jobs, grid_s, got, ref):
    gp, sp, am = got
    gp_r, sp_r, am_r = ref
    assert_close(gp, gp_r, what="rack goodput")
    assert_close(sp, sp_r, what="rack speedup")
    assert np.array_equal(am == 0xFFFF, am_r == 0xFFFF)
    fields = ("alpha_grad", "beta_grad", "alpha_local", "beta_local", "alpha_node", "beta_node", "alpha_rack",
              "beta_rack", "gamma", "phi", "m0", "m_max_total")
    for j, K, N in np.argwhere(am != am_r):
        i, s = divmod(int(am[j, K, N]), grid_s)
        par = [float(getattr(jobs, f)[j]) for f in fields]
        g, ok = oracle.goodput_rack(*par, int(K), int(N), 2, int(jobs.m_grid[j, i]), s)
        assert ok and g >= gp_r[j, K, N] * (1 - REL_TOL)


@pytest.mark.parametrize("cfg", [synth.TINY, synth.TESTBED], ids=lambda c: c.name)
def test_rack_table_matches_oracle(gpu, oracle, cfg):
    cl, jobs = setup(cfg)
    jobs.alpha_rack, jobs.beta_rack = synth.draw_rack_pair(jobs, cfg.seed + 50)
    two, rack = _tables(gpu, cfg, cl, jobs, jobs.alpha_rack, jobs.beta_rack)
    ref = oracle.build_speedup_table_rack(jobs, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s)
    _check_rack_table(oracle, jobs, cfg.grid_s, rack, ref)
    assert not rack[0][:, :, :2].any() and rack[0][:, :, 2:].any()
    valid = rack[0] > 0
    assert np.all(rack[0][valid] <= two[0][valid]) and np.any(rack[0][valid] < two[0][valid])   # crossing racks is slower here
    # rack pair = node pair: the rack class is the node class, bit for bit
    _, same = _tables(gpu, cfg, cl, jobs, jobs.alpha_node, jobs.beta_node)
    for a, b in zip(same, two):
        assert np.array_equal(a[:, :, 2:], b[:, :, 2:])


def test_rack_table_large_config_sampled_jobs(gpu, oracle):
    cfg = synth.LARGE
    cl, jobs = setup(cfg)
    jobs.alpha_rack, jobs.beta_rack = synth.draw_rack_pair(jobs, 77)
    _, rack = _tables(gpu, cfg, cl, jobs, jobs.alpha_rack, jobs.beta_rack)
    idx = np.unique(np.concatenate([np.arange(0, 1024, 16), [1, 511, 1023]]))      # 66 jobs
    sub = jobs.take(idx)
    ref = oracle.build_speedup_table_rack(sub, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s)
    _check_rack_table(oracle, sub, cfg.grid_s, tuple(a[idx] for a in rack), ref)


def _fitness_case(seed, P, J, nodes, gpn, per_rack, density=0.2):
    rng = np.random.default_rng(seed)
    cl = synth.uniform_cluster(nodes, gpn)
    table = rng.uniform(0.05, 4.0, (J, cl.k_max + 1, cl.n_max + 1)).astype(np.float32)
    table_rack = (table * rng.uniform(0.3, 0.9, table.shape)).astype(np.float32)
    pop = synth.random_raw_population(P, J, cl, seed + 1, density=density, v_hi=gpn)
    cur = synth.random_raw_population(1, J, cl, seed + 2, density=density, v_hi=gpn)[0]
    pop[0] = cur
    rf = rng.uniform(0.0, 1.0, J).astype(np.float32)
    active = (rng.uniform(size=J) < 0.9).astype(np.uint8)
    return cl, table, table_rack, synth.rack_of_nodes(nodes, per_rack), pop, cur, rf, active


@pytest.mark.parametrize("p", [-1.0, 0.5, 1.0, 0.0, -2.5])
@pytest.mark.parametrize("shape", [(5, 9, 77, 16, 4, 4), (6, 3, 700, 64, 8, 16), (7, 4, 300, 13, 2, 5)])
def test_fitness_with_racks_matches_oracle(gpu, oracle, shape, p):
    torch, api = gpu
    seed, P, J, nodes, gpn, per_rack = shape
    cl, table, table_rack, rack, pop, cur, rf, active = _fitness_case(seed, P, J, nodes, gpn, per_rack)
    s = api.Scheduler(node_capacity=cl.node_capacity, num_jobs=J, grid_m=1, grid_s=1, population=P, speedup_floor=1e-3,
                      stream=torch.cuda.current_stream().cuda_stream)
    s.set_racks(rack)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    d_pop, d_t, d_tr, d_cur, d_rf, d_act = (dev(a) for a in (pop, table, table_rack, cur, rf, active))
    out = torch.full((P,), -1.0, dtype=torch.float32, device="cuda")
    s.eval_fitness_racks(d_pop, d_t, d_tr, out, p=p, cur=d_cur, realloc_factor=d_rf, active=d_act)
    s.sync_status()
    ref = oracle.eval_fitness_racks(pop, table.astype(np.float64), table_rack.astype(np.float64), rack, cl.k_max, cl.n_max,
                                    p, 1e-3, cur=cur, realloc=rf.astype(np.float64), active=active)
    assert_close(out.cpu().numpy(), ref, what="fitness with racks p=%g" % p)
    # racks that do not matter (same table twice): the two-class fitness, same bits
    same = torch.empty_like(out)
    s.eval_fitness_racks(d_pop, d_t, d_t, same, p=p, cur=d_cur, realloc_factor=d_rf, active=d_act)
    plain = torch.empty_like(out)
    s.eval_fitness(d_pop, d_t, plain, p=p, cur=d_cur, realloc_factor=d_rf, active=d_act)
    s.sync_status()
    assert np.array_equal(same.cpu().numpy().view(np.uint32), plain.cpu().numpy().view(np.uint32))
    assert not np.array_equal(out.cpu().numpy(), plain.cpu().numpy())       # and here the racks do matter
    s.close()


def test_fitness_with_racks_every_matrix_of_a_3x2_cluster(gpu, oracle):
    torch, api = gpu
    J, nodes, gpn = 3, 3, 2
    mats = np.ascontiguousarray(np.array(list(itertools.product(range(gpn + 1), repeat=J * nodes)), np.int16)
                                .reshape(-1, J, nodes))
    rng = np.random.default_rng(3)
    k_max, n_max = 6, 3
    table = rng.uniform(0.2, 2.5, (J, k_max + 1, n_max + 1)).astype(np.float32)
    table_rack = (table * 0.5).astype(np.float32)
    rack = np.array([0, 0, 1], np.int16)
    cur = mats[5000].copy()
    rf = np.array([0.9, 0.0, 0.7], np.float32)
    s = api.Scheduler(node_capacity=np.full(nodes, gpn, np.int16), num_jobs=J, grid_m=1, grid_s=1, population=1,
                      speedup_floor=1e-3, k_max=k_max, n_max=n_max, stream=torch.cuda.current_stream().cuda_stream)
    s.set_racks(rack)
    d = lambda a: torch.from_numpy(a).cuda()
    d_pop, d_t, d_tr, d_cur, d_rf = d(mats), d(table), d(table_rack), d(cur), d(rf)
    for p in (-1.0, 0.5, 1.0):
        out = torch.empty(mats.shape[0], dtype=torch.float32, device="cuda")
        s.eval_fitness_racks(d_pop, d_t, d_tr, out, p=p, cur=d_cur, realloc_factor=d_rf)
        s.sync_status()
        ref = oracle.eval_fitness_racks(mats, table.astype(np.float64), table_rack.astype(np.float64), rack, k_max, n_max,
                                        p, 1e-3, cur=cur, realloc=rf.astype(np.float64))
        assert_close(out.cpu().numpy(), ref, what="3x2 with racks p=%g" % p)
    s.close()


@pytest.mark.parametrize("cfg,per_rack", [(synth.TINY, 2), (synth.TESTBED, 4),
                                          (synth.Config("racks-300-jobs", 32, 8, 300, 31, 16, 8, 24, 6, num_elite=2,
                                                        mutate_prob=0.2, init_prob=0.3, with_history=True,
                                                        random_cur=True), 8)], ids=lambda c: getattr(c, "name", str(c)))
def test_round_with_racks(gpu, oracle, cfg, per_rack):
    """A round with racks equals the entry points called one by one (tables, initial population,
    generations, eval_fitness_racks), and its final fitness is the oracle's on the round's own tables."""
    torch, api = gpu
    cl, jobs = setup(cfg)
    cur = cfg.cur(jobs)
    jobs.alpha_rack, jobs.beta_rack = synth.draw_rack_pair(jobs, cfg.seed + 9)
    rack = synth.rack_of_nodes(cfg.num_nodes, per_rack)
    gens = min(cfg.generations, 12)
    dev = "cuda:0"
    d_ar, d_br = torch.from_numpy(jobs.alpha_rack).cuda(), torch.from_numpy(jobs.beta_rack).cuda()
    P, J, NN = cfg.population, cfg.num_jobs, cfg.num_nodes
    res = {}
    for with_racks in (True, False):
        s = api.scheduler_for(cfg, stream=torch.cuda.current_stream().cuda_stream)
        if with_racks:
            s.set_racks(rack, d_ar, d_br)
        dj = api.DeviceJobs(jobs, dev, torch)
        d_cur = torch.from_numpy(cur).cuda()
        best = torch.empty((J, NN), dtype=torch.int16, device=dev)
        bf = torch.zeros(1, dtype=torch.float32, device=dev)
        s.schedule_round(dj, d_cur, best, bf, round=4, generations=gens)
        s.sync_status()
        pop = torch.empty((P, J, NN), dtype=torch.int16, device=dev)
        fit = torch.empty(P, dtype=torch.float32, device=dev)
        s.get_population(pop, fit)
        res[with_racks] = (pop.cpu().numpy(), fit.cpu().numpy(), best.cpu().numpy(), float(bf.item()))
        if not with_racks:
            s.close()
            continue
        # stepwise
        sp = torch.empty(s.table_shape, dtype=torch.float32, device=dev)
        spr = torch.empty_like(sp)
        s.build_speedup_table(dj, None, sp, None)
        s.build_speedup_table_rack(dj, d_ar, d_br, None, spr, None)
        rf = torch.empty(J, dtype=torch.float32, device=dev)
        s.compute_realloc_factor(dj, rf)
        a = torch.empty((P, J, NN), dtype=torch.int16, device=dev)
        b = torch.empty_like(a)
        f = torch.empty(P, dtype=torch.float32, device=dev)
        kw = dict(p=cfg.p, cur=d_cur, realloc_factor=rf, active=dj.tensors["active"])
        s.init_population(dj, d_cur, a, round=4)
        s.eval_fitness_racks(a, sp, spr, f, **kw)
        for g in range(gens):
            s.ga_generation(dj, a, f, b, round=4, generation=g)
            a, b = b, a
            s.eval_fitness_racks(a, sp, spr, f, **kw)
        s.sync_status()
        assert np.array_equal(a.cpu().numpy(), res[True][0])
        assert np.array_equal(f.cpu().numpy().view(np.uint32), res[True][1].view(np.uint32))
        i = int(np.argmax(res[True][1]))
        assert np.array_equal(res[True][2], res[True][0][i]) and res[True][3] == res[True][1][i]
        ref = oracle.eval_fitness_racks(res[True][0], sp.cpu().numpy().astype(np.float64),
                                        spr.cpu().numpy().astype(np.float64), rack, cl.k_max, cl.n_max, cfg.p,
                                        cfg.speedup_floor, cur=cur, realloc=rf.cpu().numpy().astype(np.float64),
                                        active=jobs.active)
        assert_close(res[True][1], ref, what="round fitness with racks")
        for c in range(0, P, 5):
            assert feasible(res[True][0][c], cl.node_capacity, jobs.k_cap, cl.n_max)
        s.close()
    assert not np.array_equal(res[True][1], res[False][1])          # the racks changed the search
