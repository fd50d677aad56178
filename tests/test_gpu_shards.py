"""A generation made in slices (ga_generation_shard) is the generation made at once, bit for
bit: the population search of Sec. 4.3 shards by candidate.  The slices are made one after the
other on the one GPU here; tests/test_dist_cpu.py covers the gathering between real ranks."""
import numpy as np
import pytest

from helpers import setup
from paper_2008_12260_b200 import dist as pdist
from paper_2008_12260_b200 import synth

pytestmark = pytest.mark.gpu

CASES = [
    synth.TINY,
    synth.TESTBED,
    synth.Config("shard-odd-nodes", 7, 3, 23, 41, 16, 8, 37, 5, num_elite=3, mutate_prob=0.3, init_prob=0.4,
                 with_history=True, random_cur=True),                                  # general fallback kernels
    synth.Config("shard-300-jobs", 32, 8, 300, 42, 16, 8, 26, 4, num_elite=2, mutate_prob=0.2, init_prob=0.3,
                 with_history=True, random_cur=True),                                  # several row batches
]


@pytest.mark.parametrize("cfg", CASES, ids=lambda c: c.name)
@pytest.mark.parametrize("world", [2, 3])
def test_slices_of_a_generation_equal_the_generation(cfg, world):
    import torch
    from paper_2008_12260_b200 import api

    cl, jobs = setup(cfg)
    dev = "cuda:0"
    s = api.scheduler_for(cfg, stream=torch.cuda.current_stream().cuda_stream)
    dj = api.DeviceJobs(jobs, dev, torch)
    P, J, NN = cfg.population, cfg.num_jobs, cfg.num_nodes
    d_cur = torch.from_numpy(cfg.cur(jobs)).cuda()
    sp = torch.empty(s.table_shape, dtype=torch.float32, device=dev)
    s.build_speedup_table(dj, None, sp, None)
    a = torch.empty((P, J, NN), dtype=torch.int16, device=dev)
    f = torch.empty(P, dtype=torch.float32, device=dev)
    s.init_population(dj, d_cur, a, round=3)
    s.eval_fitness(a, sp, f, p=cfg.p, active=dj.tensors["active"])

    def make_children(pop, fit, first, count, g):
        out = torch.full((count, J, NN), -9, dtype=torch.int16, device=dev)
        s.ga_generation_shard(dj, pop, fit, out, first_child=first, round=3, generation=g)
        return out

    def evaluate(children):
        out = torch.empty(children.shape[0], dtype=torch.float32, device=dev)
        s.eval_fitness(children, sp, out, p=cfg.p, active=dj.tensors["active"])
        return out

    pop, fit = a, f
    for g in range(3):
        # the generation at once
        whole = torch.empty_like(pop)
        s.ga_generation(dj, pop, fit, whole, round=3, generation=g)
        wfit = evaluate(whole)
        # the same generation in `world` slices, as `world` ranks would make them
        parts, pfit = [], []
        for r in range(world):
            b, e = pdist.shard_range(P, r, world)
            ch = make_children(pop, fit, b, e - b, g)
            parts.append(ch)
            pfit.append(evaluate(ch))
        s.sync_status()
        got, gfit = torch.cat(parts), torch.cat(pfit)
        assert np.array_equal(got.cpu().numpy(), whole.cpu().numpy())
        assert np.array_equal(gfit.cpu().numpy().view(np.uint32), wfit.cpu().numpy().view(np.uint32))
        pop, fit = whole, wfit
    # the single-process path of the sharded driver is the plain loop
    p1, f1 = pdist.evolve_sharded(make_children, evaluate, a, f, 3, 0, 1)
    s.sync_status()
    assert np.array_equal(p1.cpu().numpy(), pop.cpu().numpy())
    # slices outside the population are refused
    with pytest.raises(api.SchedError):
        s.ga_generation_shard(dj, a, f, torch.empty((2, J, NN), dtype=torch.int16, device=dev), first_child=P - 1,
                              round=3, generation=0)
    s.close()
