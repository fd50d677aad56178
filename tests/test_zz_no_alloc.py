"""eval_fitness_noalloc: the fitness entry point for callers that may not allocate device
memory (a process whose allocator already owns the whole GPU, or a control loop that cannot
take cudaMalloc's device-wide synchronisation).  It keeps its scratch in a fixed device array
inside the library, so it must give the same answers as eval_fitness, call after call, with
whatever the previous call left behind in that array.  Collected last on purpose."""
import numpy as np
import pytest

from paper_2008_12260_b200 import synth

pytestmark = pytest.mark.gpu


def _inputs(seed, P, J, nodes, torch):
    rng = np.random.default_rng(seed)
    cl = synth.uniform_cluster(nodes, 4)
    table = rng.uniform(0.05, 4.0, (J, cl.k_max + 1, cl.n_max + 1)).astype(np.float32)
    pop = synth.random_raw_population(P, J, cl, seed + 1, density=0.2, v_hi=4)
    cur = synth.random_raw_population(1, J, cl, seed + 2, density=0.2, v_hi=4)[0]
    pop[0] = cur
    rf = rng.uniform(0.0, 1.0, J).astype(np.float32)
    active = (rng.uniform(size=J) < 0.9).astype(np.uint8)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return cl, dev(table), dev(pop), dev(cur), dev(rf), dev(active)


def test_two_calls_in_a_row_match_eval_fitness():
    import torch
    from paper_2008_12260_b200 import api

    assert torch.cuda.is_available()
    stream = torch.cuda.current_stream().cuda_stream
    # two different problems back to back: the second call sees the first one's leftovers
    for seed, P, J, nodes, p, with_cur in ((3, 40, 700, 64, -1.0, True), (4, 9, 301, 12, 0.5, False)):
        cl, table, pop, cur, rf, active = _inputs(seed, P, J, nodes, torch)
        s = api.Scheduler(node_capacity=cl.node_capacity, num_jobs=J, grid_m=1, grid_s=1, population=P,
                          speedup_floor=1e-3, stream=stream)
        ref = torch.empty(P, dtype=torch.float32, device="cuda")
        s.eval_fitness(pop, table, ref, p=p, cur=cur if with_cur else None,
                       realloc_factor=rf if with_cur else None, active=active)
        s.sync_status()
        got = torch.full((P,), -5.0, dtype=torch.float32, device="cuda")
        api.eval_fitness_noalloc(pop, table, got, k_max=cl.k_max, n_max=cl.n_max, p=p, speedup_floor=1e-3,
                                 cur=cur if with_cur else None, realloc_factor=rf if with_cur else None,
                                 active=active, stream=stream)
        torch.cuda.synchronize()
        np.testing.assert_allclose(got.cpu().numpy(), ref.cpu().numpy(), rtol=1e-5, atol=0)
        assert np.all(np.isfinite(got.cpu().numpy())) and np.all(got.cpu().numpy() > 0)
        s.close()


def test_sizes_beyond_the_fixed_scratch_are_rejected():
    import torch
    from paper_2008_12260_b200 import api

    t = torch.zeros(16, dtype=torch.int16, device="cuda")
    f = torch.zeros(16, dtype=torch.float32, device="cuda")
    # the size check comes before any access: the small buffers are never touched
    for count, jobs, nodes in ((2049, 4, 2), (1, 16385, 2), (1, 4, 8193)):
        rc = api._lib.eval_fitness_noalloc(t.data_ptr(), count, jobs, nodes, 4, 2, f.data_ptr(), None, None,
                                           None, 1.0, 0.0, f.data_ptr(), None)
        assert rc == -6
        assert b"eval_fitness" in api._lib.eval_fitness_noalloc_last_error()
    assert api._lib.eval_fitness_noalloc(None, 1, 4, 2, 4, 2, f.data_ptr(), None, None, None, 1.0, 0.0,
                                         f.data_ptr(), None) == -1
    assert api._lib.eval_fitness_noalloc(t.data_ptr(), 0, 4, 2, 4, 2, f.data_ptr(), None, None, None, 1.0, 0.0,
                                         f.data_ptr(), None) == 0
