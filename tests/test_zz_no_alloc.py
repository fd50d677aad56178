"""eval_fitness_noalloc: the fitness entry point for callers that may not allocate device
memory (a process whose allocator already owns the whole GPU, or a control loop that cannot
take cudaMalloc's device-wide synchronisation).  It keeps its scratch in a fixed device array
inside the library, so it must give the same answers as eval_fitness, call after call, with
whatever the previous call left behind in that array.  Collected last on purpose."""
import numpy as np
import pytest

from paper_2008_12260_b200 import synth

pytestmark = pytest.mark.gpu

REL_TOL = 1e-5   # the tolerance of every fitness parity test


def _inputs(seed, P, J, nodes, torch, k_max=None, n_max=None):
    rng = np.random.default_rng(seed)
    cl = synth.uniform_cluster(nodes, 4)
    k_max = cl.k_max if k_max is None else k_max
    n_max = cl.n_max if n_max is None else n_max
    table = rng.uniform(0.05, 4.0, (J, k_max + 1, n_max + 1)).astype(np.float32)
    pop = synth.random_raw_population(P, J, cl, seed + 1, density=0.2 if nodes <= 64 else 0.01, v_hi=4)
    cur = synth.random_raw_population(1, J, cl, seed + 2, density=0.2 if nodes <= 64 else 0.01, v_hi=4)[0]
    pop[0] = cur
    rf = rng.uniform(0.0, 1.0, J).astype(np.float32)
    active = (rng.uniform(size=J) < 0.9).astype(np.uint8)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    host = (table, pop, cur, rf, active)
    return cl, k_max, n_max, host, tuple(dev(a) for a in host)


# (seed, candidates, jobs, nodes, exponent, with current allocation, table dims or None)
CASES = (
    (3, 40, 700, 64, -1.0, True, None),
    (4, 9, 301, 12, 0.5, False, None),       # a different problem: sees the first call's leftovers
    (5, 7, 513, 24, 0.0, True, None),        # geometric mean
    (6, 5, 130, 16, -2.5, False, None),      # generic exponent
    (7, 2048, 8, 8, 1.0, True, None),        # the largest candidate count
    (8, 1, 16384, 260, -1.0, False, (8, 4)), # the largest job count, rows split into many small chunks
)


def test_calls_in_a_row_match_eval_fitness_and_the_oracle(oracle):
    import torch
    from paper_2008_12260_b200 import api

    assert torch.cuda.is_available()
    stream = torch.cuda.current_stream().cuda_stream
    for seed, P, J, nodes, p, with_cur, dims in CASES:
        cl, k_max, n_max, host, devs = _inputs(seed, P, J, nodes, torch, *(dims or (None, None)))
        h_table, h_pop, h_cur, h_rf, h_active = host
        table, pop, cur, rf, active = devs
        s = api.Scheduler(node_capacity=cl.node_capacity, num_jobs=J, grid_m=1, grid_s=1, population=P,
                          speedup_floor=1e-3, k_max=k_max, n_max=n_max, stream=stream)
        ref = torch.empty(P, dtype=torch.float32, device="cuda")
        s.eval_fitness(pop, table, ref, p=p, cur=cur if with_cur else None,
                       realloc_factor=rf if with_cur else None, active=active)
        s.sync_status()
        kw = dict(k_max=k_max, n_max=n_max, p=p, speedup_floor=1e-3, cur=cur if with_cur else None,
                  realloc_factor=rf if with_cur else None, active=active, stream=stream)
        got = torch.full((P,), -5.0, dtype=torch.float32, device="cuda")
        api.eval_fitness_noalloc(pop, table, got, **kw)
        torch.cuda.synchronize()
        # what the entry point is for: a further call leaves the device's free memory as it found it
        free_before = torch.cuda.mem_get_info()[0]
        got2 = torch.full((P,), -7.0, dtype=torch.float32, device="cuda")
        free_mid = torch.cuda.mem_get_info()[0]       # torch's own output buffer, if it had to grow its cache
        api.eval_fitness_noalloc(pop, table, got2, **kw)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_mid <= free_before
        g, g2, r = got.cpu().numpy(), got2.cpu().numpy(), ref.cpu().numpy()
        # the existing entry point: within the tolerance of the fitness tests, and in fact the same
        # bits (same kernels, same chunks, same order of the sums)
        np.testing.assert_allclose(g, r, rtol=REL_TOL, atol=0)
        assert np.array_equal(g.view(np.uint32), r.view(np.uint32))
        assert np.array_equal(g2.view(np.uint32), r.view(np.uint32))
        # and the oracle (Eq. 14 in fp64) on the same inputs
        want = oracle.eval_fitness(h_pop, h_table.astype(np.float64), k_max, n_max, p, 1e-3,
                                   cur=h_cur if with_cur else None,
                                   realloc=h_rf.astype(np.float64) if with_cur else None, active=h_active)
        np.testing.assert_allclose(g, want, rtol=REL_TOL, atol=0)
        assert np.all(np.isfinite(g)) and np.all(g > 0)
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
