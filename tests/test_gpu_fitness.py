"""Parity of eval_fitness (CUDA) against the oracle: element by element on small and
ragged shapes, on the five configurations' shapes, and at the stress workload's full row
and table sizes."""
import numpy as np
import pytest

from helpers import REL_TOL, assert_close
from paper_2008_12260_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2008_12260_b200 import api
    assert torch.cuda.is_available()
    return torch, api


def _run(gpu, pop, table, cap, p, floor=1e-3, cur=None, rf=None, active=None, k_max=None, n_max=None,
         host=False):
    torch, api = gpu
    dev = torch.device("cuda:0")
    P, J, N = pop.shape
    s = api.Scheduler(node_capacity=cap, num_jobs=J, grid_m=1, grid_s=1, population=max(P, 1),
                      speedup_floor=floor, k_max=k_max, n_max=n_max,
                      stream=torch.cuda.current_stream().cuda_stream)
    assert tuple(table.shape) == s.table_shape
    if host:
        out = np.full(P, -7.0, np.float32)
        s.eval_fitness_host(np.ascontiguousarray(pop), np.ascontiguousarray(table), out, p=p, cur=cur,
                            realloc_factor=rf, active=active)
        s.close()
        return out
    t = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    d_pop = pop if isinstance(pop, torch.Tensor) else t(pop)
    out = torch.full((P,), -7.0, dtype=torch.float32, device=dev)
    s.eval_fitness(d_pop, t(table), out, p=p, cur=t(cur), realloc_factor=t(rf), active=t(active))
    s.sync_status()
    first = out.cpu().numpy()
    out.fill_(-9.0)
    s.eval_fitness(d_pop, t(table), out, p=p, cur=t(cur), realloc_factor=t(rf), active=t(active))
    s.sync_status()
    assert np.array_equal(first.view(np.uint32), out.cpu().numpy().view(np.uint32))   # reproducible bits
    s.close()
    return first


def _case(seed, P, J, nodes, gpn=4, density=0.2):
    rng = np.random.default_rng(seed)
    cl = synth.uniform_cluster(nodes, gpn)
    k_max, n_max = cl.k_max, cl.n_max
    table = rng.uniform(0.05, 4.0, (J, k_max + 1, n_max + 1)).astype(np.float32)
    table[:, 0, :] = 0; table[:, :, 0] = 0
    pop = synth.random_raw_population(P, J, cl, seed + 1, density=density, v_hi=gpn)
    cur = synth.random_raw_population(1, J, cl, seed + 2, density=density, v_hi=gpn)[0]
    cur[::3] = 0                                   # pending jobs
    pop[0] = cur                                   # an unchanged candidate
    pop[1::4, ::2] = cur[::2]                      # partly unchanged candidates
    rf = rng.uniform(0.0, 1.0, J).astype(np.float32)
    active = (rng.uniform(size=J) < 0.85).astype(np.uint8)
    return cl, table, pop, cur, rf, active


@pytest.mark.parametrize("nodes", [1, 3, 4, 6, 12, 16, 40, 64, 100, 256, 1000])
@pytest.mark.parametrize("p", [-1.0, 0.5, 1.0])
def test_row_widths(gpu, oracle, nodes, p):
    cl, table, pop, cur, rf, active = _case(nodes, P=9, J=301, nodes=nodes)
    got = _run(gpu, pop, table, cl.node_capacity, p, cur=cur, rf=rf, active=active)
    ref = oracle.eval_fitness(pop, table.astype(np.float64), cl.k_max, cl.n_max, p, 1e-3, cur=cur,
                              realloc=rf.astype(np.float64), active=active)
    assert_close(got, ref, what="fitness nodes=%d p=%g" % (nodes, p))


@pytest.mark.parametrize("p", [0.0, -3.0, 2.0, -10.0])
def test_other_exponents(gpu, oracle, p):
    cl, table, pop, cur, rf, active = _case(7, P=17, J=130, nodes=24)
    got = _run(gpu, pop, table, cl.node_capacity, p, cur=cur, rf=rf)
    ref = oracle.eval_fitness(pop, table.astype(np.float64), cl.k_max, cl.n_max, p, 1e-3, cur=cur,
                              realloc=rf.astype(np.float64))
    assert_close(got, ref, what="fitness p=%g" % p)


def test_no_penalty_variants_and_floor(gpu, oracle):
    cl, table, pop, cur, rf, active = _case(11, P=8, J=64, nodes=16)
    base = oracle.eval_fitness(pop, table.astype(np.float64), cl.k_max, cl.n_max, -1.0, 0.0)
    assert_close(_run(gpu, pop, table, cl.node_capacity, -1.0, floor=0.0), base)
    assert_close(_run(gpu, pop, table, cl.node_capacity, -1.0, floor=0.0, cur=cur), base)     # no factors
    assert_close(_run(gpu, pop, table, cl.node_capacity, -1.0, floor=0.0, rf=rf), base)       # no cur
    ones = np.ones_like(rf)
    assert_close(_run(gpu, pop, table, cl.node_capacity, -1.0, floor=0.0, cur=cur, rf=ones), base)
    ref = oracle.eval_fitness(pop, table.astype(np.float64), cl.k_max, cl.n_max, -1.0, 0.25, cur=cur,
                              realloc=rf.astype(np.float64))
    assert_close(_run(gpu, pop, table, cl.node_capacity, -1.0, floor=0.25, cur=cur, rf=rf), ref)


def test_degenerate_inputs(gpu, oracle):
    cl, table, pop, cur, rf, active = _case(13, P=5, J=40, nodes=8)
    none = np.zeros(40, np.uint8)
    assert not _run(gpu, pop, table, cl.node_capacity, -1.0, active=none).any()          # no active job
    empty = np.zeros_like(pop)
    ref = oracle.eval_fitness(empty, table.astype(np.float64), cl.k_max, cl.n_max, 1.0, 1e-3)
    assert_close(_run(gpu, empty, table, cl.node_capacity, 1.0), ref)                     # all floor
    big = np.full_like(pop, 3000)                                                         # K, N clamp to the table edge
    ref = oracle.eval_fitness(big, table.astype(np.float64), cl.k_max, cl.n_max, 1.0, 1e-3)
    assert_close(_run(gpu, big, table, cl.node_capacity, 1.0), ref)
    top = np.full_like(pop, 32767)
    ref = oracle.eval_fitness(top, table.astype(np.float64), cl.k_max, cl.n_max, 1.0, 1e-3)
    assert_close(_run(gpu, top, table, cl.node_capacity, 1.0), ref)
    zero_count = _run(gpu, pop[:0], table, cl.node_capacity, 1.0)
    assert zero_count.shape == (0,)
    one_job = _case(14, P=3, J=1, nodes=8)
    ref = oracle.eval_fitness(one_job[2], one_job[1].astype(np.float64), 32, 8, -1.0, 1e-3)
    assert_close(_run(gpu, one_job[2], one_job[1], one_job[0].node_capacity, -1.0), ref)


def test_host_buffer_entry_point(gpu, oracle):
    cl, table, pop, cur, rf, active = _case(15, P=6, J=77, nodes=16)
    got = _run(gpu, pop, table, cl.node_capacity, -1.0, cur=cur, rf=rf, active=active, host=True)
    dev = _run(gpu, pop, table, cl.node_capacity, -1.0, cur=cur, rf=rf, active=active)
    assert np.array_equal(got.view(np.uint32), dev.view(np.uint32))


def test_large_config_shape(gpu, oracle):
    """256 nodes x 8 GPUs, 1024 jobs: the launch shape of the large configuration, with a
    random current allocation and the penalty on; 24 candidates against the oracle."""
    cl, table, pop, cur, rf, active = _case(17, P=24, J=1024, nodes=256, gpn=8, density=0.01)
    got = _run(gpu, pop, table, cl.node_capacity, -1.0, cur=cur, rf=rf)
    ref = oracle.eval_fitness(pop, table.astype(np.float64), 64, 64, -1.0, 1e-3, cur=cur,
                              realloc=rf.astype(np.float64))
    assert_close(got, ref, what="large")


@pytest.mark.parametrize("p", [-1.0, 0.5, 1.0])
def test_stress_workload_full_row_size(gpu, oracle, p):
    """2048 nodes, 8192 jobs, fp32 [8192][65][65] tables (138 MB): one 64-candidate chunk of
    the stress population in the bench's launch configuration, every candidate against the oracle."""
    torch, api = gpu
    st = synth.STRESS
    table = synth.stress_speedup_table(st["num_jobs"], 64, 64, 8, st["seed"])
    pop = synth.stress_population(64, st["num_jobs"], st["num_nodes"], 8, st["seed"], device="cuda:0")
    cap = synth.uniform_cluster(st["num_nodes"], 8).node_capacity
    got = _run(gpu, pop, table, cap, p)
    ref = oracle.eval_fitness(pop.cpu().numpy(), table.astype(np.float64), 64, 64, p, 1e-3)   # all 64 candidates
    assert_close(got, ref, what="stress p=%g" % p)
    assert np.all(got > 0) and np.all(np.isfinite(got))
    rows = pop[0].to(torch.int64)
    assert int((rows > 0).sum(-1).max()) <= 64 and float((rows.sum(-1) == 0).float().mean()) > 0.4
