"""Parity of build_speedup_table (CUDA, fp32) against the fp64 oracle."""
import numpy as np
import pytest

from helpers import assert_close, check_table, setup, with_fair_share
from paper_2008_12260_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2008_12260_b200 import api
    assert torch.cuda.is_available()
    return torch, api


def _gpu_table(gpu, cl, jobs, grid_s, k_max=None, n_max=None, want_goodput=True, want_argmax=True):
    torch, api = gpu
    dev = torch.device("cuda:0")
    s = api.Scheduler(node_capacity=cl.node_capacity, num_jobs=jobs.num_jobs, grid_m=jobs.m_grid.shape[1],
                      grid_s=grid_s, population=1, k_max=k_max, n_max=n_max,
                      stream=torch.cuda.current_stream().cuda_stream)
    dj = api.DeviceJobs(jobs, dev, torch)
    gp = torch.full(s.table_shape, -1.0, dtype=torch.float32, device=dev) if want_goodput else None
    sp = torch.full(s.table_shape, -1.0, dtype=torch.float32, device=dev)
    am = torch.full(s.table_shape, 7, dtype=torch.uint16, device=dev) if want_argmax else None
    s.build_speedup_table(dj, gp, sp, am)
    s.sync_status()
    out = (None if gp is None else gp.cpu().numpy(), sp.cpu().numpy(),
           None if am is None else am.cpu().numpy())
    s.close()
    return out


@pytest.mark.parametrize("cfg", [synth.TINY, synth.TESTBED], ids=lambda c: c.name)
def test_table_matches_oracle(gpu, oracle, cfg):
    cl, jobs = setup(cfg)
    gp, sp, am = _gpu_table(gpu, cl, jobs, cfg.grid_s)
    gp_r, sp_r, am_r = oracle.build_speedup_table(jobs, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s)
    ndiff = check_table(oracle, jobs, cfg.grid_s, gp, sp, am, gp_r, sp_r, am_r)
    assert ndiff < 0.05 * am.size
    fk, fn = int(jobs.fair_k[0]), int(jobs.fair_n[0])
    assert np.all(sp[:, fk, fn] == 1.0)       # Eq. 15: exactly one at the fair share


def test_large_config_sampled_jobs(gpu, oracle):
    """Full-size launch (1024 jobs, 128 x 32 grid); the oracle checks a sample of jobs."""
    cfg = synth.LARGE
    cl, jobs = setup(cfg)
    gp, sp, am = _gpu_table(gpu, cl, jobs, cfg.grid_s)
    idx = np.unique(np.concatenate([np.arange(0, 1024, 16), [1, 17, 255, 256, 511, 777, 1000, 1023]]))   # 71 jobs
    sub = jobs.take(idx)
    gp_r, sp_r, am_r = oracle.build_speedup_table(sub, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s)
    check_table(oracle, sub, cfg.grid_s, gp[idx], sp[idx], am[idx], gp_r, sp_r, am_r)
    # properties that hold for every job at any size
    assert np.all(sp[:, int(jobs.fair_k[0]), int(jobs.fair_n[0])] == 1.0)
    assert np.all(gp[:, 0, :] == 0) and np.all(gp[:, :, 0] == 0)
    K = np.arange(65)[:, None]; N = np.arange(65)[None, :]
    valid = (N >= 1) & (K >= N) & (K <= 8 * N)
    assert np.all((gp > 0) == valid[None])
    assert np.all(gp[:, 2:9, 1] >= gp[:, 2:9, 2])           # local sync never slower than node sync here
    for K_ in (16, 33, 64):                                 # Eq. 9: N >= 2 columns agree
        cols = [n for n in range(2, 65) if valid[K_, n]]
        assert np.all(gp[:, K_, cols] == gp[:, K_, cols[:1]])


@pytest.mark.parametrize("grid_m,grid_s", [(7, 1), (40, 3), (200, 5), (33, 16)])
def test_ragged_grids(gpu, oracle, grid_m, grid_s):
    cl = synth.Cluster(np.array([8, 4, 4, 2, 1, 0], np.int16))      # heterogeneous nodes
    jobs = synth.draw_jobs(11, 21, grid_m, 16, cl.k_max)
    jobs = with_fair_share(jobs, cl)
    gp, sp, am = _gpu_table(gpu, cl, jobs, grid_s)
    gp_r, sp_r, am_r = oracle.build_speedup_table(jobs, cl.node_capacity, cl.k_max, cl.n_max, grid_s)
    check_table(oracle, jobs, grid_s, gp, sp, am, gp_r, sp_r, am_r)


def test_degenerate_jobs(gpu, oracle):
    cl = synth.uniform_cluster(4, 4)
    jobs = synth.draw_jobs(6, 3, 32, 8, cl.k_max)
    # prior-driven exploration (Sec. 4.1): unexplored sync parameters are zero
    jobs.alpha_local[0] = jobs.beta_local[0] = 0.0
    jobs.beta_local[1] = jobs.beta_node[1] = 0.0
    jobs.alpha_local[2] = jobs.beta_local[2] = jobs.alpha_node[2] = jobs.beta_node[2] = 0.0
    jobs.gamma[3] = 1.0
    jobs.gamma[4] = 10.0
    jobs.m_max_total[5] = jobs.m0[5]            # only M = M0 is allowed: many (K, N) infeasible
    jobs = with_fair_share(jobs, cl)
    gp, sp, am = _gpu_table(gpu, cl, jobs, 8)
    gp_r, sp_r, am_r = oracle.build_speedup_table(jobs, cl.node_capacity, cl.k_max, cl.n_max, 8)
    check_table(oracle, jobs, 8, gp, sp, am, gp_r, sp_r, am_r)
    assert (gp_r[5] == 0).sum() > (gp_r[0] == 0).sum()


def test_invalid_fair_share_and_optional_outputs(gpu, oracle):
    cl = synth.uniform_cluster(4, 4)
    jobs = synth.draw_jobs(5, 4, 32, 8, cl.k_max)
    jobs = with_fair_share(jobs, cl, fair=(3, 1))
    jobs.fair_k[1], jobs.fair_n[1] = 9, 1         # does not fit one node: no denominator
    jobs.fair_k[2], jobs.fair_n[2] = 500, 700     # outside the table
    jobs.fair_k[3], jobs.fair_n[3] = -1, -1
    gp, sp, am = _gpu_table(gpu, cl, jobs, 8, want_goodput=False, want_argmax=False)
    assert gp is None and am is None
    gp_r, sp_r, am_r = oracle.build_speedup_table(jobs, cl.node_capacity, cl.k_max, cl.n_max, 8)
    assert_close(sp, sp_r, what="speedup")
    assert not sp[1].any() and not sp[2].any() and not sp[3].any() and sp[0].any()


def test_single_job_and_custom_dims(gpu, oracle):
    cl = synth.uniform_cluster(3, 8)
    jobs = with_fair_share(synth.draw_jobs(1, 9, 32, 8, 24), cl)
    gp, sp, am = _gpu_table(gpu, cl, jobs, 8, k_max=20, n_max=2)
    gp_r, sp_r, am_r = oracle.build_speedup_table(jobs, cl.node_capacity, 20, 2, 8)
    assert gp.shape == (1, 21, 3)
    check_table(oracle, jobs, 8, gp, sp, am, gp_r, sp_r, am_r)
