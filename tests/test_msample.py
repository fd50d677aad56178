"""The total-batch sampling search of Sec. 4.3 and the non-adaptive jobs of Sec. 4.2:
oracle pins (hand-worked cases, relations to the grid search) and CUDA parity."""
import numpy as np
import pytest

from helpers import REL_TOL, assert_close, setup, with_fair_share
from paper_2008_12260_b200 import synth


def _one_job(**kw):
    jobs = synth.draw_jobs(1, 0, 4, 4, 8)
    for f, v in dict(alpha_grad=1.0, beta_grad=0.02, alpha_local=4.0, beta_local=0.0, alpha_node=4.0,
                     beta_node=0.0, gamma=2.0, phi=1200.0, m0=400.0, m_max_total=12800.0).items():
        getattr(jobs, f)[:] = v
    for f, v in kw.items():
        getattr(jobs, f)[:] = v
    jobs.fair_k = np.array([1], np.int32); jobs.fair_n = np.array([1], np.int32)
    return jobs


def test_hand_worked_candidate(oracle):
    # K = 4 on one node, candidate M = 1200, per-GPU limit 100: per_gpu = 300, s = 2, m = 100,
    # M' = 1200.  T_grad = 3, T_sync = 4, gamma = 2 -> 5; T_iter = 2*3 + 5 = 11;
    # efficiency = (1200 + 400)/(1200 + 1200) = 2/3; goodput = 1200/11 * 2/3 = 800/11
    jobs = _one_job()
    cap = np.array([4], np.int16)
    gp, sp, am = oracle.build_speedup_table_msample(jobs, cap, 4, 1, np.array([[1200]], np.int32),
                                                    np.array([100], np.int32))
    assert gp[0, 4, 1] == pytest.approx(800 / 11, rel=1e-6) and am[0, 4, 1] == 0
    # K = 3: per_gpu = 400, s = 3, m = 100, M' = 1200: T_sync = 4 (beta 0), T_iter = 3*3 + 5 = 14
    assert gp[0, 3, 1] == pytest.approx(1200 / 14 * 2 / 3, rel=1e-6)
    # K = 1: per_gpu = 1200, s = 11, m = 100: no sync, T_iter = 12 * 3
    assert gp[0, 1, 1] == pytest.approx(1200 / 36 * 2 / 3, rel=1e-6)
    # rounding up: M = 1000 on K = 3 -> per_gpu = 334, s = 3, m = 84, M' = 1008
    gp2, _, _ = oracle.build_speedup_table_msample(jobs, cap, 4, 1, np.array([[1000]], np.int32),
                                                   np.array([100], np.int32))
    tg = 1 + 0.02 * 84
    t_it = 3 * tg + (tg ** 2 + 16) ** 0.5
    assert gp2[0, 3, 1] == pytest.approx(1008 / t_it * (1600 / (1200 + 1008)), rel=1e-6)
    # a candidate whose run batch exceeds the limit is dropped: M_max = 1000 < 1008
    jobs_lim = _one_job(m_max_total=1000.0)
    gp3, _, am3 = oracle.build_speedup_table_msample(jobs_lim, cap, 4, 1, np.array([[1000]], np.int32),
                                                     np.array([100], np.int32))
    assert gp3[0, 3, 1] == 0 and am3[0, 3, 1] == 0xFFFF


def test_non_adaptive_job(oracle):
    # fixed batch M0 = 400, efficiency 1: K = 4 -> per_gpu 100, s 0, m 100: T_iter = 5; goodput 80
    jobs = _one_job()
    cap = np.array([4], np.int16)
    ms = np.array([[1200, 5000]], np.int32)
    gp, _, am = oracle.build_speedup_table_msample(jobs, cap, 4, 1, ms, np.array([100], np.int32),
                                                   adaptive=np.array([0], np.uint8))
    assert gp[0, 4, 1] == pytest.approx(400 / 5, rel=1e-6) and am[0, 4, 1] == 0
    # the noise scale plays no part
    jobs2 = _one_job(phi=7.0)
    gp2, _, _ = oracle.build_speedup_table_msample(jobs2, cap, 4, 1, ms, np.array([100], np.int32),
                                                   adaptive=np.array([0], np.uint8))
    assert np.array_equal(gp, gp2)


def test_relation_to_grid_search(oracle):
    """A candidate M that the grid search also reaches with the same (m, s) gives the same
    goodput; with the candidates {K m (s+1)} of all grid points the sampling search can only
    differ by choosing fewer accumulation steps, never a different batch."""
    cfg = synth.TINY
    cl, jobs = setup(cfg)
    gg, _, ag = oracle.build_speedup_table(jobs, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s)
    ms = synth.make_m_samples(jobs.m0, jobs.m_max_total, 64)
    gp, sp, am = oracle.build_speedup_table_msample(jobs, cl.node_capacity, cl.k_max, cl.n_max, ms, jobs.m_max_gpu)
    assert np.array_equal(gp > 0, gg > 0)                       # same feasible (K, N) set for these inputs
    ratio = gp[gg > 0] / gg[gg > 0]
    assert ratio.min() > 0.8 and ratio.max() < 1.25             # two searches of the same landscape
    fk, fn = int(jobs.fair_k[0]), int(jobs.fair_n[0])
    assert np.all(sp[:, fk, fn] == 1.0)
    # single-GPU, single candidate equal to a grid point with s = 0: identical value
    j = 0
    m = int(jobs.m_grid[j, -1])
    M = max(m, int(jobs.m0[j]))
    g1, _, _ = oracle.build_speedup_table_msample(jobs, cl.node_capacity, cl.k_max, cl.n_max,
                                                  np.full((cfg.num_jobs, 1), M, np.int32), jobs.m_max_gpu)
    par = [float(getattr(jobs, f)[j]) for f in synth.JOB_F32_FIELDS]
    if M == m:
        assert g1[j, 1, 1] == oracle.goodput(*par, 1, 1, m, 0)[0]


@pytest.mark.gpu
@pytest.mark.parametrize("cfg,G", [(synth.TINY, 16), (synth.TESTBED, 64), (synth.TESTBED, 7)], ids=["tiny", "testbed", "ragged"])
def test_cuda_matches_oracle(oracle, cfg, G):
    import torch
    from paper_2008_12260_b200 import api

    cl, jobs = setup(cfg)
    ms = synth.make_m_samples(jobs.m0, jobs.m_max_total, G)
    rng = np.random.default_rng(3)
    adaptive = (rng.uniform(size=cfg.num_jobs) < 0.7).astype(np.uint8)
    s = api.scheduler_for(cfg, stream=torch.cuda.current_stream().cuda_stream)
    dj = api.DeviceJobs(jobs, "cuda:0", torch)
    dev = "cuda:0"
    for ad in (None, adaptive):
        gp = torch.full(s.table_shape, -1.0, dtype=torch.float32, device=dev)
        sp = torch.full(s.table_shape, -1.0, dtype=torch.float32, device=dev)
        am = torch.full(s.table_shape, 9, dtype=torch.uint16, device=dev)
        s.build_speedup_table_msample(dj, torch.from_numpy(ms).to(dev), torch.from_numpy(jobs.m_max_gpu).to(dev),
                                      gp, sp, am, adaptive=None if ad is None else torch.from_numpy(ad).to(dev))
        s.sync_status()
        gp_r, sp_r, am_r = oracle.build_speedup_table_msample(jobs, cl.node_capacity, cl.k_max, cl.n_max, ms,
                                                              jobs.m_max_gpu, adaptive=ad)
        assert_close(gp.cpu().numpy(), gp_r, what="goodput")
        assert_close(sp.cpu().numpy(), sp_r, what="speedup")
        am_g = am.cpu().numpy()
        assert np.array_equal(am_g == 0xFFFF, am_r == 0xFFFF)
        # where the chosen candidate differs, its goodput (from the oracle) must be within tolerance
        diff = np.argwhere(am_g != am_r)
        assert len(diff) < 0.02 * am_g.size
        for j, K, N in diff[:40]:
            one = jobs.take(np.array([j]))
            g1, _, _ = oracle.build_speedup_table_msample(one, cl.node_capacity, cl.k_max, cl.n_max,
                                                          ms[j:j + 1, am_g[j, K, N]:am_g[j, K, N] + 1], jobs.m_max_gpu[j:j + 1],
                                                          adaptive=None if ad is None else ad[j:j + 1], want_argmax=False)
            assert g1[0, K, N] >= gp_r[j, K, N] * (1 - REL_TOL)
    s.close()


@pytest.mark.gpu
def test_cuda_large_sampled(oracle):
    import torch
    from paper_2008_12260_b200 import api

    cfg = synth.LARGE
    cl, jobs = setup(cfg)
    ms = synth.make_m_samples(jobs.m0, jobs.m_max_total, 128)
    s = api.scheduler_for(cfg, stream=torch.cuda.current_stream().cuda_stream)
    dj = api.DeviceJobs(jobs, "cuda:0", torch)
    gp = torch.empty(s.table_shape, dtype=torch.float32, device="cuda:0")
    sp = torch.empty_like(gp)
    s.build_speedup_table_msample(dj, torch.from_numpy(ms).cuda(), torch.from_numpy(jobs.m_max_gpu).cuda(), gp, sp)
    s.sync_status()
    idx = np.array([0, 5, 300, 1023])
    sub = jobs.take(idx)
    gp_r, sp_r, _ = oracle.build_speedup_table_msample(sub, cl.node_capacity, cl.k_max, cl.n_max, ms[idx],
                                                       jobs.m_max_gpu[idx], want_argmax=False)
    assert_close(gp.cpu().numpy()[idx], gp_r, what="goodput")
    assert_close(sp.cpu().numpy()[idx], sp_r, what="speedup")
    s.close()
