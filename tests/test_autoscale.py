"""The goodput-driven auto-scaling rule (Sec. 5.3): oracle pins and CUDA parity."""
import numpy as np
import pytest

from helpers import setup
from paper_2008_12260_b200 import synth


def test_hand_cases(oracle):
    # one job, nodes of 4 GPUs: g(1 node) = 3.5 of an ideal 4, g(2 nodes) = 4.0 of an ideal 8
    g = np.zeros((1, 9, 3), np.float32)
    g[0, 1, 1] = 1.0; g[0, 4, 1] = 3.5; g[0, 8, 2] = 4.0
    assert oracle.autoscale_targets(g, 8, 2, 4, [1], 2 / 3, 0.5).tolist() == [2]     # 3.5 > 2.67, 4.0 >= 4.0
    assert oracle.autoscale_targets(g, 8, 2, 4, [1], 0.9, 0.5).tolist() == [1]       # 3.5 <= 3.6: stay
    assert oracle.autoscale_targets(g, 8, 2, 4, [1], 2 / 3, 0.51).tolist() == [1]    # 4.0 < 4.08: no target
    assert oracle.autoscale_targets(g, 8, 2, 4, [2], 0.1, 0.1).tolist() == [2]       # already at the limit
    assert oracle.autoscale_targets(g, 8, 2, 4, [0], 0.1, 0.1).tolist() == [0]       # no nodes: untouched
    assert oracle.autoscale_targets(g, 8, 2, 4, [7], 0.1, 0.1).tolist() == [7]       # outside the table
    # n_max = 3 nodes of 4 GPUs would need 12 > k_max = 8 GPUs: the search stops at 2 nodes.
    # (A second job with large entries follows, so that a read past row k_max would show.)
    g = np.zeros((2, 9, 4), np.float32)
    g[0, 1, 1] = 1.0; g[0, 4, 1] = 3.5; g[0, 8, 2] = 4.0
    g[1] = 100.0
    assert oracle.autoscale_targets(g, 8, 3, 4, [1, 0], 2 / 3, 0.5).tolist() == [2, 0]
    assert oracle.autoscale_targets(g, 8, 3, 4, [3, 0], 0.1, 0.1).tolist() == [3, 0]


def test_properties_on_model_tables(oracle):
    cfg = synth.TESTBED
    cl, jobs = setup(cfg)
    gp, _, _ = oracle.build_speedup_table(jobs, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s, want_argmax=False)
    g32 = gp.astype(np.float32)
    cur = np.ones(cfg.num_jobs, np.int32)
    prev = None
    for U in (0.2, 0.5, 2 / 3, 0.9, 1.1):
        t = oracle.autoscale_targets(g32, cl.k_max, cl.n_max, 4, cur, U, 0.5)
        assert np.all(t >= cur) and np.all(t <= cl.n_max)                 # never scales down
        if prev is not None:
            assert np.all((t > cur) <= (prev > cur))                      # a stricter U scales fewer jobs
        prev = t
    assert np.all(oracle.autoscale_targets(g32, cl.k_max, cl.n_max, 4, cur, 1.1, 0.5) == cur)  # g/K <= g(1) here
    lo = oracle.autoscale_targets(g32, cl.k_max, cl.n_max, 4, cur, 0.2, 0.3)
    hi = oracle.autoscale_targets(g32, cl.k_max, cl.n_max, 4, cur, 0.2, 0.7)
    assert np.all(lo >= hi)                                               # a looser L reaches at least as far
    # the target satisfies its defining inequality and no larger node count does
    for j in range(cfg.num_jobs):
        n = int(lo[j])
        if n > 1:
            assert g32[j, 4 * n, n] >= np.float32(np.float32(np.float32(0.3) * np.float32(4 * n)) * g32[j, 1, 1])
            for m in range(n + 1, cl.n_max + 1):
                assert g32[j, 4 * m, m] < np.float32(np.float32(np.float32(0.3) * np.float32(4 * m)) * g32[j, 1, 1])


@pytest.mark.gpu
@pytest.mark.parametrize("cfg", [synth.TESTBED, synth.LARGE], ids=lambda c: c.name)
def test_cuda_matches_oracle(oracle, cfg):
    import torch
    from paper_2008_12260_b200 import api

    cl, jobs = setup(cfg)
    s = api.scheduler_for(cfg, stream=torch.cuda.current_stream().cuda_stream)
    dj = api.DeviceJobs(jobs, "cuda:0", torch)
    gp = torch.empty(s.table_shape, dtype=torch.float32, device="cuda:0")
    sp = torch.empty_like(gp)
    s.build_speedup_table(dj, gp, sp, None)
    rng = np.random.default_rng(1)
    cur = rng.integers(0, 5, cfg.num_jobs).astype(np.int32)
    cur[:3] = [0, 99, -2]
    g_host = gp.cpu().numpy()
    for U, L in ((2 / 3, 0.5), (0.3, 0.2), (0.5, 0.45), (1.5, 0.5)):
        out = torch.full((cfg.num_jobs,), -7, dtype=torch.int32, device="cuda:0")
        s.autoscale_targets(gp, torch.from_numpy(cur).cuda(), out, gpus_per_node=cfg.gpus_per_node, U=U, L=L)
        s.sync_status()
        ref = oracle.autoscale_targets(g_host, cl.k_max, cl.n_max, cfg.gpus_per_node, cur, U, L)
        assert np.array_equal(out.cpu().numpy(), ref)
    assert (ref >= np.minimum(cur, ref)).all()
    s.close()
