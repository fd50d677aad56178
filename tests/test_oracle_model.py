"""Pins of the oracle's goodput model against what the paper and the mathematics fix."""
import math
import os

import numpy as np
import pytest

from paper_2008_12260_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden", "goodput_worked_examples.txt")


def test_worked_examples(oracle):
    n = 0
    for line in open(GOLD):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        f = line.split()
        params = [float(x) for x in f[:10]]
        K, N, m, s = (int(x) for x in f[10:14])
        num, den = float(f[14]), float(f[15])
        g, ok = oracle.goodput(*params, K, N, m, s)
        assert ok
        assert g == pytest.approx(num / den, rel=1e-13)
        n += 1
    assert n == 6


def test_efficiency_closed_forms(oracle):
    # Eq. 6: exactly 1 at M = M0, in (0, 1] beyond, decreasing in M, -> 1 as phi -> inf
    for phi in (1.0, 1e2, 1e5):
        for m0 in (64.0, 256.0):
            assert oracle.efficiency(phi, m0, m0) == 1.0
            prev = 1.0
            for mult in (2, 4, 8, 32):
                e = oracle.efficiency(phi, m0, mult * m0)
                assert 0.0 < e < prev
                prev = e
    assert oracle.efficiency(1e18, 64.0, 2048.0) == pytest.approx(1.0, abs=1e-12)
    # doubling the batch at phi = M0 costs exactly one third: (M0+M0)/(M0+2M0)
    assert oracle.efficiency(128.0, 128.0, 256.0) == pytest.approx(2.0 / 3.0, rel=1e-15)


def test_t_sync_cases(oracle):
    # Eq. 9
    assert oracle.t_sync(0.3, 0.1, 0.9, 0.2, 1, 1) == 0.0
    assert oracle.t_sync(0.3, 0.1, 0.9, 0.2, 2, 1) == pytest.approx(0.3)
    assert oracle.t_sync(0.3, 0.1, 0.9, 0.2, 5, 1) == pytest.approx(0.3 + 0.1 * 3)
    assert oracle.t_sync(0.3, 0.1, 0.9, 0.2, 2, 2) == pytest.approx(0.9)
    assert oracle.t_sync(0.3, 0.1, 0.9, 0.2, 7, 3) == pytest.approx(0.9 + 0.2 * 5)


def test_overlap_limits(oracle):
    # Eq. 10: gamma = 1 is the sum, gamma -> inf the max, always between the two
    rng = np.random.default_rng(0)
    for _ in range(200):
        tg, ts = rng.uniform(1e-3, 3.0, 2)
        assert oracle.t_iter(tg, ts, 1.0, 0) == pytest.approx(tg + ts, rel=1e-14)
        assert oracle.t_iter(tg, ts, 100.0, 0) == pytest.approx(max(tg, ts), rel=1e-2)
        prev = tg + ts
        for gamma in (1.5, 2.0, 4.0, 10.0):
            t = oracle.t_iter(tg, ts, gamma, 0)
            assert max(tg, ts) <= t <= prev + 1e-15
            prev = t
        # Eq. 11: each accumulation step adds exactly one T_grad
        assert oracle.t_iter(tg, ts, 3.0, 5) - oracle.t_iter(tg, ts, 3.0, 2) == pytest.approx(3 * tg, rel=1e-12)
    assert oracle.t_iter(3.0, 4.0, 2.0, 0) == pytest.approx(5.0, rel=1e-15)
    assert oracle.t_iter(3.0, 0.0, 7.0, 2) == pytest.approx(9.0, rel=1e-15)


def test_single_replica_throughput_independent_of_s(oracle):
    # K = 1 -> T_sync = 0 -> THROUGHPUT = m / (a_g + b_g m) whatever s (Eq. 7, 9, 11)
    a_g, b_g, m = 0.05, 0.002, 64
    for s in range(6):
        M = m * (s + 1)
        g, ok = oracle.goodput(a_g, b_g, 0.3, 0.3, 0.9, 0.9, 4.0, 500.0, 64.0, 1e9, 1, 1, m, s)
        assert ok
        thr = g / oracle.efficiency(500.0, 64.0, M)
        assert thr == pytest.approx(m / (a_g + b_g * m), rel=1e-13)


def test_feasibility_window(oracle):
    # only M0 <= M <= M_max is considered (Sec. 3, Sec. 3.1 upper limit)
    args = (0.05, 0.002, 0.01, 0.001, 0.03, 0.003, 2.0, 500.0, 128.0, 4096.0)
    assert not oracle.goodput(*args, 1, 1, 127, 0)[1]
    assert oracle.goodput(*args, 1, 1, 128, 0)[1]
    assert oracle.goodput(*args, 4, 2, 128, 7)[1]          # M = 4096
    assert not oracle.goodput(*args, 4, 2, 129, 7)[1]
    assert not oracle.goodput(*args, 2, 3, 128, 0)[1]      # more nodes than replicas


def _tiny_table(oracle, seed=0):
    cfg = synth.TINY
    jobs = draw = synth.draw_jobs(cfg.num_jobs, seed, cfg.grid_m, cfg.grid_s, 16)
    cl = cfg.cluster()
    fk, fn = oracle.fair_share(cl.node_capacity, jobs.num_jobs, cl.k_max)
    jobs.fair_k = np.full(jobs.num_jobs, fk, np.int32)
    jobs.fair_n = np.full(jobs.num_jobs, fn, np.int32)
    gp, sp, am = oracle.build_speedup_table(jobs, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s)
    return cfg, cl, jobs, gp, sp, am


def test_table_structure(oracle):
    cfg, cl, jobs, gp, sp, am = _tiny_table(oracle)
    KD, ND = cl.k_max + 1, cl.n_max + 1
    assert gp.shape == (8, KD, ND)
    G = cfg.gpus_per_node
    for K in range(KD):
        for N in range(ND):
            valid = N >= 1 and K >= N and K <= N * G
            if not valid:
                assert np.all(gp[:, K, N] == 0) and np.all(sp[:, K, N] == 0) and np.all(am[:, K, N] == 0xFFFF)
            else:
                assert np.all(gp[:, K, N] > 0) and np.all(am[:, K, N] != 0xFFFF)
    # Eq. 9 only distinguishes one node from several: columns N >= 2 agree where both valid
    for K in range(4, 9):
        assert np.array_equal(gp[:, K, 2], gp[:, K, 3]) or K > 2 * G or K < 3
    # node-level synchronisation is costlier than local in these inputs -> never faster
    for K in range(2, 5):
        assert np.all(gp[:, K, 1] >= gp[:, K, 2])
    # Eq. 15: speedup is exactly 1 at the fair share
    fk, fn = int(jobs.fair_k[0]), int(jobs.fair_n[0])
    assert (fk, fn) == (2, 1)
    assert np.all(sp[:, fk, fn] == 1.0)
    np.testing.assert_allclose(sp * gp[:, fk:fk + 1, fn:fn + 1], gp, rtol=1e-14)


def test_table_entry_is_the_grid_maximum(oracle):
    # the entry must dominate every grid point and be attained at the reported argmax
    cfg, cl, jobs, gp, sp, am = _tiny_table(oracle, seed=5)
    rng = np.random.default_rng(1)
    for _ in range(40):
        j = int(rng.integers(0, 8)); N = int(rng.integers(1, 5)); K = int(rng.integers(N, 4 * N + 1))
        par = [float(getattr(jobs, f)[j]) for f in synth.JOB_F32_FIELDS]
        best = 0.0
        for i in range(cfg.grid_m):
            for s in range(cfg.grid_s):
                g, ok = oracle.goodput(*par, K, N, int(jobs.m_grid[j, i]), s)
                if ok:
                    assert g <= gp[j, K, N]
                    best = max(best, g)
        assert best == gp[j, K, N]
        i, s = divmod(int(am[j, K, N]), cfg.grid_s)
        assert oracle.goodput(*par, K, N, int(jobs.m_grid[j, i]), s)[0] == gp[j, K, N]


def test_goodput_bounds(oracle):
    # goodput <= throughput < K / beta_grad (Eq. 7, 8: T_iter >= beta_grad m (s+1))
    cfg, cl, jobs, gp, sp, am = _tiny_table(oracle, seed=2)
    for K in range(1, cl.k_max + 1):
        assert np.all(gp[:, K, :].max(axis=1) < K / jobs.beta_grad.astype(np.float64))


def test_speedup_time_scale_invariance(oracle):
    # multiplying every alpha, beta by c rescales all goodputs by 1/c: speedups unchanged
    cfg, cl, jobs, gp, sp, am = _tiny_table(oracle, seed=3)
    scaled = jobs.take(slice(None))
    for f in ("alpha_grad", "beta_grad", "alpha_local", "beta_local", "alpha_node", "beta_node"):
        setattr(scaled, f, (getattr(jobs, f) * np.float32(4.0)))   # power of two: exact in fp32
    gp2, sp2, am2 = oracle.build_speedup_table(scaled, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s)
    np.testing.assert_allclose(gp2 * 4.0, gp, rtol=1e-13)
    np.testing.assert_allclose(sp2, sp, rtol=1e-13)
    assert np.array_equal(am, am2)


def test_argmax_tie_break(oracle):
    # duplicate grid values give exact ties: the smaller grid index must win; with
    # K = 1 and phi huge, goodput is m/(a+bm) whatever s: the smallest s must win
    jobs = synth.draw_jobs(1, 0, 4, 4, 4)
    jobs.m_grid = np.array([[64, 64, 64, 64]], np.int32)
    jobs.phi[:] = 1e30
    jobs.m0[:] = 64
    jobs.m_max_total[:] = 64 * 32
    jobs.fair_k = np.array([1], np.int32); jobs.fair_n = np.array([1], np.int32)
    cap = np.array([4], np.int16)
    gp, sp, am = oracle.build_speedup_table(jobs, cap, 4, 1, 4)
    assert am[0, 1, 1] == 0                     # i = 0, s = 0
    assert am[0, 2, 1] // 4 == 0


def test_fair_share(oracle):
    cap = np.full(16, 4, np.int16)
    assert oracle.fair_share(cap, 48, 64) == (1, 1)
    assert oracle.fair_share(cap, 8, 64) == (8, 2)
    assert oracle.fair_share(cap, 16, 64) == (4, 1)
    assert oracle.fair_share(cap, 1, 64) == (64, 16)
    assert oracle.fair_share(cap, 1000, 64) == (1, 1)     # less than one GPU each: 1-GPU goodput
    assert oracle.fair_share(np.array([8, 2, 2], np.int16), 2, 64) == (6, 1)
    assert oracle.fair_share(np.full(256, 8, np.int16), 3, 64) == (64, 8)


def test_realloc_factor(oracle):
    # (T - R delta)/(T + delta): 1 at delta = 0, hand values, clamped to [0, 1]
    age = np.array([600, 600, 60, 300], np.float32)
    r = np.array([0, 2, 5, 1], np.int32)
    assert np.all(oracle.realloc_factor(age, r, 0.0) == 1.0)
    f = oracle.realloc_factor(age, r, 30.0)
    np.testing.assert_allclose(f, [600 / 630, 540 / 630, 0.0, 270 / 330], rtol=1e-15)
