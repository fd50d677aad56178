"""Pins of the oracle's rack-level extension (the third synchronisation pair named after Eq. 9):
hand-worked values, the case analysis of T_sync, reductions to the two-class model, and an
independent evaluation of the fitness with racks."""
import itertools
import os

import numpy as np
import pytest

from helpers import with_fair_share
from paper_2008_12260_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden", "goodput_rack_worked_examples.txt")


def _jobs_with_rack(jobs, factor_a=1.0, factor_b=1.0):
    jobs.alpha_rack = (jobs.alpha_node * factor_a).astype(np.float32)
    jobs.beta_rack = (jobs.beta_node * factor_b).astype(np.float32)
    return jobs


def test_worked_examples_with_racks(oracle):
    n = 0
    for line in open(GOLD):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        f = line.split()
        params = [float(x) for x in f[:12]]
        K, N, R, m, s = (int(x) for x in f[12:17])
        num, den = float(f[17]), float(f[18])
        g, ok = oracle.goodput_rack(*params, K, N, R, m, s)
        assert ok
        assert g == pytest.approx(num / den, rel=1e-13)
        n += 1
    assert n == 6


def test_t_sync_rack_cases(oracle):
    pairs = (0.3, 0.1, 0.9, 0.2, 2.5, 0.4)
    assert oracle.t_sync_rack(*pairs, 1, 1, 1) == 0.0
    assert oracle.t_sync_rack(*pairs, 5, 1, 1) == pytest.approx(0.3 + 0.1 * 3)       # one node: local pair
    assert oracle.t_sync_rack(*pairs, 2, 2, 1) == pytest.approx(0.9)                 # one rack: node pair
    assert oracle.t_sync_rack(*pairs, 7, 3, 1) == pytest.approx(0.9 + 0.2 * 5)
    assert oracle.t_sync_rack(*pairs, 2, 2, 2) == pytest.approx(2.5)                 # two racks: rack pair
    assert oracle.t_sync_rack(*pairs, 7, 3, 2) == pytest.approx(2.5 + 0.4 * 5)
    assert oracle.t_sync_rack(*pairs, 7, 3, 3) == oracle.t_sync_rack(*pairs, 7, 3, 2)  # only "several racks" matters
    # with one rack occupied it is Eq. 9 itself
    for K, N in ((1, 1), (4, 1), (4, 2), (9, 4)):
        assert oracle.t_sync_rack(*pairs, K, N, 1) == oracle.t_sync(*pairs[:4], K, N)


@pytest.mark.parametrize("cfg", [synth.TINY, synth.TESTBED], ids=lambda c: c.name)
def test_rack_pair_equal_to_node_pair_gives_the_two_class_tables(oracle, cfg):
    cl = cfg.cluster()
    jobs = _jobs_with_rack(with_fair_share(cfg.jobs(), cl))
    gp, sp, am = oracle.build_speedup_table(jobs, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s)
    gr, sr, ar = oracle.build_speedup_table_rack(jobs, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s)
    assert np.array_equal(gr[:, :, 2:], gp[:, :, 2:]) and np.array_equal(sr[:, :, 2:], sp[:, :, 2:])
    assert np.array_equal(ar[:, :, 2:], am[:, :, 2:])
    assert not gr[:, :, :2].any() and not sr[:, :, :2].any() and np.all(ar[:, :, :2] == 0xFFFF)
    assert gr[:, :, 2:].any()


def test_slower_rack_links_lower_the_table_and_it_is_a_grid_maximum(oracle):
    cfg = synth.TINY
    cl = cfg.cluster()
    jobs = _jobs_with_rack(with_fair_share(cfg.jobs(), cl), 3.0, 2.0)
    gp, sp, _ = oracle.build_speedup_table(jobs, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s)
    gr, sr, ar = oracle.build_speedup_table_rack(jobs, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s)
    valid = gr > 0
    assert valid.any() and np.array_equal(valid[:, :, 2:], gp[:, :, 2:] > 0)
    assert np.all(gr[valid] < gp[valid])                      # strictly slower synchronisation
    # same denominator as the two-class table: the ratio of the two speedups is the ratio of the goodputs
    np.testing.assert_allclose(sr[valid] / sp[valid], gr[valid] / gp[valid], rtol=1e-12)
    # an entry is the brute-force maximum over the grid, attained at its argmax
    rng = np.random.default_rng(1)
    for _ in range(40):
        j, K, N = (int(x) for x in (rng.integers(jobs.num_jobs), rng.integers(2, cl.k_max + 1), rng.integers(2, cl.n_max + 1)))
        if not valid[j, K, N]:
            continue
        par = [float(getattr(jobs, f)[j]) for f in ("alpha_grad", "beta_grad", "alpha_local", "beta_local", "alpha_node",
                                                    "beta_node", "alpha_rack", "beta_rack", "gamma", "phi", "m0",
                                                    "m_max_total")]
        best = 0.0
        for i in range(cfg.grid_m):
            for s in range(cfg.grid_s):
                g, ok = oracle.goodput_rack(*par, K, N, 2, int(jobs.m_grid[j, i]), s)
                if ok:
                    best = max(best, g)
        assert gr[j, K, N] == best
        i, s = divmod(int(ar[j, K, N]), cfg.grid_s)
        assert oracle.goodput_rack(*par, K, N, 2, int(jobs.m_grid[j, i]), s)[0] == best


def _numpy_fitness_racks(mats, table, table_rack, rack, k_max, n_max, p, floor, cur, rf):
    A = mats.astype(np.int64)
    K = np.clip(A.sum(-1), 0, k_max)
    N = np.minimum((A > 0).sum(-1), n_max)
    lo = np.where(A > 0, rack[None, None, :], 10 ** 6).min(-1)
    hi = np.where(A > 0, rack[None, None, :], -1).max(-1)
    several = (N >= 1) & (lo != hi)
    j = np.arange(A.shape[1])[None, :]
    x = np.where(several, table_rack[j, K, N], table[j, K, N])
    changed = (A != cur[None].astype(np.int64)).any(-1) & (cur.sum(-1) > 0)[None, :]
    x = np.maximum(np.where(changed, x * rf[None, :], x), floor)
    if p == 1.0:
        return x.mean(1)
    if p == -1.0:
        return x.shape[1] / (1.0 / x).sum(1)
    return (x ** p).mean(1) ** (1.0 / p)


def test_fitness_with_racks_exhaustive_and_reductions(oracle):
    """Every 3-job matrix on 3 nodes x 2 GPUs (19 683) with nodes 0, 1 in rack 0 and node 2 in
    rack 1, against an independent numpy evaluation; one rack for all nodes gives Eq. 14 as before."""
    rng = np.random.default_rng(7)
    J, nodes, k_max, n_max = 3, 3, 6, 3
    table = rng.uniform(0.2, 2.5, (J, k_max + 1, n_max + 1))
    table_rack = table * rng.uniform(0.3, 0.9, table.shape)
    for t in (table, table_rack):
        t[:, 0, :] = 0.0
        t[:, :, 0] = 0.0
    rack = np.array([0, 0, 1], np.int16)
    cur = np.array([[1, 0, 0], [0, 0, 0], [1, 0, 1]], np.int16)
    rf = np.array([0.9, 0.5, 0.7])
    mats = np.array(list(itertools.product(range(3), repeat=J * nodes)), np.int16).reshape(-1, J, nodes)
    for p in (-1.0, 1.0, 0.5):
        ref = _numpy_fitness_racks(mats, table, table_rack, rack, k_max, n_max, p, 1e-3, cur, rf)
        got = oracle.eval_fitness_racks(mats, table, table_rack, rack, k_max, n_max, p, 1e-3, cur=cur, realloc=rf)
        np.testing.assert_allclose(got, ref, rtol=1e-12)
        one = oracle.eval_fitness_racks(mats, table, table_rack, np.zeros(3, np.int16), k_max, n_max, p, 1e-3, cur=cur,
                                        realloc=rf)
        assert np.array_equal(one, oracle.eval_fitness(mats, table, k_max, n_max, p, 1e-3, cur=cur, realloc=rf))
        same = oracle.eval_fitness_racks(mats, table, table, rack, k_max, n_max, p, 1e-3, cur=cur, realloc=rf)
        assert np.array_equal(same, one)
    # a hand case: job 0 on nodes 0 and 2 (two racks), job 1 on nodes 0 and 1 (one rack), job 2 on node 2
    A = np.array([[[1, 0, 1], [1, 1, 0], [0, 0, 2]]], np.int16)
    want = (table_rack[0, 2, 2] + table[1, 2, 2] + table[2, 2, 1]) / 3.0
    assert oracle.eval_fitness_racks(A, table, table_rack, rack, k_max, n_max, 1.0, 0.0)[0] == pytest.approx(want, rel=1e-15)
