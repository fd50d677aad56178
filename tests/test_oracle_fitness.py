"""Pins of the oracle's fitness (Eq. 14, the re-allocation penalty) against library power
means, closed forms and exhaustive enumeration on a sub-tiny cluster."""
import itertools

import numpy as np
import pytest
import scipy.stats as st


def _lookup(pop, table, k_max, n_max):
    K = np.clip(pop.astype(np.int64).sum(-1), 0, k_max)
    N = np.minimum((pop > 0).sum(-1), n_max)
    J = pop.shape[1]
    return table[np.arange(J)[None, :], K, N]


def _random_case(seed, P=6, J=7, nodes=5, k_max=12, n_max=5):
    rng = np.random.default_rng(seed)
    table = rng.uniform(0.05, 3.0, (J, k_max + 1, n_max + 1))
    pop = np.where(rng.uniform(size=(P, J, nodes)) < 0.4, rng.integers(1, 4, (P, J, nodes)), 0).astype(np.int16)
    return pop, table, k_max, n_max


@pytest.mark.parametrize("p", [1.0, -1.0, 0.0, 0.5, -3.0, 2.0])
def test_power_mean_matches_library(oracle, p):
    pop, table, k_max, n_max = _random_case(1)
    x = _lookup(pop, table, k_max, n_max)
    got = oracle.eval_fitness(pop, table, k_max, n_max, p, 0.0)
    if p == 1.0:
        ref = x.mean(axis=1)
    elif p == -1.0:
        ref = st.hmean(x, axis=1)
    elif p == 0.0:
        ref = st.gmean(x, axis=1)
    else:
        ref = st.pmean(x, p, axis=1)
    np.testing.assert_allclose(got, ref, rtol=1e-12)


def test_power_mean_inequalities_and_bounds(oracle):
    pop, table, k_max, n_max = _random_case(2, P=20)
    x = _lookup(pop, table, k_max, n_max)
    f = {p: oracle.eval_fitness(pop, table, k_max, n_max, p, 0.0) for p in (-10.0, -1.0, 0.0, 0.5, 1.0)}
    assert np.all(f[-10.0] <= f[-1.0]) and np.all(f[-1.0] <= f[0.0])
    assert np.all(f[0.0] <= f[0.5]) and np.all(f[0.5] <= f[1.0])
    for v in f.values():
        assert np.all(v >= x.min(axis=1) * (1 - 1e-12)) and np.all(v <= x.max(axis=1) * (1 + 1e-12))
    # p -> -inf approaches the minimum speedup
    np.testing.assert_allclose(oracle.eval_fitness(pop, table, k_max, n_max, -200.0, 0.0), x.min(axis=1), rtol=2e-2)


def test_all_equal_speedups(oracle):
    pop, table, k_max, n_max = _random_case(3)
    table[:] = 1.75
    for p in (-1.0, 0.0, 0.5, 1.0, -4.0):
        np.testing.assert_allclose(oracle.eval_fitness(pop, table, k_max, n_max, p, 0.0), 1.75, rtol=1e-13)


def test_penalty_hand_example(oracle):
    # two jobs, one node pair; table value depends on K only
    table = np.zeros((2, 5, 3))
    table[0, :, :] = np.array([0, 1, 2, 3, 4])[:, None]
    table[1, :, :] = np.array([0, 0.5, 1, 1.5, 2])[:, None]
    cur = np.array([[2, 0], [1, 0]], np.int16)
    pop = np.array([[[2, 0], [1, 0]],      # unchanged: x = (2, 0.5)
                    [[2, 0], [0, 1]],      # job 1 moved: x = (2, 0.5 * 0.5)
                    [[1, 1], [1, 0]]],     # job 0 changed: x = (2 * 0.25, 0.5)
                   np.int16)
    rf = np.array([0.25, 0.5])
    got = oracle.eval_fitness(pop, table, 4, 2, -1.0, 0.0, cur=cur, realloc=rf)
    np.testing.assert_allclose(got, [2 / (0.5 + 2), 2 / (0.5 + 4), 2 / (2 + 2)], rtol=1e-15)
    # no current allocation, or a factor of one (delta = 0): no penalty at all
    base = oracle.eval_fitness(pop, table, 4, 2, -1.0, 0.0)
    np.testing.assert_allclose(oracle.eval_fitness(pop, table, 4, 2, -1.0, 0.0, cur=cur, realloc=np.ones(2)), base)
    # a pending job (no GPUs now) is never penalised
    cur0 = np.array([[0, 0], [1, 0]], np.int16)
    got0 = oracle.eval_fitness(pop, table, 4, 2, 1.0, 0.0, cur=cur0, realloc=rf)
    np.testing.assert_allclose(got0, [(2 + 0.5) / 2, (2 + 0.25) / 2, (2 + 0.5) / 2], rtol=1e-15)


def test_floor_and_inactive(oracle):
    table = np.zeros((3, 3, 2))
    table[:, 1, 1] = [1.0, 2.0, 4.0]
    pop = np.array([[[1], [1], [0]]], np.int16)          # job 2 has no GPUs: speedup 0
    assert oracle.eval_fitness(pop, table, 2, 1, -1.0, 0.0)[0] == 0.0
    got = oracle.eval_fitness(pop, table, 2, 1, -1.0, 1e-3)[0]
    assert got == pytest.approx(3.0 / (1.0 + 0.5 + 1000.0), rel=1e-14)
    act = np.array([1, 1, 0], np.uint8)
    assert oracle.eval_fitness(pop, table, 2, 1, -1.0, 1e-3, active=act)[0] == pytest.approx(2 / 1.5, rel=1e-14)
    assert oracle.eval_fitness(pop, table, 2, 1, 1.0, 1e-3, active=np.zeros(3, np.uint8))[0] == 0.0


def test_out_of_range_rows_are_clamped(oracle):
    table = np.arange(2 * 3 * 3, dtype=np.float64).reshape(2, 3, 3) + 1
    pop = np.array([[[9, 9, 9], [-5, 0, 0]]], np.int16)  # K = 27 -> 2, N = 3 -> 2; K = -5 -> 0, N = 0
    got = oracle.eval_fitness(pop, table, 2, 2, 1.0, 0.0)[0]
    assert got == pytest.approx((table[0, 2, 2] + table[1, 0, 0]) / 2)


def test_exhaustive_sub_tiny(oracle):
    """Every 3-job allocation matrix on 2 nodes with entries 0..2 (3^6 = 729), p = -1 with
    penalty and floor: the oracle against an independent numpy/scipy evaluation."""
    rng = np.random.default_rng(5)
    J, nodes, k_max, n_max = 3, 2, 4, 2
    table = rng.uniform(0.2, 2.5, (J, k_max + 1, n_max + 1))
    table[:, 0, :] = 0.0
    table[:, :, 0] = 0.0
    cur = np.array([[1, 0], [0, 0], [1, 1]], np.int16)
    rf = np.array([0.9, 0.5, 0.7])
    mats = np.array(list(itertools.product(range(3), repeat=J * nodes)), np.int16).reshape(-1, J, nodes)
    assert mats.shape[0] == 729
    x = _lookup(mats, table, k_max, n_max)
    changed = (mats != cur[None]).any(-1) & (cur.sum(-1) > 0)[None, :]
    x = np.maximum(np.where(changed, x * rf[None, :], x), 1e-3)
    for p in (-1.0, 1.0, 0.5):
        ref = st.pmean(x, p, axis=1)
        got = oracle.eval_fitness(mats, table, k_max, n_max, p, 1e-3, cur=cur, realloc=rf)
        np.testing.assert_allclose(got, ref, rtol=1e-12)
