"""Pins of the oracle's genetic operators: ranking against numpy sorting, hand-worked
mutation and repair cases, repair post-conditions (exhaustively on a sub-tiny cluster),
and the statistics of selection / crossover / mutation that their definitions imply."""
import itertools
import math

import numpy as np
import pytest

from paper_2008_12260_b200 import synth

U32 = 1 << 32


def test_rank_matches_stable_sort(oracle):
    rng = np.random.default_rng(0)
    f = rng.normal(size=300).astype(np.float32)
    f[10] = f[200] = f[77]                    # ties: lower index first
    f[5] = -0.0; f[6] = 0.0                   # -0 sorts below +0 in the total order
    f[8] = np.inf; f[9] = -np.inf
    r = oracle.rank(f)
    order = np.lexsort((np.arange(f.size), -f.astype(np.float64)))
    # lexsort treats -0 == +0 (tie by index: 5 first); the total order puts +0 first
    exp = np.empty(f.size, np.int32); exp[order] = np.arange(f.size)
    a, b = exp[5], exp[6]
    exp[5], exp[6] = max(a, b), min(a, b)
    assert r.tolist() == exp.tolist()
    assert sorted(r.tolist()) == list(range(f.size))


def _w_for(n, of):
    """smallest 32-bit word w with floor(w * of / 2^32) == n"""
    return -(-n * U32 // of)


def test_mutate_row_hand_cases(oracle):
    row = [0, 2, 0, 1, 0, 3]
    thr = 1000
    # not selected: w0 >= thr
    assert oracle.mutate_row(row, [1000, 0, 0, 0], thr).tolist() == row
    # grow (op 0) on node 4
    assert oracle.mutate_row(row, [999, _w_for(0, 3), 123, _w_for(4, 6)], thr).tolist() == [0, 2, 0, 1, 1, 3]
    # shrink (op 1): occupied nodes ascending are 1, 3, 5; pick the third
    assert oracle.mutate_row(row, [0, _w_for(1, 3), _w_for(2, 3), 77], thr).tolist() == [0, 2, 0, 1, 0, 2]
    # shrink to empty
    assert oracle.mutate_row(row, [0, _w_for(1, 3), _w_for(1, 3), 77], thr).tolist() == [0, 2, 0, 0, 0, 3]
    # relocate (op 2): second occupied node (3) onto node 0; onto an occupied node adds
    assert oracle.mutate_row(row, [0, _w_for(2, 3), _w_for(1, 3), _w_for(0, 6)], thr).tolist() == [1, 2, 0, 0, 0, 3]
    assert oracle.mutate_row(row, [0, _w_for(2, 3), _w_for(0, 3), _w_for(5, 6)], thr).tolist() == [0, 0, 0, 1, 0, 5]
    # relocate onto itself: nothing
    assert oracle.mutate_row(row, [0, _w_for(2, 3), _w_for(0, 3), _w_for(1, 6)], thr).tolist() == row
    # shrink / relocate of an empty row: nothing; grow still works
    empty = [0, 0, 0]
    assert oracle.mutate_row(empty, [0, _w_for(1, 3), 5, 5], thr).tolist() == empty
    assert oracle.mutate_row(empty, [0, _w_for(2, 3), 5, 5], thr).tolist() == empty
    assert oracle.mutate_row(empty, [0, 0, 5, U32 - 1], thr).tolist() == [0, 0, 1]


def test_repair_hand_example(oracle):
    cap = np.array([2, 2, 2], np.int16)
    A = np.array([[2, 1, 0], [1, 1, 0], [0, 0, 3], [0, 1, 1]], np.int16)
    out = oracle.repair_with_offsets(A, cap, np.full(4, 64, np.int32), 6, 3, [1, 3, 0], [0, 2, 3])
    # row pass: job 2 clipped to the node size.  interference: node 0 keeps job 1 (first
    # distributed job from offset 1), node 1 keeps job 3 (from offset 3), node 2 has only
    # job 3 distributed.  capacity: node 2 holds 2 + 1 > 2, taken from job 3 (offset 3).
    assert out.tolist() == [[0, 0, 0], [1, 0, 0], [0, 0, 2], [0, 1, 0]]


def test_repair_row_caps_hand_example(oracle):
    cap = np.full(4, 2, np.int16)
    A = np.array([[2, 2, 2, 2]], np.int16)
    out = oracle.repair_with_offsets(A, cap, np.array([5], np.int32), 8, 4, [0] * 4, [0] * 4)
    assert out.tolist() == [[2, 2, 1, 0]]          # 3 replicas too many: from the last node down
    out = oracle.repair_with_offsets(A, cap, np.array([5], np.int32), 8, 2, [0] * 4, [0] * 4)
    assert out.tolist() == [[2, 2, 0, 0]]          # then at most n_max nodes: the last ones go
    out = oracle.repair_with_offsets(np.array([[-3, 7, 1, 0]], np.int16), cap, np.array([64], np.int32), 8, 4,
                                     [0] * 4, [0] * 4)
    assert out.tolist() == [[0, 2, 1, 0]]
    out = oracle.repair_with_offsets(A, cap, np.array([64], np.int32), 8, 4, [0] * 4, [0] * 4,
                                     active=np.array([0], np.uint8))
    assert out.tolist() == [[0, 0, 0, 0]]


def test_capacity_pass_rotation(oracle):
    # one node of 3 GPUs, four single-node jobs with 2 each: excess 5, walk from job 2:
    # job 2 loses 2, job 3 loses 2, job 0 loses 1
    cap = np.array([3], np.int16)
    A = np.array([[2], [2], [2], [2]], np.int16)
    out = oracle.repair_with_offsets(A, cap, np.full(4, 64, np.int32), 3, 1, [0], [2])
    assert out.ravel().tolist() == [1, 2, 0, 0]


def _check_post_conditions(A_in, A_out, cap, k_cap, n_max):
    A_in = np.clip(A_in.astype(np.int64), 0, None)
    o = A_out.astype(np.int64)
    assert np.all(o >= 0)
    assert np.all(o <= np.minimum(A_in, cap[None, :]))                 # removal only
    assert np.all(o.sum(0) <= cap)                                     # node capacity
    assert np.all(o.sum(1) <= k_cap)                                   # replica cap per job
    occ = (o > 0)
    assert np.all(occ.sum(1) <= n_max)
    dist = occ.sum(1) >= 2
    assert np.all((occ & dist[:, None]).sum(0) <= 1)                   # <= 1 distributed job per node


def test_repair_post_conditions_random(oracle):
    cl = synth.uniform_cluster(6, 4)
    raw = synth.random_raw_population(40, 9, cl, seed=3, density=0.45, v_hi=6)
    k_cap = np.array([3, 64, 64, 5, 64, 64, 8, 64, 64], np.int32)
    for c in range(raw.shape[0]):
        out = oracle.repair(raw[c], cl.node_capacity, k_cap, 24, 6, 11, 2, c, 7)
        _check_post_conditions(raw[c], out, cl.node_capacity.astype(np.int64), np.minimum(k_cap, 24), 6)
        again = oracle.repair(out, cl.node_capacity, k_cap, 24, 6, 999, 5, c + 1, 3)   # any stream
        assert np.array_equal(again, out)                                            # fixed point


def test_repair_identity_on_feasible(oracle):
    cl = synth.uniform_cluster(16, 4)
    for seed in range(5):
        A = synth.random_feasible_allocation(cl, 48, seed)
        out = oracle.repair(A, cl.node_capacity, np.full(48, 64, np.int32), 64, 16, 1, 0, 0, 0)
        assert np.array_equal(out, A)


def test_repair_exhaustive_sub_tiny(oracle):
    """All 3-job matrices on 2 nodes x 2 GPUs with entries 0..2: post-conditions, fixed
    point, and minimal removal in the capacity pass (each column loses exactly its excess
    once interference has been resolved)."""
    cap = np.array([2, 2], np.int16)
    k_cap = np.full(3, 4, np.int32)
    for vals in itertools.product(range(3), repeat=6):
        A = np.array(vals, np.int16).reshape(3, 2)
        for oi, oc in (([0, 0], [0, 0]), ([1, 2], [2, 1])):
            out = oracle.repair_with_offsets(A, cap, k_cap, 4, 2, oi, oc)
            _check_post_conditions(A, out, cap.astype(np.int64), k_cap, 2)
            assert np.array_equal(oracle.repair_with_offsets(out, cap, k_cap, 4, 2, [2, 0], [1, 1]), out)
            # interference pass by hand: distributed jobs are those with both entries > 0
            dist = (A > 0).all(1)
            mid = A.copy()
            for n in range(2):
                idx = [j for j in [(oi[n] + t) % 3 for t in range(3)] if dist[j]]
                for j in idx[1:]:
                    mid[j, n] = 0
            assert np.array_equal(out.sum(0), np.minimum(mid.sum(0), 2))
            feasible = A.sum(0).max() <= 2 and dist.sum() <= 1
            if feasible:
                assert np.array_equal(out, A)


def _signature_population(P, J, nodes):
    """parent i puts i+1 replicas of job j on node j % nodes: a row identifies its parent"""
    pop = np.zeros((P, J, nodes), np.int16)
    for i in range(P):
        for j in range(J):
            pop[i, j, j % nodes] = i + 1
    return pop


def test_selection_and_crossover_statistics(oracle):
    """With huge nodes and no mutation the repair is the identity, so every child row is a
    verbatim parent row.  Elites must be the top-ranked parents; other children must mix
    exactly two parents; a parent of rank r wins a binary tournament with probability
    (2(P - r) - 1) / P^2; the two parents contribute about half the rows each."""
    P, J, nodes, E = 32, 40, 8, 3
    cap = np.full(nodes, 30000, np.int16)
    k_cap = np.full(J, 64, np.int32)
    pop = _signature_population(P, J, nodes)
    rng = np.random.default_rng(4)
    fit = rng.uniform(0, 1, P).astype(np.float32)
    rank = oracle.rank(fit)
    order = np.argsort(rank)
    wins = np.zeros(P)
    from_b = []
    for gen in range(60):
        child = oracle.ga_generation(pop, fit, cap, k_cap, 64, 8, E, 0, 42, 1, gen)
        src = child.max(axis=2).astype(np.int64) - 1            # [P][J] parent index per row
        assert np.array_equal(child, pop[src, np.arange(J)[None, :]])
        for c in range(E):
            assert np.all(src[c] == order[c])
        for c in range(E, P):
            parents = np.unique(src[c])
            assert parents.size <= 2
            for q in parents:
                wins[rank[q]] += 1.0 / parents.size * 2          # both tournaments when pa == pb
            if parents.size == 2:
                from_b.append(np.mean(src[c] == parents[1]))
    total = wins.sum()
    expect = np.array([(2 * (P - r) - 1) / P**2 for r in range(P)]) * total
    chi2 = ((wins - expect) ** 2 / expect).sum()
    assert chi2 < 70.0                                           # 31 dof
    assert np.corrcoef(wins, expect)[0, 1] > 0.9
    assert abs(np.mean(from_b) - 0.5) < 0.03
    # A fair coin per row over J = 40 rows leaves the minority parent about 0.44 of them
    # (0.5 - E|Binomial(40, 1/2)/40 - 1/2|); a coin biased to 3/4 would leave it 0.25.
    minority = np.minimum(from_b, 1.0 - np.asarray(from_b))
    assert 0.41 < minority.mean() < 0.47


def test_mutation_statistics(oracle):
    """Threshold 2^32 - 1 mutates (almost surely) every row of every non-elite child: each
    row then differs from its parent's by one grow (+1 on one node), one shrink (-1), or
    one relocate (sum preserved), each about a third of the time."""
    P, J, nodes = 64, 1, 8          # a single job: no interference between distributed rows
    cap = np.full(nodes, 30000, np.int16)
    k_cap = np.full(J, 64, np.int32)
    pop = np.zeros((P, J, nodes), np.int16)
    pop[:, :, 2] = 3; pop[:, :, 5] = 4                           # every parent row identical
    fit = np.linspace(0, 1, P).astype(np.float32)
    counts = {"grow": 0, "shrink": 0, "move": 0, "same": 0}
    for gen in range(60):
        child = oracle.ga_generation(pop, fit, cap, k_cap, 64, 8, 1, U32 - 1, 9, 0, gen)
        assert np.array_equal(child[0], pop[P - 1])              # elite untouched
        d = child[1:].astype(np.int64) - pop[0][None].astype(np.int64)
        for row in d.reshape(-1, nodes):
            nz = row[row != 0]
            if nz.size == 0:
                counts["same"] += 1
            elif nz.size == 1 and nz[0] == 1:
                counts["grow"] += 1
            elif nz.size == 1 and nz[0] == -1:
                counts["shrink"] += 1
            else:
                assert row.sum() == 0 and nz.size == 2 and (nz.min() in (-3, -4))
                counts["move"] += 1
    n = sum(counts.values())
    assert abs(counts["grow"] / n - 1 / 3) < 0.03
    assert abs(counts["shrink"] / n - 1 / 3) < 0.03
    # a relocate lands on its own node with probability 1/8 and then changes nothing
    assert abs(counts["move"] / n - (1 / 3) * (7 / 8)) < 0.03
    assert abs(counts["same"] / n - (1 / 3) * (1 / 8)) < 0.02


def test_mutation_rate(oracle):
    P, J, nodes = 16, 64, 4
    cap = np.full(nodes, 30000, np.int16)
    pop = np.zeros((P, J, nodes), np.int16)
    fit = np.zeros(P, np.float32)
    thr = synth.prob_to_threshold(0.25)
    changed = 0
    for gen in range(30):
        child = oracle.ga_generation(pop, fit, cap, np.full(J, 64, np.int32), 64, 4, 0, thr, 5, 3, gen)
        changed += (child != 0).any(axis=2).sum()
    # on an empty row only "grow" (one op in three) has an effect
    assert abs(changed / (30 * P * J) - 0.25 / 3) < 0.01


def test_init_population(oracle):
    cfg = synth.TESTBED
    cl = cfg.cluster()
    cur = cfg.cur()
    k_cap = np.full(cfg.num_jobs, cl.k_max, np.int32)
    pop = oracle.init_population(20, cur, cfg.num_jobs, cl.node_capacity, k_cap, cl.k_max, cl.n_max,
                                 synth.prob_to_threshold(0.2), 1, 0)
    assert np.array_equal(pop[0], cur)
    diff_rows = (pop[1:] != cur[None]).any(axis=2).sum(axis=1)
    assert diff_rows.min() >= 1 and diff_rows.max() < cfg.num_jobs // 2
    for c in range(20):
        _check_post_conditions(pop[c], pop[c], cl.node_capacity.astype(np.int64), k_cap, cl.n_max)
    same = oracle.init_population(5, cur, cfg.num_jobs, cl.node_capacity, k_cap, cl.k_max, cl.n_max, 0, 1, 0)
    assert all(np.array_equal(same[c], cur) for c in range(5))
    empty = oracle.init_population(3, None, 4, cl.node_capacity, np.full(4, 64, np.int32), 64, 16, 0, 1, 0)
    assert not empty.any()


def test_round_improves_and_is_deterministic(oracle):
    cfg = synth.TINY
    cl = cfg.cluster()
    jobs = cfg.jobs()
    fk, fn = oracle.fair_share(cl.node_capacity, cfg.num_jobs, cl.k_max)
    jobs.fair_k = np.full(cfg.num_jobs, fk, np.int32); jobs.fair_n = np.full(cfg.num_jobs, fn, np.int32)
    args = (jobs, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s, cfg.population, cfg.p, cfg.delta_sec,
            cfg.speedup_floor, cfg.num_elite, synth.prob_to_threshold(cfg.mutate_prob),
            synth.prob_to_threshold(cfg.init_prob), 0, 0)
    cur = cfg.cur()
    b0, f0 = oracle.schedule_round(*args, 0, cur)
    b1, f1 = oracle.schedule_round(*args, 30, cur)
    b2, f2 = oracle.schedule_round(*args, 30, cur)
    assert np.array_equal(b1, b2) and f1 == f2
    assert f1 >= f0 and f1 > 0.3
    _check_post_conditions(b1, b1, cl.node_capacity.astype(np.int64), jobs.k_cap, cl.n_max)
    # elitism: the best fitness never decreases with more generations
    fs = [oracle.schedule_round(*args, g, cur)[1] for g in (0, 1, 2, 5, 10)]
    assert all(b >= a for a, b in zip(fs, fs[1:]))
