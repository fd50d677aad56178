"""Trace replay: host-side input generation and bookkeeping (CPU), and a few rounds on the
GPU checked against the oracle."""
import numpy as np
import pytest

from helpers import REL_TOL, feasible
from paper_2008_12260_b200 import synth


def test_trace_inputs_and_bookkeeping():
    from paper_2008_12260_b200 import trace
    tr = trace.TraceReplay()
    assert tr.num_rounds == 480
    n_active = []
    for k in (0, 1, 60, 240, 479):
        jobs, cur = tr.round_inputs(k)
        t = 60.0 * k
        expect = (tr.arrive <= t) & (t < tr.arrive + tr.life)
        assert np.array_equal(jobs.active.astype(bool), expect)
        assert np.all(jobs.phi >= tr.phi0.astype(np.float32) * 0.999) and np.all(jobs.phi <= tr.phi0 * 10.001)
        assert not cur[~expect].any()
        n_active.append(int(expect.sum()))
        total = 64 // max(n_active[-1], 1)
        assert jobs.fair_k[0] == min(max(total, 1), 64)
    assert max(n_active) > 5
    # a running job whose row changes is counted as re-allocated once; a pending one is not
    jobs, cur = tr.round_inputs(100)
    act = np.nonzero(jobs.active)[0]
    cur[:] = 0
    cur[act[0], 0] = 2
    best = cur.copy()
    best[act[0], 0] = 1            # running job shrinks
    best[act[1], 1] = 1            # pending job starts
    tr.commit(100, jobs, cur, best)
    assert tr.restarts[act[0]] == 1 and tr.restarts[act[1]] == 0
    assert np.array_equal(tr.cur, best)
    tr.reset()
    assert not tr.restarts.any() and not tr.cur.any()


@pytest.mark.gpu
def test_trace_rounds_on_gpu(oracle):
    import torch
    from paper_2008_12260_b200 import api, trace

    tr = trace.TraceReplay(generations=30)
    cfg, cl = tr.cfg, tr.cluster
    stream = torch.cuda.Stream()
    s = api.scheduler_for(cfg, stream=stream.cuda_stream)
    checked = []

    def check(k, jobs, cur, best, fit):
        act = jobs.active.astype(bool)
        assert feasible(best, cl.node_capacity, jobs.k_cap, cl.n_max)
        assert not best[~act].any()
        if k % 7 == 0 and act.any():
            _, sp, _ = oracle.build_speedup_table(jobs, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s,
                                                  want_argmax=False)
            rf = oracle.realloc_factor(jobs.age_sec, jobs.num_restarts, cfg.delta_sec)
            ref = oracle.eval_fitness(best[None], sp, cl.k_max, cl.n_max, cfg.p, cfg.speedup_floor, cur=cur,
                                      realloc=rf, active=jobs.active)[0]
            assert abs(fit - ref) <= 3 * REL_TOL * abs(ref)
            keep = oracle.eval_fitness(cur[None], sp, cl.k_max, cl.n_max, cfg.p, cfg.speedup_floor, cur=cur,
                                       realloc=rf, active=jobs.active)[0]
            assert fit >= keep * (1 - 3 * REL_TOL)        # never worse than keeping the allocation
            checked.append(k)

    fits, used = trace.replay(s, tr, torch, rounds=40, first_round=30, on_round=check)
    assert len(checked) >= 5 and max(used) <= 64 and max(used) > 0
    # a second replay from the same state reproduces the same rounds (graph replay included)
    tr.reset()
    fits2, used2 = trace.replay(s, tr, torch, rounds=40, first_round=30)
    tr.reset()
    fits3, used3 = trace.replay(s, tr, torch, rounds=40, first_round=30)
    assert fits2 == fits3 and used2 == used3
    s.close()
