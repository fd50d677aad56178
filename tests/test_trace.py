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
            _, sp_ref, _ = oracle.build_speedup_table(jobs, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s,
                                                      want_argmax=False)
            d_sp = torch.empty(s.table_shape, dtype=torch.float32, device="cuda:0")
            s.get_round_tables(None, d_sp)
            stream.synchronize()
            sp = d_sp.cpu().numpy().astype(np.float64)     # the round's own table: within 1e-5 of the oracle's,
            on = act                                       # and the fitness is then checked on that very table
            np.testing.assert_allclose(sp[on], sp_ref[on], rtol=REL_TOL, atol=0)
            rf = oracle.realloc_factor(jobs.age_sec, jobs.num_restarts, cfg.delta_sec)
            ref = oracle.eval_fitness(best[None], sp, cl.k_max, cl.n_max, cfg.p, cfg.speedup_floor, cur=cur,
                                      realloc=rf, active=jobs.active)[0]
            assert abs(fit - ref) <= REL_TOL * abs(ref)
            keep = oracle.eval_fitness(cur[None], sp, cl.k_max, cl.n_max, cfg.p, cfg.speedup_floor, cur=cur,
                                       realloc=rf, active=jobs.active)[0]
            assert fit >= keep * (1 - REL_TOL)        # never worse than keeping the allocation
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


def test_progress_bookkeeping():
    """Progress-coupled replay, host side only: work is fixed on a job's first round, progress
    integrates goodput over 60 s minus the restart delay, completion time is interpolated."""
    from paper_2008_12260_b200 import trace
    tr = trace.ProgressReplay()
    k = 40
    jobs, cur = tr.round_inputs(k)
    act = np.nonzero(jobs.active)[0]
    assert act.size >= 2
    a, b = int(act[0]), int(act[1])
    best = cur.copy()
    best[a, 0] = 2                       # job a (pending) starts: allocation changed -> 30 s delay
    g_kn = np.zeros(tr.cfg.num_jobs); g_1 = np.ones(tr.cfg.num_jobs)
    g_kn[a] = 3.0
    tr.advance(k, jobs, cur, best, g_kn, g_1)
    assert tr.work[a] == pytest.approx(tr.life[a] * 1.0) and np.isinf(tr.work[~(jobs.active > 0)]).all()
    assert tr.done[a] == pytest.approx(3.0 * 30.0) and tr.done[b] == 0.0
    # unchanged allocation next round: full 60 s
    jobs2, cur2 = tr.round_inputs(k + 1)
    assert np.array_equal(cur2[a], best[a])
    tr.advance(k + 1, jobs2, cur2, cur2.copy(), g_kn, g_1)
    assert tr.done[a] == pytest.approx(3.0 * 90.0)
    assert jobs2.phi[a] > tr.phi0[a] * 0.999           # phi follows the work done
    # finishing: give job a all its remaining work in half an interval
    rem = tr.work[a] - tr.done[a]
    g_kn[a] = rem / 30.0
    jobs3, cur3 = tr.round_inputs(k + 2)
    tr.advance(k + 2, jobs3, cur3, cur3.copy(), g_kn, g_1)
    assert tr.finish[a] == pytest.approx((k + 2) * 60.0 + 30.0)
    assert not tr.cur[a].any()
    jobs4, _ = tr.round_inputs(k + 3)
    assert jobs4.active[a] == 0
    assert tr.completion_times().size == 1


@pytest.mark.gpu
def test_progress_replay_on_gpu(oracle):
    import torch
    from paper_2008_12260_b200 import api, trace

    tr = trace.ProgressReplay(generations=20)
    cfg, cl = tr.cfg, tr.cluster
    s = api.scheduler_for(cfg, stream=torch.cuda.Stream().cuda_stream)
    seen = []

    def check(k, jobs, cur, best, fit, g_kn):
        if k % 15 == 3 and jobs.active.any():
            gp, _, _ = oracle.build_speedup_table(jobs, cl.node_capacity, cl.k_max, cl.n_max, cfg.grid_s,
                                                  want_argmax=False)
            K = np.minimum(best.sum(1), cl.k_max); N = np.minimum((best > 0).sum(1), cl.n_max)
            ref = gp[np.arange(cfg.num_jobs), K, N]
            on = jobs.active > 0
            np.testing.assert_allclose(g_kn[on], ref[on], rtol=REL_TOL, atol=0)
            seen.append(k)

    fits = trace.replay_progress(s, tr, torch, rounds=120, on_round=check)
    assert len(seen) >= 6
    jct = tr.completion_times()
    assert jct.size >= 3 and np.all(jct > 0) and np.all(np.isfinite(jct))
    assert np.all(tr.done[~np.isnan(tr.finish)] >= tr.work[~np.isnan(tr.finish)] * (1 - 1e-12))
    s.close()
