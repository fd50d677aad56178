"""Shared set-up for the tests: seeded inputs with the fair share filled in, and the
comparison rules of the parity tests."""
import numpy as np

from paper_2008_12260_b200 import synth

REL_TOL = 1e-5   # tables and fitness: relative tolerance of the CUDA path against the oracle


def with_fair_share(jobs, cluster, fair=None):
    from paper_2008_12260_b200.synth import Jobs  # noqa: F401
    cap = np.maximum(cluster.node_capacity.astype(np.int64), 0)
    n_act = int(jobs.active.sum())
    if fair is None:
        k = int(cap.sum()) // n_act if n_act > 0 else int(cap.sum())
        k = min(max(k, 1), cluster.k_max)
        fair = (k, -(-k // int(cap.max())))
    jobs.fair_k = np.full(jobs.num_jobs, fair[0], np.int32)
    jobs.fair_n = np.full(jobs.num_jobs, fair[1], np.int32)
    return jobs


def setup(cfg):
    cl = cfg.cluster()
    jobs = with_fair_share(cfg.jobs(), cl)
    return cl, jobs


def assert_close(got, ref, rel=REL_TOL, what=""):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    assert np.array_equal(ref == 0, got == 0), what + ": zero pattern differs"
    nz = ref != 0
    if nz.any():
        err = np.abs(got[nz] - ref[nz]) / np.abs(ref[nz])
        assert err.max() <= rel, "%s: max relative error %.3g > %.1g" % (what, err.max(), rel)


def check_table(oracle, jobs, grid_s, gp_gpu, sp_gpu, am_gpu, gp_ref, sp_ref, am_ref):
    """1e-5 relative on goodput and speedup; where the argmax differs, the oracle's goodput
    at the GPU's (m, s) must be within 1e-5 of the oracle's optimum."""
    assert_close(gp_gpu, gp_ref, what="goodput")
    assert_close(sp_gpu, sp_ref, what="speedup")
    assert np.array_equal(am_gpu == 0xFFFF, am_ref == 0xFFFF)
    diff = np.argwhere(am_gpu != am_ref)
    for j, K, N in diff:
        i, s = divmod(int(am_gpu[j, K, N]), grid_s)
        par = [float(getattr(jobs, f)[j]) for f in synth.JOB_F32_FIELDS]
        g, ok = oracle.goodput(*par, int(K), int(N), int(jobs.m_grid[j, i]), s)
        assert ok, (j, K, N, i, s)
        assert g >= gp_ref[j, K, N] * (1 - REL_TOL), (j, K, N, g, gp_ref[j, K, N])
    return len(diff)


def feasible(A, cap, k_cap, n_max):
    A = A.astype(np.int64)
    occ = A > 0
    dist = occ.sum(1) >= 2
    return bool((A >= 0).all() and (A.sum(0) <= cap).all() and (A.sum(1) <= k_cap).all()
                and (occ.sum(1) <= n_max).all() and ((occ & dist[:, None]).sum(0) <= 1).all())
