"""ctypes front end of the CPU oracle (test infrastructure, not part of the product).

Only the tests, the smoke check and the benchmark's CPU-baseline leg import this
package.  It compiles `polluxsched_oracle.c` with gcc on first use and exposes thin
numpy wrappers; all arithmetic lives in the C file.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "polluxsched_oracle.c")
_SO = os.path.join(_HERE, "liboracle.so")
_lib = None

SLOT_SELECT, SLOT_XOVER, SLOT_MUTATE, SLOT_REPAIR_INTF, SLOT_REPAIR_CAP, SLOT_INIT = range(6)
GEN_INIT = 0xFFFFFFFF


def build(force: bool = False) -> str:
    """Compile the oracle into oracle/liboracle.so (no-op when up to date)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fPIC",
                               "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_efficiency.restype = C.c_double
        _lib.oracle_efficiency.argtypes = [C.c_double] * 3
        _lib.oracle_t_grad.restype = C.c_double
        _lib.oracle_t_grad.argtypes = [C.c_double] * 3
        _lib.oracle_t_sync.restype = C.c_double
        _lib.oracle_t_sync.argtypes = [C.c_double] * 4 + [C.c_int] * 2
        _lib.oracle_t_iter.restype = C.c_double
        _lib.oracle_t_iter.argtypes = [C.c_double] * 3 + [C.c_int]
        _lib.oracle_goodput.restype = C.c_double
        _lib.oracle_goodput.argtypes = [C.c_double] * 10 + [C.c_int] * 4 + [C.c_void_p]
        _lib.oracle_num_threads.restype = C.c_int
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dtype):
    return None if a is None else np.ascontiguousarray(a, dtype=dtype)


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def philox4x32_10(ctr, key):
    ctr = _c(ctr, np.uint32)
    key = _c(key, np.uint32)
    out = np.empty(4, dtype=np.uint32)
    lib().oracle_philox4x32_10(_p(ctr), _p(key), _p(out))
    return out


def draw(seed, rnd, idx, cand, gen, slot):
    out = np.empty(4, dtype=np.uint32)
    lib().oracle_draw(C.c_uint64(seed), C.c_uint32(rnd), C.c_uint32(idx), C.c_uint32(cand),
                      C.c_uint32(gen), C.c_uint32(slot), _p(out))
    return out


def efficiency(phi, m0, M):
    return float(lib().oracle_efficiency(phi, m0, M))


def t_grad(alpha, beta, m):
    return float(lib().oracle_t_grad(alpha, beta, m))


def t_sync(alpha_local, beta_local, alpha_node, beta_node, K, N):
    return float(lib().oracle_t_sync(alpha_local, beta_local, alpha_node, beta_node, K, N))


def t_iter(tg, ts, gamma, s):
    return float(lib().oracle_t_iter(tg, ts, gamma, s))


def goodput(alpha_grad, beta_grad, alpha_local, beta_local, alpha_node, beta_node, gamma, phi,
            m0, m_max_total, K, N, m, s):
    """Returns (goodput, feasible)."""
    ok = C.c_int(0)
    g = lib().oracle_goodput(alpha_grad, beta_grad, alpha_local, beta_local, alpha_node, beta_node,
                             gamma, phi, m0, m_max_total, K, N, m, s, C.byref(ok))
    return float(g), bool(ok.value)


def fair_share(node_capacity, num_active, k_max):
    cap = _c(node_capacity, np.int16)
    fk, fn = C.c_int32(0), C.c_int32(0)
    rc = lib().oracle_fair_share(cap.shape[0], _p(cap), int(num_active), int(k_max),
                                 C.byref(fk), C.byref(fn))
    if rc != 0:
        raise ValueError("oracle_fair_share: bad arguments")
    return fk.value, fn.value


_F32_FIELDS = ("alpha_grad", "beta_grad", "alpha_local", "beta_local", "alpha_node", "beta_node",
               "gamma", "phi", "m0", "m_max_total")


def _job_args(jobs):
    arrs = [_c(getattr(jobs, f), np.float32) for f in _F32_FIELDS]
    return arrs


def build_speedup_table(jobs, node_capacity, k_max, n_max, grid_s, want_argmax=True):
    """jobs: any object with the fp32 fields, m_grid [J][Gm], fair_k, fair_n.
    Returns (goodput f64 [J][KD][ND], speedup f64, argmax u16 or None)."""
    cap = _c(node_capacity, np.int16)
    fa = _job_args(jobs)
    mg = _c(jobs.m_grid, np.int32)
    fk = _c(jobs.fair_k, np.int32)
    fn = _c(jobs.fair_n, np.int32)
    J, Gm = mg.shape
    shape = (J, k_max + 1, n_max + 1)
    gp = np.zeros(shape, dtype=np.float64)
    sp = np.zeros(shape, dtype=np.float64)
    am = np.zeros(shape, dtype=np.uint16) if want_argmax else None
    rc = lib().oracle_build_speedup_table(
        J, cap.shape[0], _p(cap), int(k_max), int(n_max), int(Gm), int(grid_s),
        *[_p(a) for a in fa], _p(mg), _p(fk), _p(fn), _p(gp), _p(sp), _p(am))
    if rc != 0:
        raise ValueError("oracle_build_speedup_table: bad arguments")
    return gp, sp, am


def realloc_factor(age_sec, num_restarts, delta):
    a = _c(age_sec, np.float32)
    r = _c(num_restarts, np.int32)
    out = np.empty(a.shape[0], dtype=np.float64)
    lib().oracle_realloc_factor(a.shape[0], _p(a), _p(r), C.c_double(delta), _p(out))
    return out


def eval_fitness(pop, speedup, k_max, n_max, p, floor, cur=None, realloc=None, active=None):
    pop = _c(pop, np.int16)
    P, J, N = pop.shape
    sp = _c(speedup, np.float64)
    assert sp.shape == (J, k_max + 1, n_max + 1)
    cur = _c(cur, np.int16)
    rf = _c(realloc, np.float64)
    act = _c(active, np.uint8)
    out = np.empty(P, dtype=np.float64)
    rc = lib().oracle_eval_fitness(P, J, N, int(k_max), int(n_max), _p(pop), _p(sp), _p(cur), _p(rf),
                                   _p(act), C.c_double(p), C.c_double(floor), _p(out))
    if rc != 0:
        raise ValueError("oracle_eval_fitness: bad arguments")
    return out


def rank(fitness_f32):
    bits = _c(fitness_f32, np.float32).view(np.uint32)
    out = np.empty(bits.shape[0], dtype=np.int32)
    lib().oracle_rank(bits.shape[0], _p(bits), _p(out))
    return out


def mutate_row(row, w, thr):
    row = np.array(row, dtype=np.int16)
    w = _c(w, np.uint32)
    lib().oracle_mutate_row(_p(row), row.shape[0], _p(w), C.c_uint32(thr))
    return row


def repair_with_offsets(A, node_capacity, k_cap, k_max, n_max, intf_offset, cap_offset, active=None):
    A = np.array(A, dtype=np.int16)
    J, N = A.shape
    cap = _c(node_capacity, np.int16)
    kc = _c(k_cap, np.int32)
    oi = _c(intf_offset, np.uint32)
    oc = _c(cap_offset, np.uint32)
    act = _c(active, np.uint8)
    rc = lib().oracle_repair_with_offsets(J, N, _p(cap), _p(kc), int(k_max), int(n_max), _p(act),
                                          _p(A), _p(oi), _p(oc))
    if rc != 0:
        raise ValueError("oracle_repair_with_offsets: bad arguments")
    return A


def repair(A, node_capacity, k_cap, k_max, n_max, seed, rnd, cand, gen, active=None):
    A = np.array(A, dtype=np.int16)
    J, N = A.shape
    cap = _c(node_capacity, np.int16)
    kc = _c(k_cap, np.int32)
    act = _c(active, np.uint8)
    rc = lib().oracle_repair(J, N, _p(cap), _p(kc), int(k_max), int(n_max), _p(act), _p(A),
                             C.c_uint64(seed), C.c_uint32(rnd), C.c_uint32(cand), C.c_uint32(gen))
    if rc != 0:
        raise ValueError("oracle_repair: bad arguments")
    return A


def ga_generation(pop_in, fitness_f32, node_capacity, k_cap, k_max, n_max, num_elite, thr_mutate,
                  seed, rnd, gen, active=None):
    pop = _c(pop_in, np.int16)
    P, J, N = pop.shape
    bits = _c(fitness_f32, np.float32).view(np.uint32)
    cap = _c(node_capacity, np.int16)
    kc = _c(k_cap, np.int32)
    act = _c(active, np.uint8)
    out = np.empty_like(pop)
    rc = lib().oracle_ga_generation(P, J, N, _p(cap), _p(kc), int(k_max), int(n_max), _p(act),
                                    int(num_elite), C.c_uint32(thr_mutate), C.c_uint64(seed),
                                    C.c_uint32(rnd), C.c_uint32(gen), _p(pop), _p(bits), _p(out))
    if rc != 0:
        raise ValueError("oracle_ga_generation: bad arguments")
    return out


def init_population(P, cur, J, node_capacity, k_cap, k_max, n_max, thr_init, seed, rnd, active=None):
    cap = _c(node_capacity, np.int16)
    N = cap.shape[0]
    kc = _c(k_cap, np.int32)
    act = _c(active, np.uint8)
    cur = _c(cur, np.int16)
    out = np.empty((P, J, N), dtype=np.int16)
    rc = lib().oracle_init_population(P, J, N, _p(cap), _p(kc), int(k_max), int(n_max), _p(act),
                                      C.c_uint32(thr_init), C.c_uint64(seed), C.c_uint32(rnd),
                                      _p(cur), _p(out))
    if rc != 0:
        raise ValueError("oracle_init_population: bad arguments")
    return out


def schedule_round(jobs, node_capacity, k_max, n_max, grid_s, P, p, delta, floor, num_elite,
                   thr_mutate, thr_init, seed, rnd, generations, cur):
    cap = _c(node_capacity, np.int16)
    N = cap.shape[0]
    fa = _job_args(jobs)
    mg = _c(jobs.m_grid, np.int32)
    J, Gm = mg.shape
    kc = _c(jobs.k_cap, np.int32)
    fk = _c(jobs.fair_k, np.int32)
    fn = _c(jobs.fair_n, np.int32)
    age = _c(jobs.age_sec, np.float32)
    nr = _c(jobs.num_restarts, np.int32)
    act = _c(jobs.active, np.uint8)
    cur = _c(cur, np.int16)
    best = np.empty((J, N), dtype=np.int16)
    bf = C.c_double(0.0)
    rc = lib().oracle_schedule_round(
        int(P), J, N, _p(cap), int(k_max), int(n_max), int(Gm), int(grid_s),
        *[_p(a) for a in fa], _p(mg), _p(kc), _p(fk), _p(fn), _p(age), _p(nr), _p(act),
        C.c_double(p), C.c_double(delta), C.c_double(floor), int(num_elite), C.c_uint32(thr_mutate),
        C.c_uint32(thr_init), C.c_uint64(seed), C.c_uint32(rnd), int(generations), _p(cur), _p(best),
        C.byref(bf))
    if rc != 0:
        raise ValueError("oracle_schedule_round: bad arguments")
    return best, bf.value


def autoscale_targets(goodput_f32, k_max, n_max, gpus_per_node, cur_nodes, U, L):
    g = _c(goodput_f32, np.float32)
    cn = _c(cur_nodes, np.int32)
    out = np.empty(cn.shape[0], dtype=np.int32)
    rc = lib().oracle_autoscale_targets(cn.shape[0], int(k_max), int(n_max), int(gpus_per_node), _p(g), _p(cn),
                                        C.c_float(U), C.c_float(L), _p(out))
    if rc != 0:
        raise ValueError("oracle_autoscale_targets: bad arguments")
    return out


def build_speedup_table_msample(jobs, node_capacity, k_max, n_max, m_samples, m_max_gpu, adaptive=None,
                                want_argmax=True):
    """Tables from the paper's total-batch sampling search (Sec. 4.3) and, for jobs with
    adaptive == 0, the fixed-batch rule of Sec. 4.2."""
    cap = _c(node_capacity, np.int16)
    fa = _job_args(jobs)
    ms = _c(m_samples, np.int32)
    mm = _c(m_max_gpu, np.int32)
    ad = _c(adaptive, np.uint8)
    fk = _c(jobs.fair_k, np.int32)
    fn = _c(jobs.fair_n, np.int32)
    J, G = ms.shape
    shape = (J, k_max + 1, n_max + 1)
    gp = np.zeros(shape, dtype=np.float64)
    sp = np.zeros(shape, dtype=np.float64)
    am = np.zeros(shape, dtype=np.uint16) if want_argmax else None
    rc = lib().oracle_build_speedup_table_msample(
        J, cap.shape[0], _p(cap), int(k_max), int(n_max), int(G), *[_p(a) for a in fa], _p(ms), _p(mm), _p(ad),
        _p(fk), _p(fn), _p(gp), _p(sp), _p(am))
    if rc != 0:
        raise ValueError("oracle_build_speedup_table_msample: bad arguments")
    return gp, sp, am


def set_threads(n: int):
    """Threads of the oracle's parallel loops (1 = single core; 0 = all)."""
    lib().oracle_set_threads(int(n))


def t_sync_rack(alpha_local, beta_local, alpha_node, beta_node, alpha_rack, beta_rack, K, N, R):
    f = lib().oracle_t_sync_rack
    f.restype = C.c_double
    f.argtypes = [C.c_double] * 6 + [C.c_int] * 3
    return float(f(alpha_local, beta_local, alpha_node, beta_node, alpha_rack, beta_rack, K, N, R))


def goodput_rack(alpha_grad, beta_grad, alpha_local, beta_local, alpha_node, beta_node, alpha_rack, beta_rack,
                 gamma, phi, m0, m_max_total, K, N, R, m, s):
    """Returns (goodput, feasible) with the three-class T_sync."""
    f = lib().oracle_goodput_rack
    f.restype = C.c_double
    f.argtypes = [C.c_double] * 12 + [C.c_int] * 5 + [C.c_void_p]
    ok = C.c_int(0)
    g = f(alpha_grad, beta_grad, alpha_local, beta_local, alpha_node, beta_node, alpha_rack, beta_rack, gamma, phi,
          m0, m_max_total, K, N, R, m, s, C.byref(ok))
    return float(g), bool(ok.value)


def build_speedup_table_rack(jobs, node_capacity, k_max, n_max, grid_s, want_argmax=True):
    """Third-class tables (allocations that span racks); jobs also carries alpha_rack, beta_rack."""
    cap = _c(node_capacity, np.int16)
    fa = _job_args(jobs)
    ar = _c(jobs.alpha_rack, np.float32)
    br = _c(jobs.beta_rack, np.float32)
    mg = _c(jobs.m_grid, np.int32)
    fk = _c(jobs.fair_k, np.int32)
    fn = _c(jobs.fair_n, np.int32)
    J, Gm = mg.shape
    shape = (J, k_max + 1, n_max + 1)
    gp = np.zeros(shape, dtype=np.float64)
    sp = np.zeros(shape, dtype=np.float64)
    am = np.zeros(shape, dtype=np.uint16) if want_argmax else None
    rc = lib().oracle_build_speedup_table_rack(
        J, cap.shape[0], _p(cap), int(k_max), int(n_max), int(Gm), int(grid_s),
        *[_p(a) for a in fa[:6]], _p(ar), _p(br), *[_p(a) for a in fa[6:]], _p(mg), _p(fk), _p(fn), _p(gp), _p(sp),
        _p(am))
    if rc != 0:
        raise ValueError("oracle_build_speedup_table_rack: bad arguments")
    return gp, sp, am


def eval_fitness_racks(pop, speedup, speedup_rack, node_rack, k_max, n_max, p, floor, cur=None, realloc=None,
                       active=None):
    pop = _c(pop, np.int16)
    P, J, N = pop.shape
    sp = _c(speedup, np.float64)
    spr = _c(speedup_rack, np.float64)
    assert sp.shape == (J, k_max + 1, n_max + 1) and spr.shape == sp.shape
    rack = _c(node_rack, np.int16)
    assert rack.shape == (N,)
    cur = _c(cur, np.int16)
    rf = _c(realloc, np.float64)
    act = _c(active, np.uint8)
    out = np.empty(P, dtype=np.float64)
    rc = lib().oracle_eval_fitness_racks(P, J, N, int(k_max), int(n_max), _p(pop), _p(sp), _p(spr), _p(rack), _p(cur),
                                         _p(rf), _p(act), C.c_double(p), C.c_double(floor), _p(out))
    if rc != 0:
        raise ValueError("oracle_eval_fitness_racks: bad arguments")
    return out
