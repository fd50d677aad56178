"""Thin ctypes binding over libpolluxsched.so: same names as the C ABI, argument
marshalling only.  PyTorch tensors supply device memory and the CUDA stream; every step
of the method runs in the library's kernels.  There is no fallback: if the compiled
library is missing, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# POLLUXSCHED_LIB selects another build of the library (e.g. libpolluxsched_checked.so)
LIB_PATH = os.environ.get("POLLUXSCHED_LIB") or os.path.join(_HERE, "libpolluxsched.so")

SCHED_OK = 0
ERRORS = {-1: "INVALID_ARG", -2: "BAD_CONFIG", -3: "CUDA", -4: "TIMEOUT", -5: "NOT_FINITE", -6: "TOO_LARGE"}

EXPORTS = (
    "sched_init", "sched_fair_share", "sched_destroy", "sched_last_error", "sched_sync_status", "sched_launch_count",
    "build_speedup_table", "build_speedup_table_msample", "sched_set_racks", "build_speedup_table_rack", "eval_fitness_racks", "fit_throughput_model", "compute_realloc_factor", "autoscale_targets", "eval_fitness", "repair_population",
    "init_population", "ga_generation", "ga_generation_shard", "schedule_round", "schedule_round_host",
    "sched_get_population", "sched_get_round_tables", "sched_round_speedup_table", "eval_fitness_host",
    "sched_set_kernel_timing", "sched_num_kernel_kinds", "sched_kernel_kind_name",
    "sched_read_kernel_timing", "sched_measure_peaks", "sched_set_graphs", "sched_set_store_budget", "sched_store_moves", "eval_fitness_noalloc", "eval_fitness_noalloc_last_error",
)


class SchedConfig(C.Structure):
    _fields_ = [
        ("num_nodes", C.c_int32), ("num_jobs", C.c_int32), ("k_max", C.c_int32), ("n_max", C.c_int32),
        ("grid_m", C.c_int32), ("grid_s", C.c_int32), ("population", C.c_int32),
        ("p", C.c_float), ("delta_sec", C.c_float), ("speedup_floor", C.c_float),
        ("thr_mutate", C.c_uint32), ("thr_init", C.c_uint32), ("num_elite", C.c_int32),
        ("seed", C.c_uint64),
    ]


_JOB_FIELDS = ("alpha_grad", "beta_grad", "alpha_local", "beta_local", "alpha_node", "beta_node",
               "gamma", "phi", "m0", "m_max_total", "m_grid", "k_cap", "fair_k", "fair_n",
               "age_sec", "num_restarts", "active")


class SchedJobs(C.Structure):
    _fields_ = [(name, C.c_void_p) for name in _JOB_FIELDS]


class SchedError(RuntimeError):
    def __init__(self, code, message):
        super().__init__("%s (%d): %s" % (ERRORS.get(code, "?"), code, message))
        self.code = code


def load_library(path: str = LIB_PATH):
    if not os.path.exists(path):
        raise ImportError(
            "%s not found: build it with `python -m paper_2008_12260_b200.build` "
            "(there is no CPU fallback)" % path)
    lib = C.CDLL(path)
    vp, i32, u32, f32 = C.c_void_p, C.c_int32, C.c_uint32, C.c_float
    lib.sched_init.argtypes = [C.POINTER(SchedConfig), vp, vp, C.POINTER(vp)]
    lib.sched_destroy.argtypes = [vp]
    lib.sched_fair_share.argtypes = [vp, i32, i32, i32, C.POINTER(i32), C.POINTER(i32)]
    lib.sched_last_error.argtypes = [vp]
    lib.sched_last_error.restype = C.c_char_p
    lib.sched_sync_status.argtypes = [vp]
    lib.sched_launch_count.argtypes = [vp]
    lib.sched_launch_count.restype = C.c_int64
    lib.build_speedup_table.argtypes = [vp, C.POINTER(SchedJobs), vp, vp, vp]
    lib.build_speedup_table_msample.argtypes = [vp, C.POINTER(SchedJobs), vp, i32, vp, vp, vp, vp, vp]
    lib.sched_set_racks.argtypes = [vp, vp, vp, vp]
    lib.build_speedup_table_rack.argtypes = [vp, C.POINTER(SchedJobs), vp, vp, vp, vp, vp]
    lib.eval_fitness_racks.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp, f32, vp]
    lib.fit_throughput_model.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, vp]
    lib.compute_realloc_factor.argtypes = [vp, C.POINTER(SchedJobs), vp]
    lib.autoscale_targets.argtypes = [vp, vp, vp, i32, f32, f32, vp]
    lib.eval_fitness.argtypes = [vp, vp, i32, vp, vp, vp, vp, f32, vp]
    lib.repair_population.argtypes = [vp, C.POINTER(SchedJobs), vp, i32, u32, u32, u32]
    lib.init_population.argtypes = [vp, C.POINTER(SchedJobs), vp, u32, vp]
    lib.ga_generation.argtypes = [vp, C.POINTER(SchedJobs), vp, vp, vp, u32, u32]
    lib.ga_generation_shard.argtypes = [vp, C.POINTER(SchedJobs), vp, vp, i32, i32, vp, u32, u32]
    lib.schedule_round.argtypes = [vp, C.POINTER(SchedJobs), vp, u32, i32, vp, vp]
    lib.schedule_round_host.argtypes = [vp, C.POINTER(SchedJobs), vp, u32, i32, vp, vp]
    lib.sched_get_population.argtypes = [vp, vp, vp]
    lib.sched_get_round_tables.argtypes = [vp, vp, vp]
    lib.sched_round_speedup_table.argtypes = [vp]
    lib.sched_round_speedup_table.restype = vp
    lib.eval_fitness_host.argtypes = [vp, vp, i32, vp, vp, vp, vp, f32, vp]
    lib.sched_set_kernel_timing.argtypes = [vp, i32]
    lib.sched_set_graphs.argtypes = [vp, i32]
    lib.sched_measure_peaks.argtypes = [vp, vp, C.c_uint64, i32, C.POINTER(C.c_double), C.POINTER(C.c_double),
                                        C.POINTER(C.c_double)]
    lib.sched_set_store_budget.argtypes = [vp, C.c_uint64]
    lib.sched_store_moves.argtypes = [vp]
    lib.sched_store_moves.restype = C.c_int64
    lib.sched_num_kernel_kinds.argtypes = []
    lib.sched_kernel_kind_name.argtypes = [i32]
    lib.sched_kernel_kind_name.restype = C.c_char_p
    lib.sched_read_kernel_timing.argtypes = [vp, vp, vp]
    lib.eval_fitness_noalloc.argtypes = [vp, i32, i32, i32, i32, i32, vp, vp, vp, vp, f32, f32, vp, vp]
    lib.eval_fitness_noalloc_last_error.argtypes = []
    lib.eval_fitness_noalloc_last_error.restype = C.c_char_p
    for name in EXPORTS:
        if getattr(lib, name).restype is C.c_int:
            getattr(lib, name).restype = C.c_int
    return lib


_lib = load_library()


def _ptr(t):
    """device/host address of a torch tensor or numpy array (None -> NULL)"""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        assert t.flags["C_CONTIGUOUS"]
        return t.ctypes.data
    assert t.is_contiguous()
    return t.data_ptr()


def fair_share(node_capacity, num_active: int, k_max: int):
    """(K_f, N_f) of the fair allocation a_f of Eq. 15 from sched_fair_share (host-only)."""
    cap = np.ascontiguousarray(node_capacity, dtype=np.int16)
    fk, fn = C.c_int32(0), C.c_int32(0)
    rc = _lib.sched_fair_share(cap.ctypes.data, cap.shape[0], int(num_active), int(k_max), C.byref(fk), C.byref(fn))
    if rc != SCHED_OK:
        raise SchedError(rc, _lib.sched_last_error(None).decode())
    return fk.value, fn.value


class DeviceJobs:
    """Per-job inputs as torch tensors on the device, plus the sched_jobs struct over them."""

    def __init__(self, jobs, device, torch):
        self.tensors = {}
        self.struct = SchedJobs()
        for name in _JOB_FIELDS:
            arr = getattr(jobs, name, None)
            if arr is None:
                setattr(self.struct, name, None)
                continue
            t = torch.from_numpy(np.ascontiguousarray(arr)).to(device)
            self.tensors[name] = t
            setattr(self.struct, name, t.data_ptr())


class HostJobs:
    """Per-job inputs as pinned host tensors (for the *_host entry points)."""

    def __init__(self, jobs, torch, pin=True):
        self.tensors = {}
        self.struct = SchedJobs()
        self.nbytes = 0
        for name in _JOB_FIELDS:
            arr = getattr(jobs, name, None)
            if arr is None:
                setattr(self.struct, name, None)
                continue
            t = torch.from_numpy(np.ascontiguousarray(arr).copy())
            if pin:
                t = t.pin_memory()
            self.tensors[name] = t
            self.nbytes += t.numel() * t.element_size()
            setattr(self.struct, name, t.data_ptr())


class Scheduler:
    """Owns one sched_ctx.  Methods mirror the C entry points one to one."""

    def __init__(self, *, node_capacity, num_jobs, grid_m, grid_s, population, p=-1.0, delta_sec=30.0,
                 speedup_floor=1e-3, thr_mutate=0, thr_init=0, num_elite=0, seed=0, k_max=None,
                 n_max=None, stream=None):
        cap = np.ascontiguousarray(node_capacity, dtype=np.int16)
        total = int(np.maximum(cap.astype(np.int64), 0).sum())
        self.cfg = SchedConfig(
            num_nodes=cap.shape[0], num_jobs=num_jobs,
            k_max=min(total, 64) if k_max is None else k_max,
            n_max=min(cap.shape[0], 64) if n_max is None else n_max,
            grid_m=grid_m, grid_s=grid_s, population=population, p=p, delta_sec=delta_sec,
            speedup_floor=speedup_floor, thr_mutate=thr_mutate, thr_init=thr_init,
            num_elite=num_elite, seed=seed)
        self.node_capacity = cap
        self._ctx = C.c_void_p()
        rc = _lib.sched_init(C.byref(self.cfg), cap.ctypes.data, stream, C.byref(self._ctx))
        if rc != SCHED_OK:
            raise SchedError(rc, _lib.sched_last_error(None).decode())

    # -- plumbing -------------------------------------------------------------------------
    @property
    def table_shape(self):
        return (self.cfg.num_jobs, self.cfg.k_max + 1, self.cfg.n_max + 1)

    def _check(self, rc):
        if rc != SCHED_OK:
            raise SchedError(rc, _lib.sched_last_error(self._ctx).decode())

    def close(self):
        if self._ctx:
            _lib.sched_destroy(self._ctx)
            self._ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def sync_status(self):
        self._check(_lib.sched_sync_status(self._ctx))

    def launch_count(self) -> int:
        return int(_lib.sched_launch_count(self._ctx))

    def set_kernel_timing(self, enable: bool):
        self._check(_lib.sched_set_kernel_timing(self._ctx, 1 if enable else 0))

    def set_graphs(self, enable: bool):
        self._check(_lib.sched_set_graphs(self._ctx, 1 if enable else 0))

    def measure_peaks(self, buffer=None, reps: int = 5):
        """(fp32 lane-ops/s, special-function ops/s, read-only stream bytes/s over `buffer`)"""
        a, b, c = C.c_double(0), C.c_double(0), C.c_double(0)
        nbytes = 0 if buffer is None else buffer.numel() * buffer.element_size()
        self._check(_lib.sched_measure_peaks(self._ctx, _ptr(buffer), nbytes, reps, C.byref(a), C.byref(b), C.byref(c)))
        return a.value, b.value, c.value

    def set_store_budget(self, nbytes: int):
        self._check(_lib.sched_set_store_budget(self._ctx, int(nbytes)))

    def store_moves(self) -> int:
        return int(_lib.sched_store_moves(self._ctx))

    def read_kernel_timing(self):
        """{kernel class: (total ms, timed launches)} since the previous read-out"""
        n = _lib.sched_num_kernel_kinds()
        ms = np.zeros(n, np.float32)
        cnt = np.zeros(n, np.int64)
        self._check(_lib.sched_read_kernel_timing(self._ctx, ms.ctypes.data, cnt.ctypes.data))
        return {_lib.sched_kernel_kind_name(k).decode(): (float(ms[k]), int(cnt[k])) for k in range(n)}

    # -- entry points ---------------------------------------------------------------------
    def build_speedup_table(self, jobs, goodput, speedup, argmax=None):
        self._check(_lib.build_speedup_table(self._ctx, C.byref(jobs.struct), _ptr(goodput),
                                             _ptr(speedup), _ptr(argmax)))

    def build_speedup_table_msample(self, jobs, m_samples, m_max_gpu, goodput, speedup, argmax=None, adaptive=None):
        self._check(_lib.build_speedup_table_msample(self._ctx, C.byref(jobs.struct), _ptr(m_samples),
                                                     m_samples.shape[1], _ptr(m_max_gpu), _ptr(adaptive),
                                                     _ptr(goodput), _ptr(speedup), _ptr(argmax)))

    def set_racks(self, node_rack, alpha_rack=None, beta_rack=None):
        rack = None if node_rack is None else np.ascontiguousarray(node_rack, dtype=np.int16)
        self._racks = (alpha_rack, beta_rack)          # keep the device arrays alive
        self._check(_lib.sched_set_racks(self._ctx, _ptr(rack), _ptr(alpha_rack), _ptr(beta_rack)))

    def build_speedup_table_rack(self, jobs, alpha_rack, beta_rack, goodput, speedup, argmax=None):
        self._check(_lib.build_speedup_table_rack(self._ctx, C.byref(jobs.struct), _ptr(alpha_rack), _ptr(beta_rack),
                                                  _ptr(goodput), _ptr(speedup), _ptr(argmax)))

    def eval_fitness_racks(self, pop, speedup, speedup_rack, fitness, *, p, cur=None, realloc_factor=None, active=None,
                           count=None):
        n = pop.shape[0] if count is None else count
        self._check(_lib.eval_fitness_racks(self._ctx, _ptr(pop), n, _ptr(speedup), _ptr(speedup_rack), _ptr(cur),
                                            _ptr(realloc_factor), _ptr(active), p, _ptr(fitness)))

    def fit_throughput_model(self, offset, k, n, m, s, t, theta0, theta_out, loss_out, *, frozen=None, max_iters=100):
        self._check(_lib.fit_throughput_model(self._ctx, theta0.shape[0], _ptr(offset), _ptr(k), _ptr(n), _ptr(m),
                                              _ptr(s), _ptr(t), _ptr(theta0), _ptr(frozen), max_iters,
                                              _ptr(theta_out), _ptr(loss_out)))

    def compute_realloc_factor(self, jobs, out):
        self._check(_lib.compute_realloc_factor(self._ctx, C.byref(jobs.struct), _ptr(out)))

    def autoscale_targets(self, goodput, cur_nodes, target_nodes, *, gpus_per_node, U=2.0 / 3.0, L=0.5):
        self._check(_lib.autoscale_targets(self._ctx, _ptr(goodput), _ptr(cur_nodes), gpus_per_node, U, L,
                                           _ptr(target_nodes)))

    def eval_fitness(self, pop, speedup, fitness, *, p, cur=None, realloc_factor=None, active=None,
                     count=None):
        n = pop.shape[0] if count is None else count
        self._check(_lib.eval_fitness(self._ctx, _ptr(pop), n, _ptr(speedup), _ptr(cur),
                                      _ptr(realloc_factor), _ptr(active), p, _ptr(fitness)))

    def repair_population(self, jobs, pop, *, round, generation, first_candidate=0, count=None):
        n = pop.shape[0] if count is None else count
        js = C.byref(jobs.struct) if jobs is not None else None
        self._check(_lib.repair_population(self._ctx, js, _ptr(pop), n, first_candidate, round, generation))

    def init_population(self, jobs, cur, pop_out, *, round):
        js = C.byref(jobs.struct) if jobs is not None else None
        self._check(_lib.init_population(self._ctx, js, _ptr(cur), round, _ptr(pop_out)))

    def ga_generation(self, jobs, pop_in, fitness_in, pop_out, *, round, generation):
        js = C.byref(jobs.struct) if jobs is not None else None
        self._check(_lib.ga_generation(self._ctx, js, _ptr(pop_in), _ptr(fitness_in), _ptr(pop_out),
                                       round, generation))

    def ga_generation_shard(self, jobs, pop_in, fitness_in, children, *, first_child, round, generation,
                            num_children=None):
        n = children.shape[0] if num_children is None else num_children
        js = C.byref(jobs.struct) if jobs is not None else None
        self._check(_lib.ga_generation_shard(self._ctx, js, _ptr(pop_in), _ptr(fitness_in), first_child, n,
                                             _ptr(children), round, generation))

    def schedule_round(self, jobs, cur, best, best_fitness, *, round, generations):
        self._check(_lib.schedule_round(self._ctx, C.byref(jobs.struct), _ptr(cur), round, generations,
                                        _ptr(best), _ptr(best_fitness)))

    def schedule_round_host(self, jobs, cur, best, best_fitness, *, round, generations):
        self._check(_lib.schedule_round_host(self._ctx, C.byref(jobs.struct), _ptr(cur), round,
                                             generations, _ptr(best), _ptr(best_fitness)))

    def get_population(self, pop_out=None, fitness_out=None):
        self._check(_lib.sched_get_population(self._ctx, _ptr(pop_out), _ptr(fitness_out)))

    def get_round_tables(self, goodput_out=None, speedup_out=None):
        self._check(_lib.sched_get_round_tables(self._ctx, _ptr(goodput_out), _ptr(speedup_out)))

    def eval_fitness_host(self, pop, speedup, fitness, *, p, cur=None, realloc_factor=None, active=None):
        self._check(_lib.eval_fitness_host(self._ctx, _ptr(pop), pop.shape[0], _ptr(speedup), _ptr(cur),
                                           _ptr(realloc_factor), _ptr(active), p, _ptr(fitness)))


def eval_fitness_noalloc(pop, speedup, fitness, *, k_max, n_max, p, speedup_floor, cur=None,
                         realloc_factor=None, active=None, stream=None, count=None):
    """Fitness of `pop` ([count][J][num_nodes] int16 on the device) without a context and
    without any device allocation inside the library: for processes whose allocator already
    owns the whole GPU, or loops that cannot take cudaMalloc's device-wide synchronisation.
    See the header for the fixed limits (count <= 2048, J <= 16384) and the sharing rules of
    its static scratch array."""
    n = pop.shape[0] if count is None else count
    rc = _lib.eval_fitness_noalloc(_ptr(pop), n, pop.shape[1], pop.shape[2], k_max, n_max, _ptr(speedup),
                                   _ptr(cur), _ptr(realloc_factor), _ptr(active), p, speedup_floor,
                                   _ptr(fitness), stream)
    if rc != SCHED_OK:
        raise SchedError(rc, _lib.eval_fitness_noalloc_last_error().decode())


def scheduler_for(cfg, jobs=None, stream=None, **overrides):
    """Scheduler for a synth.Config (sizes, knobs and thresholds taken from it)."""
    from . import synth

    cl = cfg.cluster()
    kw = dict(node_capacity=cl.node_capacity, num_jobs=cfg.num_jobs, grid_m=cfg.grid_m,
              grid_s=cfg.grid_s, population=cfg.population, p=cfg.p, delta_sec=cfg.delta_sec,
              speedup_floor=cfg.speedup_floor, thr_mutate=synth.prob_to_threshold(cfg.mutate_prob),
              thr_init=synth.prob_to_threshold(cfg.init_prob), num_elite=cfg.num_elite, seed=cfg.seed,
              stream=stream)
    kw.update(overrides)
    return Scheduler(**kw)
