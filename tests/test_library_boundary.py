"""CPU checks of the boundary: the shared library loads, exports every function the
header declares, and the host-side helpers agree with the oracle."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "polluxsched.h")


def _declared():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"^\s*(?:const\s+)?(?:int|int64_t|char|float)\s*\*?\s*(\w+)\s*\(", text, flags=re.M)
    return sorted(set(names))


@pytest.fixture(scope="module")
def lib():
    from paper_2008_12260_b200 import build
    return ctypes.CDLL(build.build())


def test_header_declares_the_five_entry_points():
    names = _declared()
    for n in ("sched_init", "build_speedup_table", "eval_fitness", "ga_generation", "schedule_round"):
        assert n in names


def test_library_exports_every_declared_symbol(lib):
    names = _declared()
    assert len(names) >= 16
    for n in names:
        assert hasattr(lib, n), n


def test_binding_names_match_header():
    from paper_2008_12260_b200 import api
    assert sorted(api.EXPORTS) == _declared()
    for n in ("build_speedup_table", "eval_fitness", "ga_generation", "schedule_round",
              "repair_population", "init_population", "compute_realloc_factor",
              "schedule_round_host", "eval_fitness_host"):
        assert hasattr(api.Scheduler, n)


def test_config_struct_layout():
    from paper_2008_12260_b200 import api
    assert ctypes.sizeof(api.SchedConfig) == 64
    assert api.SchedConfig.seed.offset == 56
    assert ctypes.sizeof(api.SchedJobs) == 17 * ctypes.sizeof(ctypes.c_void_p)


def test_init_rejects_bad_arguments_without_a_gpu(lib):
    from paper_2008_12260_b200 import api
    lib.sched_last_error.restype = ctypes.c_char_p
    ctx = ctypes.c_void_p()
    cap = np.array([4, 4], np.int16)
    good = dict(num_nodes=2, num_jobs=3, k_max=8, n_max=2, grid_m=8, grid_s=4, population=4, p=-1.0,
                delta_sec=30.0, speedup_floor=1e-3, thr_mutate=0, thr_init=0, num_elite=1, seed=1)
    assert lib.sched_init(None, cap.ctypes.data, None, ctypes.byref(ctx)) == -1
    for bad, code in (dict(num_nodes=0), -2), (dict(num_nodes=100000), -6), (dict(grid_m=4096, grid_s=32), -6), \
                     (dict(num_elite=9), -2), (dict(delta_sec=-1.0), -2), (dict(population=0), -2), \
                     (dict(k_max=5000), -6):
        cfg = api.SchedConfig(**{**good, **bad})
        rc = lib.sched_init(ctypes.byref(cfg), ctypes.c_void_p(cap.ctypes.data), None, ctypes.byref(ctx))
        assert rc == code, (bad, rc)
        assert not ctx.value
        assert lib.sched_last_error(None)
    assert lib.sched_destroy(None) == 0


def test_fair_share_helper_matches_oracle(oracle):
    from paper_2008_12260_b200 import api
    rng = np.random.default_rng(0)
    for _ in range(200):
        cap = rng.integers(0, 9, rng.integers(1, 40)).astype(np.int16)
        if cap.max() <= 0:
            continue
        n_act = int(rng.integers(0, 300))
        k_max = min(int(cap.sum()), 64)
        assert api.fair_share(cap, n_act, k_max) == oracle.fair_share(cap, n_act, k_max)


def test_fair_share_raw_abi_errors(lib):
    fk, fn = ctypes.c_int32(-7), ctypes.c_int32(-7)
    cap = np.array([4, 0, 8, -3], np.int16)
    f = lib.sched_fair_share
    f.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                  ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32)]
    assert f(cap.ctypes.data, 4, 5, 64, ctypes.byref(fk), ctypes.byref(fn)) == 0
    assert (fk.value, fn.value) == (2, 1)            # 12 GPUs over 5 jobs; the negative node counts as empty
    assert f(cap.ctypes.data, 4, 1, 64, ctypes.byref(fk), ctypes.byref(fn)) == 0
    assert (fk.value, fn.value) == (12, 2)           # ceil(12 / largest node 8)
    assert f(cap.ctypes.data, 4, 1, 5, ctypes.byref(fk), ctypes.byref(fn)) == 0 and fk.value == 5
    assert f(cap.ctypes.data, 4, 100, 64, ctypes.byref(fk), ctypes.byref(fn)) == 0 and (fk.value, fn.value) == (1, 1)
    assert f(None, 4, 5, 64, ctypes.byref(fk), ctypes.byref(fn)) == -1
    assert f(cap.ctypes.data, 0, 5, 64, ctypes.byref(fk), ctypes.byref(fn)) == -1
    assert f(cap.ctypes.data, 4, 5, 0, ctypes.byref(fk), ctypes.byref(fn)) == -1
    empty = np.zeros(3, np.int16)
    assert f(empty.ctypes.data, 3, 5, 64, ctypes.byref(fk), ctypes.byref(fn)) == -2


def test_reference_arm_inputs_do_not_load_the_product_library():
    """bench.py --impl reference times the oracle; preparing its inputs must not even import the
    binding (which would dlopen the CUDA library)."""
    import subprocess
    import sys
    code = ("import sys; sys.argv=['bench.py']; import bench, oracle; "
            "bench.large_inputs(0, oracle.fair_share); "
            "assert 'paper_2008_12260_b200.api' not in sys.modules; "
            "assert 'libpolluxsched' not in open('/proc/self/maps').read(); print('ok')")
    out = subprocess.run([sys.executable, "-c", code], cwd=ROOT, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and "ok" in out.stdout, out.stderr
