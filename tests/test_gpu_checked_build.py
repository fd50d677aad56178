"""The range-checking build of the library (-DSCHED_CHECKED): kernels test the indices they
compute from data - row slots, node numbers, list positions - and report a violation through
the status word instead of touching memory.  The row-store rounds, the randomly drawn rounds and the operator
tests run once against it; their sync_status() calls raise if any check fired."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.gpu
def test_round_and_operator_tests_pass_on_the_checked_build():
    from paper_2008_12260_b200 import build
    lib = build.build(checked=True)
    assert os.path.exists(lib)
    env = dict(os.environ, POLLUXSCHED_LIB=lib)
    cmd = [sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", "-p", "no:cacheprovider",
           os.path.join(ROOT, "tests", "test_gpu_round_kernels.py"), os.path.join(ROOT, "tests", "test_gpu_ga.py"),
           os.path.join(ROOT, "tests", "test_gpu_round_fuzz.py")]
    out = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert out.returncode == 0, out.stdout[-3000:] + out.stderr[-2000:]
    assert " passed" in out.stdout


def test_checked_build_exports_the_same_symbols():
    import ctypes
    from paper_2008_12260_b200 import api, build
    lib = ctypes.CDLL(build.build(checked=True))
    for name in api.EXPORTS:
        assert hasattr(lib, name), name
