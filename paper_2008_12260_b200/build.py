"""Builds libpolluxsched.so in-tree with nvcc for sm_100a (cross-compiles without a GPU).

    python -m paper_2008_12260_b200.build [--force] [--verbose] [--checked]

--checked builds libpolluxsched_checked.so instead: the same library compiled with
-DSCHED_CHECKED, in which kernels range-test the indices they compute from data and report a
violation through the context's status word (see csrc/common.cuh).  Select it at run time with
the environment variable POLLUXSCHED_LIB.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(ROOT, "include")
LIB = os.path.join(HERE, "libpolluxsched.so")
LIB_CHECKED = os.path.join(HERE, "libpolluxsched_checked.so")

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "--shared", "-cudart", "static",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(INCLUDE, "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    lib = LIB_CHECKED if checked else LIB
    if not force and not _stale(lib):
        return lib
    from concurrent.futures import ThreadPoolExecutor

    nvcc = os.environ.get("NVCC", "nvcc")
    objdir = os.path.join(HERE, "_build")
    os.makedirs(objdir, exist_ok=True)
    common = [f for f in NVCC_FLAGS if f not in ("--shared", "-cudart", "static")]
    common += (["-Xptxas", "-v"] if verbose else []) + ["-I", INCLUDE, "-I", CSRC]
    common += ["-DSCHED_CHECKED"] if checked else []

    def compile_one(src):
        obj = os.path.join(objdir, os.path.basename(src) + ".%d%s.o" % (os.getpid(), "c" if checked else ""))
        res = subprocess.run([nvcc] + common + ["-c", "-o", obj, src], capture_output=True, text=True)
        return src, obj, res

    with ThreadPoolExecutor(max_workers=4) as ex:          # one nvcc per translation unit
        results = list(ex.map(compile_one, sources()))
    objs = []
    for src, obj, res in results:
        if verbose or res.returncode != 0:
            sys.stderr.write(res.stdout + res.stderr)
        if res.returncode != 0:
            raise subprocess.CalledProcessError(res.returncode, "nvcc -c " + src)
        objs.append(obj)
    tmp = lib + ".tmp%d" % os.getpid()
    subprocess.check_call([nvcc, "--shared", "-cudart", "static", "-gencode", "arch=compute_100a,code=sm_100a",
                           "-o", tmp] + objs)
    os.replace(tmp, lib)
    for obj in objs:
        os.remove(obj)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, checked="--checked" in sys.argv))
