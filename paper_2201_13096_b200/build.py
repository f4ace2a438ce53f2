"""Compile the library in-tree for sm_100a (nvcc cross-compiles without a GPU).

Three shared objects come out of ``csrc/``:

* ``libspdy_dp.so``        - the product: host plan (g++) + kernels and launch code (nvcc);
* ``libspdy_dp_debug.so``  - the same sources with ``-DSPDY_DEBUG_CHECKS``: every row and table access of
  the forward kernels checks its index and reports through the plan's status word (for tests);
* ``libspdy_plan_host.so`` - ``spdy_plan.cpp`` and ``spdy_search.cpp`` alone, built with the host compiler:
  plans, their verification, the host helpers and the search loop, for machines and tests without nvcc.

Translation units compile in parallel and only when they or a header changed.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG, "csrc")
HEADERS = [os.path.join(os.path.dirname(PKG), "include", "spdy_dp.h"),
           os.path.join(CSRC, "spdy_plan.h"), os.path.join(CSRC, "spdy_device.cuh")]
HOST_SOURCES = [os.path.join(CSRC, "spdy_plan.cpp"), os.path.join(CSRC, "spdy_search.cpp")]
LIB = os.path.join(PKG, "libspdy_dp.so")
LIB_DEBUG = os.path.join(PKG, "libspdy_dp_debug.so")
LIB_HOST = os.path.join(PKG, "libspdy_plan_host.so")
OBJ_ROOT = os.path.join(PKG, "_build")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-lineinfo", "-O3", "-std=c++17",
    "--fmad=false", "--ftz=false", "--prec-div=true", "--prec-sqrt=true",
    "-Xcompiler", "-fPIC",
]
GXX_FLAGS = ["-O2", "-std=c++17", "-fPIC", "-Wall", "-Wextra"]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def cuda_sources() -> list:
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _newest(paths) -> float:
    return max(os.path.getmtime(p) for p in paths)


def _stale(target: str, deps) -> bool:
    return (not os.path.exists(target)) or os.path.getmtime(target) < _newest(deps)


def _run(cmd, log=None):
    res = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    if log is not None:
        log.append(res.stdout)
    if res.returncode != 0:
        sys.stderr.write(res.stdout)
        raise subprocess.CalledProcessError(res.returncode, cmd)


def build_host(force: bool = False) -> str:
    """``libspdy_plan_host.so``: the host side alone, host compiler only."""
    if force or _stale(LIB_HOST, HOST_SOURCES + [HEADERS[0], HEADERS[1]]):
        tmp = LIB_HOST + f".tmp{os.getpid()}"
        _run(["g++", *GXX_FLAGS, "-shared", "-o", tmp, *HOST_SOURCES])
        os.replace(tmp, LIB_HOST)
    return LIB_HOST


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Build ``libspdy_dp.so`` (or the debug library) next to this file unless it is newer than its
    sources.  Returns the library's path; with ``verbose`` the compilers' output (``-Xptxas -v``) goes
    to stdout."""
    lib = LIB_DEBUG if debug else LIB
    sources = cuda_sources()
    if not force and not _stale(lib, sources + HOST_SOURCES + HEADERS):
        return lib
    objdir = os.path.join(OBJ_ROOT, "debug" if debug else "release")
    os.makedirs(objdir, exist_ok=True)
    defines = ["-DSPDY_DEBUG_CHECKS"] if debug else []
    ptxas_opt = []
    jobs, objects, log = [], [], []
    for src in sources:
        obj = os.path.join(objdir, os.path.basename(src) + ".o")
        objects.append(obj)
        if force or verbose or _stale(obj, [src] + HEADERS):
            jobs.append([_nvcc(), *NVCC_FLAGS, *defines, *ptxas_opt, *(["-Xptxas", "-v"] if verbose else []), "-c", "-o", obj, src])
    for src in HOST_SOURCES:
        host_obj = os.path.join(objdir, os.path.basename(src) + ".o")
        objects.append(host_obj)
        if force or _stale(host_obj, [src, HEADERS[0], HEADERS[1]]):
            jobs.append(["g++", *GXX_FLAGS, *defines, "-c", "-o", host_obj, src])
    with ThreadPoolExecutor(max_workers=max(1, min(len(jobs), os.cpu_count() or 1))) as pool:
        list(pool.map(lambda cmd: _run(cmd, log), jobs))
    tmp = lib + f".tmp{os.getpid()}"
    _run([_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", tmp, *objects])
    os.replace(tmp, lib)
    if verbose:
        print("".join(log))
    return lib


def spilling_kernels(log: str) -> list:
    """Kernels that ptxas reports with register spills in a ``-Xptxas -v`` log."""
    import re

    bad = []
    for name, stores in re.findall(r"Function properties for (\S+)\n\s+\d+ bytes stack frame, (\d+) bytes spill stores", log):
        if int(stores) > 0:
            bad.append(name)
    return bad


def build_all(force: bool = False) -> None:
    """All three libraries, the product and the debug library side by side; a forced build also checks that no
    kernel of the product library spills."""
    log = []

    def product():
        if force:
            import contextlib
            import io

            buf = io.StringIO()
            with contextlib.redirect_stdout(buf):
                build(force=True, verbose=True)
            log.append(buf.getvalue())
        else:
            build()

    with ThreadPoolExecutor(max_workers=2) as pool:
        jobs = [pool.submit(product), pool.submit(build, force, False, True)]
        for job in jobs:
            job.result()
    build_host(force=force)
    bad = spilling_kernels("".join(log))
    if bad:
        raise RuntimeError("kernels with register spills: " + ", ".join(bad))


if __name__ == "__main__":
    if "--host" in sys.argv:
        print(build_host(force="--force" in sys.argv))
    else:
        print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
