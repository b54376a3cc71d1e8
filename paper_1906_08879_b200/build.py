"""Builds the CUDA library in-tree with nvcc for sm_100a.

``python paper_1906_08879_b200/build.py`` (or ``build()``; run it as a script, since
importing the package needs the library this builds) compiles every
source under ``csrc/`` into ``libplaceto.so`` next to this file. nvcc
cross-compiles without a GPU; the result is only usable on a B200.

``build(debug=True)`` (``--debug`` on the command line) makes
``libplaceto_debug.so`` from the same sources with ``-DPLACETO_DEBUG``: its
kernels check the schedule records, slot, node and state indices they stage and
report a violation through the call's status record (see
``placeto_last_status``) instead of touching memory they should not. The
binding loads it when the environment variable ``PLACETO_LIBRARY=debug`` is set.

``build(timers=True)`` (``--timers``) makes ``libplaceto_timers.so`` with
``-DPLACETO_PHASE_TIMERS``: the kernels built on tcgen05 (step 2 at d = 64 under
PLACETO_TCGEN05, step 3 at d = 64) print, from block 0, the cycles each of their
warp roles spent per phase. Selected with ``PLACETO_LIBRARY=timers``; a
measuring aid, slower than the release build.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(HERE, "libplaceto.so")
LIB_DEBUG = os.path.join(HERE, "libplaceto_debug.so")
LIB_TIMERS = os.path.join(HERE, "libplaceto_timers.so")

SOURCES = ["api.cu", "plan.cpp", "features.cu", "embed_generic.cu", "embed_d32.cu", "embed_d64.cu", "embed_mma.cu", "embed_pipe.cu", "embed_tc.cu",
           "policy_generic.cu", "policy_d32.cu", "policy_d64.cu", "episode.cu",
           "embed_rounds_d32.cu", "simulator.cu", "gradient.cu", "status.cu", "aggregator.cu", "policy_tc.cu"]

NVCC_FLAGS = ["-O3", "-std=c++17", "-lineinfo",
              "-gencode", "arch=compute_100a,code=sm_100a",
              "-Xcompiler", "-fPIC,-Wall,-Wextra", "-I", INCLUDE, "-I", CSRC]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found: the CUDA library cannot be built")
    return exe


def _stale(target: str, deps: list[str]) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False, timers: bool = False) -> str:
    """Compiles changed sources (in parallel) and links the library; returns its path."""
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    headers.append(os.path.join(INCLUDE, "placeto.h"))
    if debug and timers:
        raise ValueError("one variant at a time")
    objdir = os.path.join(HERE, "_build", "debug" if debug else "timers" if timers else "release")
    os.makedirs(objdir, exist_ok=True)
    lib = LIB_DEBUG if debug else LIB_TIMERS if timers else LIB
    flags = NVCC_FLAGS + (["-DPLACETO_DEBUG"] if debug else ["-DPLACETO_PHASE_TIMERS"] if timers else [])
    objs, jobs = [], []
    for src in SOURCES:
        path = os.path.join(CSRC, src)
        obj = os.path.join(objdir, os.path.splitext(src)[0] + ".o")
        objs.append(obj)
        if force or _stale(obj, [path] + headers + [os.path.abspath(__file__)]):
            cmd = [_nvcc(), "-c", path, "-o", obj] + flags
            if verbose:
                cmd += ["-Xptxas", "-v"]
                print(" ".join(cmd), file=sys.stderr)
            jobs.append(cmd)
    with ThreadPoolExecutor(max_workers=max(1, min(len(jobs), os.cpu_count() or 1))) as pool:
        for done in pool.map(lambda c: subprocess.run(c, check=False), jobs):
            if done.returncode != 0:
                raise RuntimeError("nvcc failed: " + " ".join(done.args))
    if jobs or not os.path.exists(lib):
        tmp = lib + ".tmp%d" % os.getpid()
        subprocess.run([_nvcc(), "-shared", "-o", tmp] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"],
                       check=True)
        os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv,
                timers="--timers" in sys.argv))
