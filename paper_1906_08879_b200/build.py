"""Builds the CUDA library in-tree with nvcc for sm_100a.

``python paper_1906_08879_b200/build.py`` (or ``build()``; run it as a script, since
importing the package needs the library this builds) compiles every
source under ``csrc/`` into ``libplaceto.so`` next to this file. nvcc
cross-compiles without a GPU; the result is only usable on a B200.
"""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(HERE, "libplaceto.so")

SOURCES = ["api.cu", "plan.cpp", "features.cu", "embed_generic.cu", "embed_d32.cu", "embed_d64.cu", "embed_mma.cu", "embed_tc.cu",
           "policy_generic.cu", "policy_d32.cu", "policy_d64.cu", "episode.cu",
           "embed_rounds_d32.cu", "simulator.cu", "gradient.cu", "status.cu"]

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


def build(force: bool = False, verbose: bool = False) -> str:
    """Compiles changed sources and links libplaceto.so; returns its path."""
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    headers.append(os.path.join(INCLUDE, "placeto.h"))
    objdir = os.path.join(HERE, "_build")
    os.makedirs(objdir, exist_ok=True)
    objs = []
    relink = force
    for src in SOURCES:
        path = os.path.join(CSRC, src)
        obj = os.path.join(objdir, os.path.splitext(src)[0] + ".o")
        objs.append(obj)
        if force or _stale(obj, [path] + headers + [os.path.abspath(__file__)]):
            cmd = [_nvcc(), "-c", path, "-o", obj] + NVCC_FLAGS
            if verbose:
                cmd += ["-Xptxas", "-v"]
                print(" ".join(cmd), file=sys.stderr)
            subprocess.run(cmd, check=True)
            relink = True
    if relink or not os.path.exists(LIB):
        tmp = LIB + ".tmp%d" % os.getpid()
        subprocess.run([_nvcc(), "-shared", "-o", tmp] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"],
                       check=True)
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
