"""Compile the CUDA sources into paper_1911_04070_b200/libbpt.so for sm_100a.

Usage: python -m paper_1911_04070_b200.build [--force] [--verbose]
nvcc cross-compiles without a GPU; the shared object stays inside the package
directory so that it travels with the source tree.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libbpt.so")
LIB_CHECK = os.path.join(HERE, "libbpt_check.so")   # the same sources with -DBPT_BOUNDS_CHECK (see csrc/bounds_check.cuh)
OBJ = os.path.join(HERE, "_build")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC"]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def _build_one(lib: str, tag: str, extra: list, force: bool, verbose: bool) -> str:
    srcs = sorted(glob.glob(os.path.join(CSRC, "*.cu")))
    deps = srcs + glob.glob(os.path.join(CSRC, "*.cuh")) + [os.path.join(HERE, "..", "include", "bpt.h")]
    newest = max(os.path.getmtime(p) for p in deps)
    if not force and os.path.exists(lib) and os.path.getmtime(lib) >= newest:
        return lib
    os.makedirs(OBJ, exist_ok=True)
    procs, objs = [], []
    for s in srcs:
        o = os.path.join(OBJ, os.path.basename(s)[:-3] + tag + ".o")
        objs.append(o)
        if not force and os.path.exists(o) and os.path.getmtime(o) >= newest:
            continue
        cmd = [_nvcc()] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-c", s, "-o", o]
        procs.append((cmd, subprocess.Popen(cmd)))
    for cmd, p in procs:
        if p.wait() != 0:
            raise RuntimeError("nvcc failed: " + " ".join(cmd))
    tmp = lib + ".tmp%d" % os.getpid()
    subprocess.check_call([_nvcc()] + NVCC_FLAGS[:2] + (["-rdc=true"] if "-rdc=true" in extra else []) + ["-shared", "-o", tmp] + objs + ["-lcudart"])
    os.replace(tmp, lib)
    return lib


def build(force: bool = False, verbose: bool = False) -> str:
    """Builds libbpt.so and the index-checking libbpt_check.so; returns the path of the first."""
    _build_one(LIB, "", [], force, verbose)
    # the checking build shares one violation record across its translation units: relocatable device code
    _build_one(LIB_CHECK, ".chk", ["-DBPT_BOUNDS_CHECK", "-rdc=true"], force, False)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
