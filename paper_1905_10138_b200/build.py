"""Builds ``libsqnn.so`` (C-ABI library: host encoder + sm_100a kernels) in-tree with nvcc."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(HERE, "libsqnn.so")
SOURCES = ["sqnn_host.cpp", "sqnn_kernels.cu", "sqnn_mma.cu"]
HEADERS = ["sqnn_blob.h", "sqnn_decode.cuh", "sqnn_launch.h"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS] + [os.path.join(INCLUDE, "sqnn.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    objdir = os.path.join(HERE, "_build")
    os.makedirs(objdir, exist_ok=True)
    common = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-I", INCLUDE, "-I", CSRC, "-Xcompiler", "-fPIC,-fopenmp,-O3"]
    if verbose:
        common += ["-Xptxas", "-v"]
    procs, objs = [], []
    for s in SOURCES:
        o = os.path.join(objdir, os.path.splitext(s)[0] + ".o")
        objs.append(o)
        procs.append(subprocess.Popen([_nvcc(), *common, "-c", os.path.join(CSRC, s), "-o", o]))
    for p in procs:
        if p.wait() != 0:
            raise RuntimeError("nvcc failed")
    subprocess.run([_nvcc(), "-shared", "-o", LIB, *objs, "-Xcompiler", "-fopenmp", "-lgomp"], check=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
