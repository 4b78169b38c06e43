"""Builds ``libsqnn.so`` (C-ABI library: host encoder + sm_100a kernels) in-tree with nvcc."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(HERE, "libsqnn.so")
SOURCES = ["sqnn_host.cpp", "sqnn_api.cu", "sqnn_mma.cu", "sqnn_search.cu"]
SHAPE_SOURCE = "sqnn_shape.cu"
# (n_out, n_in) with compile-time kernels -- the list in csrc/sqnn_shapes.h -- plus the run-time shape (0, 0)
SHAPES = [(40, 12), (40, 16), (60, 12), (80, 8), (80, 16), (100, 10), (200, 10), (0, 0)]
HEADERS = ["sqnn_blob.h", "sqnn_layout.h", "sqnn_decode.cuh", "sqnn_launch.h", "sqnn_kernels.cuh", "sqnn_gemv.cuh", "sqnn_shapes.h", SHAPE_SOURCE]


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
    jobs = []
    for s in SOURCES:
        jobs.append(([os.path.join(CSRC, s)], os.path.join(objdir, os.path.splitext(s)[0] + ".o")))
    for no, ni in SHAPES:
        jobs.append(([f"-DSQNN_NO={no}", f"-DSQNN_NI={ni}", os.path.join(CSRC, SHAPE_SOURCE)],
                     os.path.join(objdir, f"sqnn_shape_{no}x{ni}.o")))
    objs = [o for _, o in jobs]
    width = max(1, min(len(jobs), os.cpu_count() or 4))
    pending, running = list(jobs), []
    while pending or running:
        while pending and len(running) < width:
            extra, o = pending.pop(0)
            running.append(subprocess.Popen([_nvcc(), *common, "-c", *extra, "-o", o]))
        if running[0].wait() != 0:
            for r in running[1:]:
                r.wait()
            raise RuntimeError("nvcc failed")
        running.pop(0)
    subprocess.run([_nvcc(), "-shared", "-o", LIB, *objs, "-Xcompiler", "-fopenmp", "-lgomp"], check=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
