"""Compile libdarkattn.so (CUDA, sm_100a) in-tree with nvcc. No GPU is needed to build."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
LIB = os.path.join(HERE, "libdarkattn.so")
BENCH_LIB = os.path.join(HERE, "libdarkattn_bench.so")     # instruments of the benchmark (per-kernel times, MMA probe)
SOURCES = sorted(glob.glob(os.path.join(HERE, "csrc", "*.cu")))
BENCH_SOURCES = sorted(glob.glob(os.path.join(HERE, "csrc_bench", "*.cu")))
HEADERS = sorted(glob.glob(os.path.join(HERE, "csrc", "*.cuh"))) + [os.path.join(ROOT, "include", "darkattn.h"),
                                                                     os.path.join(ROOT, "include", "darkattn_bench.h")]


def stale() -> bool:
    if not os.path.exists(LIB) or not os.path.exists(BENCH_LIB):
        return True
    t = min(os.path.getmtime(LIB), os.path.getmtime(BENCH_LIB))
    return any(os.path.getmtime(f) > t for f in SOURCES + BENCH_SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objdir = os.path.join(HERE, "_build")
    os.makedirs(objdir, exist_ok=True)
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
             "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include")]
    if verbose:
        flags += ["-Xptxas", "-v"]
    # one object per translation unit, compiled side by side (only the stale ones), then one link
    jobs, objs, bench_objs = [], [], []
    newest_header = max(os.path.getmtime(h) for h in HEADERS)
    for src in SOURCES + BENCH_SOURCES:
        bench = src in BENCH_SOURCES
        obj = os.path.join(objdir, ("bench_" if bench else "") + os.path.basename(src)[:-3] + ".o")
        (bench_objs if bench else objs).append(obj)
        if force or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(src), newest_header):
            jobs.append((src, subprocess.Popen([nvcc] + flags + ["-c", src, "-o", obj])))
    failed = [src for src, pr in jobs if pr.wait() != 0]
    if failed:
        raise RuntimeError("nvcc failed for " + ", ".join(failed))
    link = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-Xcompiler", "-fPIC"]
    subprocess.run(link + ["-o", LIB] + objs, check=True)
    # the instruments use the product's plan object and error reporting: linked against it, found beside it at run time
    subprocess.run(link + ["-o", BENCH_LIB] + bench_objs + ["-L", HERE, "-l:libdarkattn.so", "-Xlinker", "-rpath=$ORIGIN"], check=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
