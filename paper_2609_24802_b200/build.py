"""Builds libtiga.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(ROOT, "include")
LIB = os.path.join(HERE, "libtiga.so")
LIB_CHECKED = os.path.join(HERE, "libtiga_checked.so")      # same sources with -DTIGA_CHECKED (range-checked indices)
SOURCES = ["csr.cu", "csr_plan.cu", "csr_attention.cu", "radius.cu", "radius_lj.cu", "radius_mlp.cu", "knn.cu"]
NVCC_FLAGS = ["-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-I" + INCLUDE, "-I" + CSRC]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Compile every CUDA source for sm_100a and link libtiga.so (or, with checked=True, the checked
    build libtiga_checked.so) next to this file."""
    headers = [os.path.join(INCLUDE, "tiga.h")] + [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".cuh")]
    objdir = os.path.join(HERE, "build_checked" if checked else "build")
    lib = LIB_CHECKED if checked else LIB
    os.makedirs(objdir, exist_ok=True)
    objs = []
    jobs = []
    for src in SOURCES:
        s = os.path.join(CSRC, src)
        o = os.path.join(objdir, src.replace(".cu", ".o"))
        objs.append(o)
        if force or _stale(o, [s] + headers):
            cmd = ([_nvcc()] + NVCC_FLAGS + (["-DTIGA_CHECKED"] if checked else []) + (["-Xptxas", "-v"] if verbose else [])
                   + ["-c", s, "-o", o])
            jobs.append(cmd)
    if jobs:
        with ThreadPoolExecutor(max_workers=len(jobs)) as ex:
            for res in ex.map(lambda c: subprocess.run(c, capture_output=True, text=True), jobs):
                if verbose or res.returncode != 0:
                    sys.stderr.write(res.stdout + res.stderr)
                if res.returncode != 0:
                    raise RuntimeError("nvcc failed")
    if force or jobs or _stale(lib, objs):
        subprocess.check_call([_nvcc(), "-shared", "-o", lib] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"])
    if not checked:
        build_bench_probe(force)
    return lib


def build_bench_probe(force: bool = False) -> str:
    """The benchmark's row-gather probe is a library of its own: it measures, it is not product."""
    src = os.path.join(HERE, "bench_probe", "row_gather_probe.cu")
    lib = os.path.join(HERE, "bench_probe", "libtiga_bench_probe.so")
    if force or _stale(lib, [src]):
        subprocess.check_call([_nvcc(), "-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
                               "-Xcompiler", "-fPIC", "-shared", src, "-o", lib])
    return lib


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv))
    if "--no-checked" not in sys.argv:
        print(build_library(force="--force" in sys.argv, checked=True))
