"""Build the CUDA shared library (sm_100a only) in-tree with nvcc.

`python -m paper_2501_12689_b200.build` compiles paper_2501_12689_b200/csrc/*.cu into
paper_2501_12689_b200/libic_cache.so.  Objects are rebuilt only when a source or header is
newer.  nvcc cross-compiles, so no GPU is needed to build.
"""
from __future__ import annotations

import concurrent.futures
import glob
import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
BUILD = os.path.join(CSRC, "_build")
LIB = os.path.join(PKG, "libic_cache.so")
LIB_DEBUG = os.path.join(PKG, "libic_cache_debug.so")   # same sources with -DIC_CACHE_DEBUG_CHECKS

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-std=c++17", "-lineinfo",
    "-Xcompiler", "-fPIC,-Wall,-Wno-unused-function",
    "-I", os.path.join(ROOT, "include"),
]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found; the CUDA library cannot be built")
    return exe


def _newest_dep() -> float:
    deps = glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(CSRC, "*.h"))
    deps += glob.glob(os.path.join(ROOT, "include", "*.h"))
    return max(os.path.getmtime(p) for p in deps)


def _compile(src: str, obj: str, verbose: bool, debug_checks: bool = False) -> str:
    cmd = [_nvcc(), *NVCC_FLAGS, "-c", src, "-o", obj]
    if debug_checks:
        cmd.insert(1, "-DIC_CACHE_DEBUG_CHECKS")
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"nvcc failed for {src}:\n{r.stdout}\n{r.stderr}")
    return r.stderr


def build(force: bool = False, verbose: bool = False, debug_checks: bool = False) -> str:
    """Compile and link libic_cache.so if anything is stale; return its path.  debug_checks: build
    libic_cache_debug.so instead, whose kernels check their indices and report a failed check through
    the status word (they never trap)."""
    os.makedirs(BUILD, exist_ok=True)
    srcs = sorted(glob.glob(os.path.join(CSRC, "*.cu")))
    dep_time = _newest_dep()
    jobs = []
    objs = []
    LIB = LIB_DEBUG if debug_checks else globals()["LIB"]
    for src in srcs:
        obj = os.path.join(BUILD, os.path.basename(src)[:-3] + (".dbg.o" if debug_checks else ".o"))
        objs.append(obj)
        stale = force or not os.path.exists(obj) or \
            os.path.getmtime(obj) < max(os.path.getmtime(src), dep_time)
        if stale:
            jobs.append((src, obj))
    if jobs:
        with concurrent.futures.ThreadPoolExecutor(max_workers=min(8, len(jobs))) as ex:
            for log in ex.map(lambda j: _compile(j[0], j[1], verbose, debug_checks), jobs):
                if verbose and log:
                    print(log, file=sys.stderr)
    if jobs or not os.path.exists(LIB) or any(os.path.getmtime(o) > os.path.getmtime(LIB) for o in objs):
        tmp = LIB + ".tmp.%d" % os.getpid()
        cmd = [_nvcc(), "-shared", "-cudart", "static", "-o", tmp, *objs, "-lpthread", "-ldl", "-lrt"]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError(f"link failed:\n{r.stdout}\n{r.stderr}")
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug_checks="--debug-checks" in sys.argv))
