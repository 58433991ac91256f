"""Builds libg10.so (the CUDA library behind the C ABI) in-tree with nvcc for sm_100a.

Every source is compiled to its own object file (in parallel, only when it or a header is newer), then linked.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
OBJ_PLAIN, OBJ_HOOKS = os.path.join(HERE, "build"), os.path.join(HERE, "build_hooks")
LIB_PLAIN, LIB_HOOKS = os.path.join(HERE, "libg10.so"), os.path.join(HERE, "libg10_hooks.so")
LIB = LIB_PLAIN
SOURCES = ["g10_api.cu", "g10_passes.cu", "g10_planner.cu", "g10_planner_lazy.cu", "g10_planner_small.cu",
           "g10_planner_one.cu", "g10_vitality_buckets.cu", "g10_prefetch.cu", "g10_emit.cu", "g10_stats.cu", "g10_cyclic.cu",
           "g10_static.cu"]
HEADERS = ["g10_device.cuh", "g10_internal.h", "g10_planner.cuh"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC"]


def _newer(path: str, than: float) -> bool:
    return os.path.getmtime(path) > than


def build(force: bool = False, verbose: bool = False, hooks: bool = False) -> str:
    """hooks=True builds libg10_hooks.so instead: the same sources with -DG10_TEST_HOOKS (used by one test that makes a
    bounded device wait run out; never loaded by the binding)."""
    nvcc = os.environ.get("NVCC", "nvcc")
    OBJ, LIB = (OBJ_HOOKS, LIB_HOOKS) if hooks else (OBJ_PLAIN, LIB_PLAIN)
    flags = NVCC_FLAGS + (["-DG10_TEST_HOOKS"] if hooks else [])
    headers = [os.path.join(CSRC, h) for h in HEADERS] + [os.path.join(ROOT, "include", "g10.h"), os.path.abspath(__file__)]
    os.makedirs(OBJ, exist_ok=True)
    sources = [f for f in SOURCES if os.path.exists(os.path.join(CSRC, f))]
    jobs = []
    for f in sources:
        src, obj = os.path.join(CSRC, f), os.path.join(OBJ, f[:-3] + ".o")
        if force or verbose or not os.path.exists(obj) or any(_newer(d, os.path.getmtime(obj)) for d in [src] + headers):
            jobs.append((src, obj))

    def compile_one(job):
        src, obj = job
        tmp = "%s.%d.tmp" % (obj, os.getpid())          # several processes may build at once: each renames a finished file
        cmd = [nvcc] + flags + (["-Xptxas", "-v"] if verbose else []) + ["-I" + os.path.join(ROOT, "include"), "-c", "-o", tmp, src]
        try:
            subprocess.check_call(cmd)
            os.replace(tmp, obj)
        finally:
            if os.path.exists(tmp):
                os.remove(tmp)

    if jobs:
        with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 4)) as pool:
            list(pool.map(compile_one, jobs))
    objs = [os.path.join(OBJ, f[:-3] + ".o") for f in sources]
    if jobs or not os.path.exists(LIB) or any(_newer(o, os.path.getmtime(LIB)) for o in objs):
        tmp = "%s.%d.tmp" % (LIB, os.getpid())
        try:
            subprocess.check_call([nvcc, "-shared", "-Wno-deprecated-gpu-targets", "-o", tmp] + objs)
            os.replace(tmp, LIB)
        finally:
            if os.path.exists(tmp):
                os.remove(tmp)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, hooks="--hooks" in sys.argv))
