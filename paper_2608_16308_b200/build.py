"""Builds libdbspmspv.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libdbspmspv.so")
LIB_CHECKED = os.path.join(HERE, "libdbspmspv_check.so")   # the range-checked build (-DDBS_BOUNDS_CHECK)
SOURCES = ("create.cu", "run.cu", "bfs.cu", "api.cu", "noalloc.cu", "measure.cu")
HEADERS = ("internal.cuh", "microkernels.cuh", "worklist.cuh", "staging.cuh", "lean_pull.cuh", "decode_batch.cuh", "mma_block.cuh", "minplus.cuh", "small_call.cuh")
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Compiles the sources that changed and links the library; checked=True builds the
    range-checked variant beside it (own object files, own .so)."""
    lib = LIB_CHECKED if checked else LIB
    extra = ["-DDBS_BOUNDS_CHECK"] if checked else []
    deps_common = [os.path.join(CSRC, h) for h in HEADERS] + [os.path.join(ROOT, "include", "dbspmspv.h"),
                                                              os.path.abspath(__file__)]
    objs, jobs = [], []
    for src in SOURCES:
        s = os.path.join(CSRC, src)
        o = os.path.join(CSRC, src.replace(".cu", ".chk.o" if checked else ".o"))
        objs.append(o)
        if force or _stale(o, [s] + deps_common):
            cmd = [_nvcc()] + NVCC_FLAGS + extra + os.environ.get("DBS_EXTRA_NVCC_FLAGS", "").split() \
                + (["-Xptxas", "-v"] if verbose else []) + ["-c", s, "-o", o]
            jobs.append(cmd)

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed: " + " ".join(cmd) + "\n" + r.stdout + r.stderr)
        return r.stderr

    if jobs:
        with ThreadPoolExecutor(max_workers=len(jobs)) as ex:
            for out in ex.map(run, jobs):
                if verbose:
                    sys.stderr.write(out)
    if jobs or force or _stale(lib, objs):
        run([_nvcc(), "-shared", "-o", lib] + objs + ["-lcudart"])
    return lib


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
