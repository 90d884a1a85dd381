"""Builds the C-ABI shared library `libaded.so` from csrc/*.cu with nvcc for sm_100a.

    python -m paper_2407_12021_b200.build [--force] [--verbose] [--debug]

Objects go to a git-ignored `_build/` folder beside this file; the library is written next to
this file so that it travels with the source tree.  `--debug` builds `libaded_debug.so` instead: the same
sources with -DADED_DEBUG_CHECKS, i.e. with index checks on slot, cache-row and bucket addressing that
report ADED_ERR_INTERNAL through the status word (the stand-in for a memory checker on machines where
none may be run); select it with the environment variable ADED_LIBRARY.
"""
from __future__ import annotations

import concurrent.futures
import glob
import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(ROOT, "include")
OBJ_DIR = os.path.join(HERE, "_build")
LIB_PATH = os.path.join(HERE, "libaded.so")

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr",
    "-I", INCLUDE, "-I", CSRC,
]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found: the CUDA library cannot be built")
    return exe


def _newest(paths) -> float:
    return max(os.path.getmtime(p) for p in paths)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    obj_dir = OBJ_DIR + ("_debug" if debug else "")
    lib_path = os.path.join(HERE, "libaded_debug.so") if debug else LIB_PATH
    flags = NVCC_FLAGS + (["-DADED_DEBUG_CHECKS"] if debug else [])
    sources = sorted(glob.glob(os.path.join(CSRC, "*.cu")))
    headers = sorted(glob.glob(os.path.join(CSRC, "*.cuh"))) + sorted(glob.glob(os.path.join(INCLUDE, "*.h")))
    if not sources:
        raise RuntimeError("no CUDA sources found")
    os.makedirs(obj_dir, exist_ok=True)
    dep_time = _newest(headers + [os.path.abspath(__file__)])
    nvcc = _nvcc()
    jobs = []
    objects = []
    for src in sources:
        obj = os.path.join(obj_dir, os.path.basename(src)[:-3] + ".o")
        objects.append(obj)
        stale = force or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(src), dep_time)
        if stale:
            jobs.append([nvcc] + flags + (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", obj])

    def run(cmd):
        res = subprocess.run(cmd, capture_output=True, text=True)
        return cmd, res

    if jobs:
        with concurrent.futures.ThreadPoolExecutor(max_workers=min(8, len(jobs))) as pool:
            for cmd, res in pool.map(run, jobs):
                if verbose or res.returncode != 0:
                    sys.stderr.write(" ".join(cmd) + "\n" + res.stdout + res.stderr)
                if res.returncode != 0:
                    raise RuntimeError(f"nvcc failed on {cmd[-3]}")
    if jobs or not os.path.exists(lib_path) or os.path.getmtime(lib_path) < _newest(objects):
        cmd = [nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", lib_path] + objects
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            sys.stderr.write(res.stdout + res.stderr)
            raise RuntimeError(f"linking {os.path.basename(lib_path)} failed")
    return lib_path


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug="--debug" in sys.argv))
