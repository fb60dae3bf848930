"""Builds the CUDA library in-tree: ``paper_2002_05814_b200/libhpl.so`` (sm_100a only)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
DEBUG = os.environ.get("HPL_DEBUG_BOUNDS") == "1"      # the bounds-checking build, selected like in hpl.lib_path()
LIB = os.path.join(HERE, "libhpl_debug.so" if DEBUG else "libhpl.so")
SOURCES = ["hpl.cpp", "directory.cpp", "plan_reduce.cpp", "plan_bcast.cpp", "sched_reduce.cpp", "sched_bcast.cpp",
           "kernels.cu", "noalloc.cu"]
HEADERS = ["context.h", "device_types.h", "sched_reduce.h", "sched_bcast.h", os.path.join("..", "..", "include", "hpl.h")]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(os.path.join(CSRC, f)) > t for f in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compiles the library if a source is newer than it.  Returns the path of the .so."""
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-shared", "-Xcompiler", "-fPIC", "-std=c++17", "-O3", "-lineinfo",
           "-gencode", "arch=compute_100a,code=sm_100a", "-x", "cu"]
    if DEBUG:
        cmd += ["-DHPL_DEBUG_BOUNDS"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, f) for f in SOURCES] + ["-ldl", "-o", LIB]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed")
    if verbose:
        sys.stderr.write(res.stderr)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
