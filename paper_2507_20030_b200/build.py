"""Build the CUDA library in-tree with nvcc for sm_100a.

    python -m paper_2507_20030_b200.build [--force] [-v] [--debug]

nvcc cross-compiles without a GPU.  The result, lib/libfaedkv.so, links the
static CUDA runtime and resolves the driver entry points it needs at run time,
so it loads on a machine without a GPU (calls then fail with a CUDA error).
--debug builds the checked variant, lib/libfaedkv_debug.so (-DFAEDKV_DEBUG:
device-side bounds checks that record a failure instead of faulting).
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB_DIR = os.path.join(_HERE, "lib")
LIB = os.path.join(LIB_DIR, "libfaedkv.so")
LIB_DEBUG = os.path.join(LIB_DIR, "libfaedkv_debug.so")
INCLUDE = os.path.join(os.path.dirname(_HERE), "include")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--shared", "-Xcompiler", "-fPIC", "-cudart", "static", "-ldl", "--threads", "2",
]


def sources() -> list[str]:
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps() -> list[str]:
    return sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(INCLUDE, "*.h"))


def is_stale(debug: bool = False) -> bool:
    lib = LIB_DEBUG if debug else LIB
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(f) > t for f in _deps())


def start(force: bool = False, verbose: bool = False, debug: bool = False):
    """Start the compilation (if the library is stale); returns (process or None, temporary path, final path)."""
    lib = LIB_DEBUG if debug else LIB
    if not force and not is_stale(debug):
        return None, None, lib
    os.makedirs(LIB_DIR, exist_ok=True)
    tmp = lib + ".tmp.%d" % os.getpid()
    cmd = ["nvcc", *NVCC_FLAGS, *(["-DFAEDKV_DEBUG"] if debug else []), "-I", INCLUDE, "-o", tmp, *sources()]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
        print(" ".join(cmd), file=sys.stderr)
    return subprocess.Popen(cmd), tmp, lib


def finish(job) -> str:
    proc, tmp, lib = job
    if proc is not None:
        if proc.wait() != 0:
            raise subprocess.CalledProcessError(proc.returncode, proc.args)
        os.replace(tmp, lib)
    return lib


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    return finish(start(force, verbose, debug))


def build_all(force: bool = False) -> list[str]:
    """The normal and the checked library, compiled side by side."""
    jobs = [start(force, False, False), start(force, False, True)]
    return [finish(j) for j in jobs]


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
