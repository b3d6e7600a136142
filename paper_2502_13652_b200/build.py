"""Builds libc2t.so (sm_100a only) next to this file with nvcc."""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
CSRC = os.path.join(_HERE, "csrc")
INCLUDE = os.path.join(_ROOT, "include")
LIB = os.path.join(_HERE, "libc2t.so")
LIB_DEBUG = os.path.join(_HERE, "libc2t_debug.so")      # the same sources with -DC2T_DEBUG_BOUNDS (index checks)
SOURCES = ["c2t_api.cu", "expand_pass.cu", "argmax_pass.cu", "topm_pass.cu", "tree_kernels.cu", "argmax_static.cu"]


def _newest_source() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(INCLUDE, "c2t.h")]
    return max(os.path.getmtime(p) for p in paths)


def build(force: bool = False, verbose: bool = False, debug_bounds: bool = False) -> str:
    """Compiles the library if it is older than its sources.  debug_bounds: the variant whose kernels check the
    indices of their own writes and report a failed check in a status bit (C2T_ST_INTERNAL)."""
    lib = LIB_DEBUG if debug_bounds else LIB
    if not force and os.path.exists(lib) and os.path.getmtime(lib) >= _newest_source():
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
           "-shared", "-Xcompiler", "-fPIC", "-I", INCLUDE, "-I", CSRC, "-o", lib]
    if debug_bounds:
        cmd += ["-DC2T_DEBUG_BOUNDS"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.check_call(cmd)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug_bounds="--debug-bounds" in sys.argv))
