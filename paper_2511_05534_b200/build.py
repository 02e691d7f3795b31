"""Builds the CUDA library (libflowmm.so) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
CSRC = os.path.join(_PKG, "csrc")
LIB_PATH = os.path.join(_PKG, "libflowmm.so")
DEBUG_LIB_PATH = os.path.join(_PKG, "libflowmm_debug.so")     # the same sources with -DFLOWMM_DEBUG (index checks)
SOURCES = ["flowmm_api.cu"]


def _newest_source_mtime() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(_ROOT, "include", "flowmm.h")]
    return max(os.path.getmtime(p) for p in paths)


def nvcc_command(out: str, verbose_ptxas: bool = False, debug: bool = False):
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared", "-cudart", "static", "-I", os.path.join(_ROOT, "include"), "-I", CSRC,
           "-o", out]
    if verbose_ptxas:
        cmd += ["-Xptxas", "-v"]
    if debug:
        cmd += ["-DFLOWMM_DEBUG"]
    return cmd + [os.path.join(CSRC, s) for s in SOURCES]


def build(force: bool = False, verbose_ptxas: bool = False, debug: bool = False) -> str:
    """Compile if the library is missing or older than any source; returns its path.  debug: the build with
    index checks (libflowmm_debug.so) instead of the release library."""
    path = DEBUG_LIB_PATH if debug else LIB_PATH
    if force or not os.path.exists(path) or os.path.getmtime(path) < _newest_source_mtime():
        tmp = path + ".%d.tmp" % os.getpid()
        subprocess.check_call(nvcc_command(tmp, verbose_ptxas, debug))
        os.replace(tmp, path)
    return path


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose_ptxas="-v" in sys.argv, debug="--debug" in sys.argv))
