"""Builds the CUDA library (libflowmm.so) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
CSRC = os.path.join(_PKG, "csrc")
LIB_PATH = os.path.join(_PKG, "libflowmm.so")
SOURCES = ["flowmm_api.cu"]


def _newest_source_mtime() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(_ROOT, "include", "flowmm.h")]
    return max(os.path.getmtime(p) for p in paths)


def nvcc_command(out: str, verbose_ptxas: bool = False):
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared", "-cudart", "static", "-I", os.path.join(_ROOT, "include"), "-I", CSRC,
           "-o", out]
    if verbose_ptxas:
        cmd += ["-Xptxas", "-v"]
    return cmd + [os.path.join(CSRC, s) for s in SOURCES]


def build(force: bool = False, verbose_ptxas: bool = False) -> str:
    """Compile if the library is missing or older than any source; returns its path."""
    if force or not os.path.exists(LIB_PATH) or os.path.getmtime(LIB_PATH) < _newest_source_mtime():
        tmp = LIB_PATH + ".%d.tmp" % os.getpid()
        subprocess.check_call(nvcc_command(tmp, verbose_ptxas))
        os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose_ptxas="-v" in sys.argv))
