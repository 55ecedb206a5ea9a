"""Builds librsd.so in-tree with nvcc for sm_100a (no GPU needed to compile)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "librsd.so")
SOURCES = ["rsd_api.cu"]
HEADERS = ["rsd_device.cuh", "rsd_scan.cuh", "rsd_verify.cuh", os.path.join("..", "..", "include", "rsd.h")]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(os.path.join(CSRC, f)) > t for f in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False, out: str = LIB, defines=()) -> str:
    """Build the library (default: in-tree librsd.so).  `out`/`defines` build a variant elsewhere, e.g. the
    small-queue build the tests use to exercise the scan kernel's overflow paths."""
    if out == LIB and not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = out + ".%d.tmp" % os.getpid()
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-shared",
           "-Xcompiler", "-fPIC", "--use_fast_math" if False else "-DRSD_BUILD", "-o", tmp]
    cmd += ["-D" + d for d in defines]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, f) for f in SOURCES]
    subprocess.check_call(cmd)
    os.replace(tmp, out)
    return out


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
