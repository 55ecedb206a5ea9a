"""Builds librsd.so in-tree with nvcc for sm_100a (no GPU needed to compile)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "librsd.so")
SOURCES = ["rsd_api.cu", "rsd_api_verify.cu"]
HEADERS = ["rsd_api_common.h", "rsd_device.cuh", "rsd_scan.cuh", "rsd_filter.cuh", "rsd_verify.cuh", "rsd_verify_walk.inc", "rsd_walk_ring.cuh", os.path.join("..", "..", "include", "rsd.h")]


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
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC",
             "-DRSD_BUILD"] + ["-D" + d for d in defines]
    if verbose:
        flags += ["-Xptxas", "-v"]
    # one object per translation unit, compiled side by side, then one link
    objs = [tmp + "." + os.path.splitext(f)[0] + ".o" for f in SOURCES]
    procs = [subprocess.Popen([nvcc] + flags + ["-c", os.path.join(CSRC, f), "-o", o]) for f, o in zip(SOURCES, objs)]
    codes = [p.wait() for p in procs]
    try:
        if any(codes):
            raise subprocess.CalledProcessError(max(codes), [nvcc] + flags + SOURCES)
        subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", tmp] + objs)
    finally:
        for o in objs:
            if os.path.exists(o):
                os.remove(o)
    os.replace(tmp, out)
    return out


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
