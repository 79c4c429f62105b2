"""Builds libcovspec.so in-tree with nvcc for sm_100a (no torch extension machinery: the library
is a plain C ABI loaded through ctypes)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libcovspec.so")
LIB_DEBUG = os.path.join(HERE, "libcovspec_debug.so")     # the same sources with -DCOVSPEC_DEBUG_BOUNDS
SOURCES = ["covspec.cu"]


def _newest(paths):
    return max(os.path.getmtime(p) for p in paths)


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + \
           [os.path.join(ROOT, "include", "covspec.h")]
    return _newest(deps) > os.path.getmtime(lib)


def build(force: bool = False, verbose: bool = False, debug_bounds: bool = False) -> str:
    """Builds the library if a source is newer than it.  debug_bounds=True builds the checked variant
    (libcovspec_debug.so): index-driven accesses test their index and report COVSPEC_ERR_BOUNDS."""
    LIB = LIB_DEBUG if debug_bounds else globals()["LIB"]
    if not force and not needs_build(LIB):
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-shared", "-Xcompiler", "-fPIC", "-O3", "-std=c++17", "-lineinfo",
           "-gencode", "arch=compute_100a,code=sm_100a",
           "-I", os.path.join(ROOT, "include"), "-I", CSRC,
           "-o", LIB] + [os.path.join(CSRC, s) for s in SOURCES]
    if debug_bounds:
        cmd.insert(1, "-DCOVSPEC_DEBUG_BOUNDS")
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed building " + os.path.basename(LIB))
    if verbose:
        sys.stderr.write(res.stderr)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv, debug_bounds="--debug-bounds" in sys.argv))
