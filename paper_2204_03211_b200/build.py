"""Builds the C-ABI shared library in-tree with nvcc for sm_100a.

    python -m paper_2204_03211_b200.build [--force] [--verbose]

The library is rebuilt when any source under csrc/ or the public header is
newer than the .so.  FMA contraction is disabled (--fmad=false) on top of the
explicit round-to-nearest intrinsics in the kernels; fast-math is never used.
"""
import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libps_b200.so")
SOURCES = [os.path.join(CSRC, "ps_service.cu"), os.path.join(CSRC, "ps_planner.cpp"), os.path.join(CSRC, "ps_peer.cpp")]


def _deps():
    return (glob.glob(os.path.join(CSRC, "*")) + glob.glob(os.path.join(ROOT, "include", "*.h")))


def nvcc_command(verbose: bool = False):
    cmd = ["nvcc", "-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "--fmad=false", "-Xcompiler", "-fPIC,-Wall,-O2", "-shared", "-cudart", "shared",
           "-I", os.path.join(ROOT, "include"), "-o", LIB] + SOURCES
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    return cmd


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and os.path.exists(LIB):
        newest = max(os.path.getmtime(p) for p in _deps())
        if os.path.getmtime(LIB) >= newest:
            return LIB
    res = subprocess.run(nvcc_command(verbose), capture_output=True, text=True)
    if verbose or res.returncode:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode:
        raise RuntimeError("nvcc failed building %s" % LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
