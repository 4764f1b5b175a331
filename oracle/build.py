"""Builds the CPU oracle shared library (test infrastructure, not product).

g++ -O2 with -ffp-contract=off so that no multiply-add pair is fused: every
binary32 operation of the canonical update is rounded once, as the header of
ps_oracle.cpp states.  No -ffast-math, no -march flags (no FMA codegen).
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "ps_oracle.cpp")
LIB = os.path.join(HERE, "libps_oracle.so")


def build(force: bool = False) -> str:
    if (not force and os.path.exists(LIB)
            and os.path.getmtime(LIB) >= os.path.getmtime(SRC)):
        return LIB
    cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math",
           "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra", "-o", LIB, SRC]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))
