"""Compile the CPU oracle (oracle/moe_oracle.cpp) into oracle/liboracle_moe.so.

Test infrastructure: called by the test fixtures, by the build check and by the
benchmark's cpu_baseline leg.  Plain g++, no CUDA, no code from the library.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "moe_oracle.cpp")
LIB = os.path.join(HERE, "liboracle_moe.so")

# -ffp-contract=off: the compiler must not fuse a*b+c on its own; the fused
# operations of the definition are the explicit std::fmaf calls only.
FLAGS = ["-O2", "-std=c++17", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared", "-fPIC"]


def build(force: bool = False) -> str:
    """Build the shared object if it is missing or older than its source; return its path."""
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    tmp = LIB + ".tmp.%d" % os.getpid()
    subprocess.run(["g++", *FLAGS, "-o", tmp, SRC], check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))
