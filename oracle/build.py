"""Compile the CPU oracle (oracle/mok_ref.c, oracle/mok_ref_mx.c, oracle/mok_ref_bwd.c) into oracle/libmok_ref.so with gcc.

Test infrastructure only.  Building the checker is not using it: the product never loads this
library.  Run `python oracle/build.py` or call `build()`.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "mok_ref.c")
SRCS = [SRC, os.path.join(HERE, "mok_ref_mx.c"), os.path.join(HERE, "mok_ref_bwd.c")]
LIB = os.path.join(HERE, "libmok_ref.so")


def build(force: bool = False) -> str:
    if (not force and os.path.exists(LIB)
            and os.path.getmtime(LIB) >= max(os.path.getmtime(f) for f in SRCS)):
        return LIB
    # No -ffast-math: the summation order written in the source is the order evaluated.
    cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-Wall", "-Wextra",
           "-o", LIB + ".tmp", *SRCS, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(LIB + ".tmp", LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))
