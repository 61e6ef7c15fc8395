"""Builds the CPU oracle (test infrastructure) into oracle/libeagle3_oracle.so with gcc.

    python oracle/build.py

-ffp-contract=off keeps every multiply and add a separate IEEE operation, which the oracle's
"tree forward == per-path sequential forward, bit for bit" property relies on.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "eagle3_oracle.c")
HDR = os.path.join(HERE, "eagle3_oracle.h")
LIB = os.path.join(HERE, "libeagle3_oracle.so")


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= max(os.path.getmtime(SRC), os.path.getmtime(HDR)):
        return LIB
    tmp = LIB + ".%d.tmp" % os.getpid()
    cmd = ["gcc", "-O2", "-ftree-vectorize", "-mavx2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
           "-std=c11", "-fPIC", "-shared", "-Wall", "-Wextra", "-Wno-unused-parameter", "-o", tmp, SRC, "-lm"]
    subprocess.run(cmd, check=True, cwd=HERE)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))
