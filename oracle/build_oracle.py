"""Compile the CPU oracle (test infrastructure) into oracle/libslonn_oracle.so.

-ffp-contract=off keeps gcc from fusing a*b+c on its own, so that the only
fused multiply-adds are the explicit fmaf() calls of the summation contract;
-mfma makes those a single hardware instruction.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "slonn_oracle.c")
OUT = os.path.join(HERE, "libslonn_oracle.so")


def build(force: bool = False) -> str:
    if (not force and os.path.exists(OUT)
            and os.path.getmtime(OUT) >= os.path.getmtime(SRC)):
        return OUT
    cmd = ["gcc", "-O2", "-std=c11", "-D_GNU_SOURCE", "-ffp-contract=off", "-mfma",
           "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra", "-o", OUT, SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return OUT


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))
