"""Compile the C part of the oracle (gcc, OpenMP) into oracle/liboracle_gemm.so."""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "gemm_oracle.c")
LIB = os.path.join(HERE, "liboracle_gemm.so")


def build(force: bool = False) -> str:
    if (not force and os.path.exists(LIB)
            and os.path.getmtime(LIB) >= os.path.getmtime(SRC)):
        return LIB
    cmd = ["gcc", "-O2", "-march=native", "-fopenmp", "-fPIC", "-shared", "-o", LIB, SRC]
    try:
        subprocess.check_call(cmd)
    except subprocess.CalledProcessError:
        # -march=native can be refused on exotic hosts; the plain build is always valid
        subprocess.check_call([c for c in cmd if c != "-march=native"])
    return LIB


if __name__ == "__main__":
    print(build(force=True))
