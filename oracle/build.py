"""Compile the CPU oracle (test infrastructure) into oracle/libsgemm_cube_oracle.so.

Flags matter for what the oracle means: no fast-math and no FMA contraction, so that every
FP32 operation in it is one IEEE round-to-nearest operation, and OpenMP only over independent
rows (no entry's summation order depends on the thread count).
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "sgemm_cube_oracle.cpp")
LIB = os.path.join(HERE, "libsgemm_cube_oracle.so")

FLAGS = ["-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
         "-shared", "-fPIC", "-std=c++17"]


def build(force: bool = False) -> str:
    if (not force and os.path.exists(LIB)
            and os.path.getmtime(LIB) >= os.path.getmtime(SRC)):
        return LIB
    tmp = LIB + ".tmp.%d" % os.getpid()
    subprocess.run(["g++", *FLAGS, SRC, "-o", tmp], check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
