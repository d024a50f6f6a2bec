"""Compile the CPU oracle (plain C, gcc) into oracle/libpq_oracle.so.

Test infrastructure: building the checker is not using it.  -ffp-contract=off keeps gcc from
fusing a*b+c on its own, so a fused multiply-add happens only where the source writes fmaf().
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "pq_oracle.c")
LIB = os.path.join(HERE, "libpq_oracle.so")


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    cmd = ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-fPIC",
           "-shared", "-Wall", "-Wextra", "-o", LIB, SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
