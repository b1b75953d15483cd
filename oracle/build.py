"""Compile the CPU oracle (plain C) into oracle/libmpe_oracle.so.

Test infrastructure: the oracle is built with FMA contraction off and without
fast-math so that every FP32 operation is the one written in the source.
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "mpe_oracle.c")
LIB = os.path.join(HERE, "libmpe_oracle.so")


def build(force: bool = False) -> str:
    deps = [SRC, os.path.join(HERE, "mpe_oracle.h")]
    if not force and os.path.exists(LIB) and all(os.path.getmtime(LIB) >= os.path.getmtime(p) for p in deps):
        return LIB
    cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
           "-Wall", "-Wextra", "-o", LIB, SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
