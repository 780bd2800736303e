"""Compile the CPU oracle (test infrastructure) into oracle/libq8_oracle.so.

Flags: -O2, no floating-point contraction and no fast-math, so that every fp32
step is one correctly rounded IEEE operation as the oracle's comments state.
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRCS = [os.path.join(HERE, "q8_oracle.cpp"), os.path.join(HERE, "q8_oracle_detect.cpp")]
LIB = os.path.join(HERE, "libq8_oracle.so")


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and all(os.path.getmtime(LIB) >= os.path.getmtime(s) for s in SRCS):
        return LIB
    cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
           "-pthread", *SRCS, "-o", LIB]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
