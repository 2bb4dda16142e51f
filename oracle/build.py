"""Compile the CPU oracle (test infrastructure) into oracle/liboracle_bitlinear.so with g++."""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "bitlinear_oracle.cpp")
LIB = os.path.join(HERE, "liboracle_bitlinear.so")


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    cmd = ["g++", "-O3", "-std=c++17", "-fopenmp", "-fno-fast-math", "-ffp-contract=off",
           "-shared", "-fPIC", SRC, "-o", LIB]
    subprocess.check_call(cmd)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
