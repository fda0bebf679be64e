"""Compile the C++ oracle into oracle/librekv_oracle.so (g++, OpenMP)."""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "rekv_oracle.cpp")
LIB = os.path.join(HERE, "librekv_oracle.so")


def build(force: bool = False) -> str:
    if force or not os.path.exists(LIB) or os.path.getmtime(LIB) < os.path.getmtime(SRC):
        subprocess.check_call(
            ["g++", "-std=c++17", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", LIB, SRC])
    return LIB


if __name__ == "__main__":
    print(build(force=True))
