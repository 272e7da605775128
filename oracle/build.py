"""Compiles the oracle (plain C++17, host only) into oracle/liboracle_ccld.so."""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "ccld_oracle.cpp")
LIB = os.path.join(HERE, "liboracle_ccld.so")


def build(force: bool = False) -> str:
    if force or not os.path.exists(LIB) or os.path.getmtime(LIB) < os.path.getmtime(SRC):
        subprocess.check_call(["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-Wall", "-o", LIB, SRC])
    return LIB


if __name__ == "__main__":
    print(build(force=True))
