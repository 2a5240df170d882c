"""Compiles the C++ oracle into ``oracle/liblc_oracle.so`` with g++ (no CUDA involved)."""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "lc_oracle.cpp")
LIB = os.path.join(HERE, "liblc_oracle.so")

# -ffp-contract=off: the fp32 subtract and add of Algorithm 1 must stay plain IEEE operations.
FLAGS = ["-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared", "-pthread", "-Wall", "-Wextra"]


def build(force: bool = False) -> str:
    if force or not os.path.exists(LIB) or os.path.getmtime(LIB) < os.path.getmtime(SRC):
        tmp = LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["g++", *FLAGS, "-o", tmp, SRC])
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
