"""Builds the oracle (test infrastructure) into oracle/libenec_oracle.so with g++. No CUDA involved."""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "enec_oracle.cpp")
LIB = os.path.join(HERE, "libenec_oracle.so")


def build(force: bool = False) -> str:
    deps = [SRC, os.path.join(HERE, "enec_oracle.h")]
    if (not force and os.path.exists(LIB)
            and all(os.path.getmtime(LIB) >= os.path.getmtime(d) for d in deps)):
        return LIB
    cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fPIC", "-shared", "-Wall", "-Wextra",
           "-o", LIB, SRC]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))
