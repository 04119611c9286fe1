"""Compile the CPU oracle (test infrastructure) into oracle/libl2kv_oracle.so.

Plain g++: no CUDA, no flags that relax floating-point semantics, and
floating-point contraction switched off so that every sum is the one written
in the source.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "l2kv_oracle.cpp")
LIB = os.path.join(HERE, "libl2kv_oracle.so")


def build(force: bool = False) -> str:
    if (not force and os.path.exists(LIB)
            and os.path.getmtime(LIB) >= os.path.getmtime(SRC)):
        return LIB
    cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fPIC", "-shared", "-pthread",
           "-Wall", "-Wextra", "-o", LIB, SRC]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))
