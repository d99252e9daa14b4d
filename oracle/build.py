"""Builds the CPU oracle (test infrastructure) into oracle/libhadfl_oracle.so with g++.

-ffp-contract=off keeps the compiler from fusing multiply-adds on its own: the oracle fuses
exactly where it calls fmaf and nowhere else.  No OpenMP, no vectorisation flags: the oracle
is timed as it stands.
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "hadfl_oracle.cpp")
LIB = os.path.join(HERE, "libhadfl_oracle.so")


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    tmp = LIB + ".tmp.%d" % os.getpid()
    cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fPIC", "-shared",
           "-Wall", "-Wextra", "-o", tmp, SRC]
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
