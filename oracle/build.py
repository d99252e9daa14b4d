"""Builds the CPU oracle (test infrastructure) into oracle/libhadfl_oracle.so with g++.

-ffp-contract=off keeps the compiler from fusing multiply-adds on its own: the oracle fuses
exactly where it calls fmaf and nowhere else.  No OpenMP, no vectorisation flags: the oracle
is timed as it stands.  build(openmp=True) makes a second library, libhadfl_oracle_omp.so, from
the same source with -fopenmp (its column loops split over the host cores; same results bit for
bit), which only the benchmark's all-cores CPU baseline and its own test load.
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "hadfl_oracle.cpp")
LIB = os.path.join(HERE, "libhadfl_oracle.so")
LIB_OMP = os.path.join(HERE, "libhadfl_oracle_omp.so")


def build(force: bool = False, openmp: bool = False) -> str:
    lib = LIB_OMP if openmp else LIB
    if not force and os.path.exists(lib) and os.path.getmtime(lib) >= os.path.getmtime(SRC):
        return lib
    tmp = lib + ".tmp.%d" % os.getpid()
    cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fPIC", "-shared",
           "-Wall", "-Wextra"] + (["-fopenmp"] if openmp else []) + ["-o", tmp, SRC]
    subprocess.run(cmd, check=True)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force=True))
    print(build(force=True, openmp=True))
