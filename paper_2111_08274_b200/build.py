"""Builds the C-ABI library (CUDA kernels for sm_100a) in-tree: paper_2111_08274_b200/libhadfl.so.

nvcc cross-compiles without a GPU.  The CUDA runtime is linked statically so that the library
loads (and its host-only functions run) on a machine without a driver.  -fmad=false and
-ffp-contract=off: the code fuses multiply-adds exactly where it calls fmaf and nowhere else.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libhadfl.so")
LIB_DEBUG = os.path.join(HERE, "libhadfl_debug.so")   # -DHADFL_DEBUG: bounds-checked kernels
SOURCES = ["hadfl.cu", "selection.cpp"]
DEPS = SOURCES + ["kernels.cuh", "philox.cuh", "debug_check.cuh", "selection.h",
                  os.path.join("..", "..", "include", "hadfl.h")]


def nvcc_path() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    return "nvcc"


def up_to_date(lib: str) -> bool:
    if not os.path.exists(lib):
        return False
    t = os.path.getmtime(lib)
    return all(os.path.getmtime(os.path.join(CSRC, d)) <= t for d in DEPS)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    lib = LIB_DEBUG if debug else LIB
    if not force and up_to_date(lib):
        return lib
    tmp = lib + ".tmp.%d" % os.getpid()
    cmd = [nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3",
           "-std=c++17", "-shared", "-Xcompiler", "-fPIC,-ffp-contract=off",
           "-cudart", "static", "-fmad=false", "-o", tmp]
    if debug:
        cmd += ["-DHADFL_DEBUG"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.run(cmd, check=True)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
