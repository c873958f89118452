"""Compile the C oracle into oracle/libtetra_oracle.so (test infrastructure only).

Building the checker is not using it: the CUDA library neither links nor loads
this file.
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "tetra_oracle.c")
HDR = os.path.join(HERE, "tetra_oracle.h")
LIB = os.path.join(HERE, "libtetra_oracle.so")


def build(force: bool = False) -> str:
    """Build the shared object if it is missing or older than its sources."""
    stale = (
        force
        or not os.path.exists(LIB)
        or os.path.getmtime(LIB) < max(os.path.getmtime(SRC), os.path.getmtime(HDR))
    )
    if stale:
        tmp = LIB + ".tmp.%d" % os.getpid()
        cmd = ["gcc", "-O2", "-std=c11", "-Wall", "-Wextra", "-fopenmp", "-shared", "-fPIC",
               "-o", tmp, SRC, "-lm"]
        subprocess.run(cmd, check=True, cwd=HERE)
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
