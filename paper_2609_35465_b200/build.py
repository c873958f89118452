"""Builds the CUDA library in-tree: paper_2609_35465_b200/libtetra_b200.so (sm_100a).

nvcc cross-compiles without a GPU.  Run:  python -m paper_2609_35465_b200.build
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libtetra_b200.so")
SOURCES = ["tetra_tables.cpp", "tetra_decode.cu", "tetra_gemv.cu", "tetra_list.cu", "tetra_batched.cu", "tetra_api.cu", "tetra_noalloc.cu", "q4_gemv.cu", "q4_list.cu", "tetra_encode.cu"]
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
         "-Xcompiler", "-fPIC", "-Xcompiler", "-Wall", "--use_fast_math"]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    deps.append(os.path.join(os.path.dirname(HERE), "include", "tetra.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not (force or _stale()):
        return LIB
    flags = list(FLAGS) + os.environ.get("TETRA_EXTRA_FLAGS", "").split()
    if verbose:
        flags += ["-Xptxas", "-v"]
    objs = []
    procs = []
    for src in SOURCES:
        obj = os.path.join(CSRC, os.path.splitext(src)[0] + ".o")
        objs.append(obj)
        procs.append(subprocess.Popen([NVCC] + flags + ["-c", os.path.join(CSRC, src), "-o", obj], cwd=CSRC))
    if any(p.wait() != 0 for p in procs):
        raise RuntimeError("nvcc failed")
    tmp = LIB + ".tmp.%d" % os.getpid()
    subprocess.run([NVCC, "-shared", "-o", tmp] + objs + ["-lcudart"], check=True, cwd=CSRC)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
