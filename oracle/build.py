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
Q4_SRC = os.path.join(HERE, "q4_oracle.c")
Q4_HDR = os.path.join(HERE, "q4_oracle.h")
Q4_LIB = os.path.join(HERE, "libq4_oracle.so")


ENC_SRC = os.path.join(HERE, "tetra_encode_oracle.c")
ENC_HDR = os.path.join(HERE, "tetra_encode_oracle.h")
ENC_LIB = os.path.join(HERE, "libtetra_encode_oracle.so")


def _build_one(lib: str, src, hdr, force: bool, extra=()) -> str:
    srcs = [src] if isinstance(src, str) else list(src)
    hdrs = [hdr] if isinstance(hdr, str) else list(hdr)
    stale = (
        force
        or not os.path.exists(lib)
        or os.path.getmtime(lib) < max(os.path.getmtime(f) for f in srcs + hdrs)
    )
    if stale:
        tmp = lib + ".tmp.%d" % os.getpid()
        cmd = ["gcc", "-O2", "-std=c11", "-Wall", "-Wextra", *extra, "-fopenmp", "-shared", "-fPIC",
               "-o", tmp, *srcs, "-lm"]
        subprocess.run(cmd, check=True, cwd=HERE)
        os.replace(tmp, lib)
    return lib


def build(force: bool = False) -> str:
    """Build the Tetra oracle if it is missing or older than its sources."""
    return _build_one(LIB, SRC, HDR, force)


def build_q4(force: bool = False) -> str:
    """Build the 4-bit group-quantisation oracle likewise."""
    # -ffp-contract=off: every product and sum is rounded as written
    return _build_one(Q4_LIB, Q4_SRC, Q4_HDR, force, extra=("-ffp-contract=off",))


def build_encode(force: bool = False) -> str:
    """Build the encoder-search oracle (it calls the Tetra oracle's decoder, so both sources go in)."""
    return _build_one(ENC_LIB, [SRC, ENC_SRC], [HDR, ENC_HDR], force)


if __name__ == "__main__":
    print(build(force=True))
    print(build_q4(force=True))
    print(build_encode(force=True))
