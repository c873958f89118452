"""Python face of the encoder-search CPU oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.

Thin ctypes marshalling over ``tetra_encode_oracle.c`` (Sec. 3.1, Eq. (2)).  Only tests, the smoke check and
the bench harness's CPU legs may import it.
"""
import ctypes as C

import numpy as np

from . import _Tables
from . import build as _build

_lib = None
_tables = None


def _load():
    global _lib, _tables
    if _lib is None:
        lib = C.CDLL(_build.build_encode())
        P = C.POINTER
        lib.to_build_tables.argtypes = [P(_Tables)]
        lib.to_build_tables.restype = C.c_int
        lib.to_encode_block.argtypes = [P(_Tables), C.c_void_p, C.c_int, P(C.c_uint64), P(C.c_double)]
        lib.to_encode_block.restype = C.c_int
        lib.to_choose_gain.argtypes = [C.c_double, C.c_double, C.c_void_p]
        lib.to_choose_gain.restype = C.c_int
        lib.to_encode_blocks.argtypes = [P(_Tables), C.c_void_p, C.c_size_t, C.c_int, C.c_double, C.c_void_p,
                                         C.c_void_p, C.c_void_p, C.c_int]
        lib.to_encode_blocks.restype = C.c_int
        tables = _Tables()
        if lib.to_build_tables(C.byref(tables)) != 0:
            raise RuntimeError("to_build_tables failed")
        _lib, _tables = lib, tables
    return _lib, _tables


def encode_blocks(w, sigma=1.0, gain=(1.0, 1.0), row_limit=2048, threads=0):
    """w: [n, 24] float64 -> (words uint64 [n] with the gain bit, cosines float64 [n])."""
    lib, tables = _load()
    w = np.ascontiguousarray(w, dtype=np.float64).reshape(-1, 24)
    g = np.ascontiguousarray(gain, dtype=np.float64)
    words = np.zeros(len(w), dtype=np.uint64)
    cos = np.zeros(len(w), dtype=np.float64)
    rc = lib.to_encode_blocks(C.byref(tables), w.ctypes.data_as(C.c_void_p), len(w), row_limit, float(sigma),
                              g.ctypes.data_as(C.c_void_p), words.ctypes.data_as(C.c_void_p),
                              cos.ctypes.data_as(C.c_void_p), threads)
    if rc != 0:
        raise ValueError("to_encode_blocks: bad row_limit")
    return words, cos


def choose_gain(c, sigma, gain):
    lib, _ = _load()
    g = np.ascontiguousarray(gain, dtype=np.float64)
    return lib.to_choose_gain(float(c), float(sigma), g.ctypes.data_as(C.c_void_p))
