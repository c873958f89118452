"""Python face of the 4-bit group-quantisation CPU oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.

Thin ctypes marshalling over ``q4_oracle.c`` (Sec. 4.1, 4.4, 5.1).  Only tests, the smoke check and the
bench harness's CPU legs may import it; the CUDA library and its binding never do.
"""
import ctypes as C

import numpy as np

from . import build as _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(_build.build_q4())
        lib.q4o_half_to_double.argtypes = [C.c_uint16]
        lib.q4o_half_to_double.restype = C.c_double
        lib.q4o_float_to_half.argtypes = [C.c_float]
        lib.q4o_float_to_half.restype = C.c_uint16
        lib.q4o_weight.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_size_t, C.c_int]
        lib.q4o_weight.restype = C.c_double
        lib.q4o_gemv.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                 C.c_int, C.c_void_p, C.c_void_p, C.c_int]
        lib.q4o_gemv.restype = C.c_int
        lib.q4o_rows.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                 C.c_int, C.c_void_p]
        lib.q4o_rows.restype = C.c_int
        _lib = lib
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def _u16(a):
    """float16 or uint16 array -> contiguous uint16 bit patterns."""
    a = np.ascontiguousarray(a)
    return a.view(np.uint16) if a.dtype == np.float16 else a.astype(np.uint16, copy=False)


def half_to_double(bits: int) -> float:
    return _load().q4o_half_to_double(int(bits))


def float_to_half(value: float) -> int:
    return _load().q4o_float_to_half(float(np.float32(value)))


def weight(q, scale, offset, K, G, n, k) -> float:
    q = np.ascontiguousarray(q, dtype=np.uint8)
    s, o = _u16(scale), _u16(offset)
    return _load().q4o_weight(_p(q), _p(s), _p(o), K, G, n, k)


def gemv(q, scale, offset, x, N, K, G, batch=1, threads=0, want_termnorm=True):
    """FP64 product; returns (y [batch, N], termnorm [batch, N] or None)."""
    q = np.ascontiguousarray(q, dtype=np.uint8)
    s, o, xx = _u16(scale), _u16(offset), _u16(x)
    if not (q.size == N * (K // 2) and s.size == N * (K // G) == o.size and xx.size == batch * K):
        raise ValueError("q4o_gemv: array sizes do not match N, K, G, batch")
    y = np.zeros((batch, N), dtype=np.float64)
    tn = np.zeros((batch, N), dtype=np.float64) if want_termnorm else None
    rc = _load().q4o_gemv(_p(q), _p(s), _p(o), _p(xx), N, K, G, batch, _p(y), _p(tn) if want_termnorm else None,
                          threads)
    if rc != 0:
        raise ValueError("q4o_gemv: bad size")
    return y, tn


def rows(q, scale, offset, ids, N, K, G):
    """float16 rows of the table for the given ids, [len(ids), K]."""
    q = np.ascontiguousarray(q, dtype=np.uint8)
    s, o = _u16(scale), _u16(offset)
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    out = np.zeros((len(ids), K), dtype=np.uint16)
    rc = _load().q4o_rows(_p(q), _p(s), _p(o), _p(ids), len(ids), N, K, G, _p(out))
    if rc == -2:
        raise IndexError("q4o_rows: id out of range")
    if rc != 0:
        raise ValueError("q4o_rows: bad size")
    return out.view(np.float16)
