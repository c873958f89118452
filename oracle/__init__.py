"""Python face of the Tetra CPU oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.

Thin ctypes marshalling over ``tetra_oracle.c``; every number comes from the C
code, which restates the paper's definitions (Sec. 3.1-3.4, Eq. (1)-(3),
Sec. 5.1) one step at a time.  Only tests, the smoke check and the bench
harness's CPU-baseline leg may import this package; the CUDA library and its
Python binding never do.
"""
import ctypes as C

import numpy as np

from . import build as _build

NCODE = 4096
NROWS = 4096
HALF = 2048
BLOB_BYTES = 18816


class _Tables(C.Structure):
    _fields_ = [
        ("golay", C.c_uint32 * NCODE),
        ("prefixes", C.c_uint8 * 128),
        ("branches", C.c_uint16 * 1024),
        ("suffixes", C.c_uint8 * 128),
        ("rows", C.c_uint32 * NROWS),
        ("n0", C.c_int32),
        ("val", (C.c_int8 * 8) * 4),
    ]


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(_build.build())
        P = C.POINTER
        lib.to_build_tables.argtypes = [P(_Tables)]
        lib.to_build_tables.restype = C.c_int
        lib.to_row_cost.argtypes = [C.c_uint32]
        lib.to_row_cls.argtypes = [C.c_uint32]
        lib.to_rank_value.argtypes = [C.c_int, C.c_int]
        lib.to_mix.argtypes = [P(_Tables), C.c_int, P(C.c_int)]
        lib.to_decode_section.argtypes = [P(_Tables), C.c_int, C.c_int, C.c_uint32, C.c_void_p]
        lib.to_decode_section.restype = None
        lib.to_decode_word.argtypes = [P(_Tables), C.c_uint64, C.c_void_p, P(C.c_int), P(C.c_int)]
        lib.to_decode_word.restype = None
        lib.to_decode_blocks.argtypes = [P(_Tables), C.c_void_p, C.c_size_t,
                                         C.c_void_p, C.c_void_p, C.c_void_p]
        lib.to_decode_blocks.restype = None
        lib.to_in_leech.argtypes = [P(_Tables), C.c_void_p]
        lib.to_table_blob.argtypes = [P(_Tables), C.c_void_p]
        lib.to_table_blob.restype = None
        lib.to_gemv.argtypes = [P(_Tables), C.c_void_p, C.c_size_t, C.c_int, C.c_int,
                                C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                                C.c_void_p, C.c_void_p, C.c_void_p, C.c_int]
        lib.to_gemv.restype = C.c_int
        _lib = lib
    return _lib


class Oracle:
    """The oracle's tables plus the calls that read them."""

    def __init__(self):
        self._lib = _load()
        self._t = _Tables()
        rc = self._lib.to_build_tables(C.byref(self._t))
        if rc != 0:
            raise RuntimeError("oracle table build failed: %d" % rc)

    # ---- tables -----------------------------------------------------
    @property
    def golay(self):
        return np.ctypeslib.as_array(self._t.golay).copy()

    @property
    def prefixes(self):
        return np.ctypeslib.as_array(self._t.prefixes).copy()

    @property
    def branches(self):
        return np.ctypeslib.as_array(self._t.branches).copy()

    @property
    def suffixes(self):
        return np.ctypeslib.as_array(self._t.suffixes).copy()

    @property
    def rows(self):
        return np.ctypeslib.as_array(self._t.rows).copy()

    @property
    def n0(self):
        return int(self._t.n0)

    def table_blob(self) -> bytes:
        buf = (C.c_uint8 * BLOB_BYTES)()
        self._lib.to_table_blob(C.byref(self._t), buf)
        return bytes(buf)

    # ---- scalar pieces ----------------------------------------------
    def row_cost(self, row: int) -> int:
        return self._lib.to_row_cost(row)

    def row_cls(self, row: int) -> int:
        return self._lib.to_row_cls(row)

    def rank_value(self, o: int, rho: int) -> int:
        return self._lib.to_rank_value(o, rho)

    def mix(self, i2: int):
        d = C.c_int()
        idx = self._lib.to_mix(C.byref(self._t), i2, C.byref(d))
        return idx, d.value

    def decode_section(self, p: int, cbyte: int, row: int) -> np.ndarray:
        y = np.zeros(8, dtype=np.int8)
        self._lib.to_decode_section(C.byref(self._t), p, cbyte, row, y.ctypes.data)
        return y

    def decode_word(self, word: int):
        y = np.zeros(24, dtype=np.int8)
        m, g = C.c_int(), C.c_int()
        self._lib.to_decode_word(C.byref(self._t), word, y.ctypes.data, C.byref(m), C.byref(g))
        return y, m.value, g.value

    def in_leech(self, y) -> bool:
        y = np.ascontiguousarray(y, dtype=np.int8)
        assert y.shape == (24,)
        return bool(self._lib.to_in_leech(C.byref(self._t), y.ctypes.data))

    # ---- bulk ----------------------------------------------------------
    def decode_blocks(self, codes: np.ndarray):
        """codes: uint8 [n, 6] -> (y int8 [n, 24], m uint8 [n], g uint8 [n])."""
        codes = np.ascontiguousarray(codes, dtype=np.uint8).reshape(-1, 6)
        n = codes.shape[0]
        y = np.zeros((n, 24), dtype=np.int8)
        m = np.zeros(n, dtype=np.uint8)
        g = np.zeros(n, dtype=np.uint8)
        self._lib.to_decode_blocks(C.byref(self._t), codes.ctypes.data, n,
                                   y.ctypes.data, m.ctypes.data, g.ctypes.data)
        return y, m, g

    def gemv(self, codes: np.ndarray, sigma, gain, x, tail=None, threads: int = 1):
        """FP64 product.  codes: uint8 [N, row_stride] (block b at byte 6 b);
        x: length 24 B + ntail, any float dtype (promoted exactly to double).
        Returns dict(y, termnorm, abssum, threads)."""
        codes = np.ascontiguousarray(codes, dtype=np.uint8)
        N, stride = codes.shape
        sigma = np.ascontiguousarray(sigma, dtype=np.float32)
        gain = np.ascontiguousarray(gain, dtype=np.float32)
        x = np.ascontiguousarray(x, dtype=np.float64)
        ntail = 0
        tail_p = None
        if tail is not None:
            tail = np.ascontiguousarray(tail, dtype=np.float64).reshape(N, -1)
            ntail = tail.shape[1]
            tail_p = tail.ctypes.data if ntail else None
        B = (x.shape[0] - ntail) // 24
        assert 24 * B + ntail == x.shape[0] and 6 * B <= stride and sigma.shape == (N,)
        out = np.zeros(N, dtype=np.float64)
        tn = np.zeros(N, dtype=np.float64)
        ab = np.zeros(N, dtype=np.float64)
        used = self._lib.to_gemv(C.byref(self._t), codes.ctypes.data, stride, N, B,
                                 sigma.ctypes.data, gain.ctypes.data, x.ctypes.data,
                                 tail_p, ntail, out.ctypes.data, tn.ctypes.data,
                                 ab.ctypes.data, threads)
        return {"y": out, "termnorm": tn, "abssum": ab, "threads": used}


_singleton = None


def get() -> Oracle:
    """A process-wide oracle instance (table build takes about a second)."""
    global _singleton
    if _singleton is None:
        _singleton = Oracle()
    return _singleton
