"""CPU-side checks of the C-ABI library: it loads, exports every symbol the
header declares, rejects bad arguments on the host, and builds the same tables
as the oracle (bit for bit)."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2609_35465_b200 import build as tbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    tbuild.build()
    from paper_2609_35465_b200 import tetra
    return tetra.lib()


def declared_functions():
    inc = os.path.join(ROOT, "include")
    src = "".join(open(os.path.join(inc, f)).read() for f in sorted(os.listdir(inc)) if f.endswith(".h"))
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(tetra_[a-z_0-9]+)\s*\(", src)))


def test_every_declared_symbol_is_exported(L):
    names = declared_functions()
    assert "tetra_gemv" in names and "tetra_build_table" in names and "tetra_decode_blocks" in names
    for n in names:
        assert hasattr(L, n), n


def test_table_export_equals_oracle_blob(L, orc):
    from paper_2609_35465_b200 import tetra
    assert tetra.tetra_table_export() == orc.table_blob()
    assert tetra.tetra_table_bytes() >= 18816 + 8


def test_host_side_argument_checks(L):
    buf = (C.c_uint8 * 64)()
    p = C.addressof(buf)
    p16 = (p + 15) & ~15
    assert L.tetra_gemv(None, p16, p16, p16, p16, 8, 24, 1, None) == -1            # null
    assert L.tetra_gemv(p16, p16, p16, p16, p16, 0, 24, 1, None) == -2             # shape
    assert L.tetra_gemv(p16, p16, p16, p16, p16, 8, 24, 17, None) == -4            # batch
    assert L.tetra_gemv(p16 + 4, p16, p16, p16, p16, 8, 24, 1, None) == -3         # alignment of codes
    assert L.tetra_gemv(p16, p16, p16, p16, p16, 8, 24 * 4096, 1, None) == -2      # K too large
    assert L.tetra_decode_blocks(None, p16, p16, None, 4, None) == -1
    assert L.tetra_decode_blocks(None, None, None, None, 0, None) == 0                # empty input
    assert L.tetra_decode_blocks(p16 + 1, p16, p16, None, 4, None) == -3
    assert L.tetra_pack_codes(p16, p16, p16, 8, 0, None) == -2
    assert L.tetra_build_table(p16, 16, None, None) == -6                          # blob too small
    assert L.tetra_table_export(p16, 10) == -6
    assert L.tetra_gemv_grouped(None, 1, p16, p16, 48, None) == -1
    assert L.tetra_gemv_list(None, 1, p16, None) == -1                               # no descriptors
    assert L.tetra_gemv_list(p16, 1, None, None) == -1                               # no table
    assert L.tetra_gemv_list(p16, 9, p16, None) in (-1, -2)                          # zeroed descriptors / too long
    assert L.tetra_gemv_grouped_run(None, p16, None) == -1
    assert L.tetra_codes_bytes(4096, 170) == 4096 * 170 * 6
    assert L.tetra_codes_bytes(9, 3) == 2 * 48 * 3                                  # rows pad to 8
    assert L.tetra_status_string(-3) == b"misaligned pointer"


def test_product_path_has_no_cpu_fallback():
    """The package never imports the oracle."""
    pkg = os.path.join(ROOT, "paper_2609_35465_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".cpp", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text and "tetra_oracle" not in text, f
