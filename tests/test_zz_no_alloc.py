"""tetra_gemv_noalloc: the product for callers that cannot allocate device
memory (a plug-in under a host application's memory pool, a loop that may not
take the allocator's lock).  Its scratch buffer is a fixed array inside the
library, shared by all calls, so the checks here run two calls in a row, the
second on a different and smaller matrix, and compare each with the ordinary
entry point on the same inputs.  This file sorts last on purpose."""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2609_35465_b200 import synth
from helpers import assert_gemv_close, make_matrix, oracle_product

pytestmark = pytest.mark.gpu


def _device(tt, table, m):
    codes = torch.from_numpy(m["codes"]).cuda()
    return dict(codes=tt.tetra_pack_codes(codes, table, m["N"], m["B"]),
                sigma=torch.from_numpy(m["sigma"]).cuda(), x=torch.from_numpy(m["x"]).cuda(),
                tail=torch.from_numpy(m["tail"]).cuda() if m["tail"] is not None else None)


def test_noalloc_matches_the_ordinary_entry_point_twice_in_a_row(orc):
    from paper_2609_35465_b200 import tetra as tt
    table = tt.tetra_build_table(synth.DEFAULT_GAIN)
    cases = [make_matrix(41, 1, 1024, 4096, True),      # 170 words per row + a tail of 16
             make_matrix(41, 2, 520, 24 * 37, True)]    # smaller: most of the scratch keeps stale data
    for m in cases:
        d = _device(tt, table, m)
        want = torch.full((1, m["N"]), float("nan"), dtype=torch.float32, device="cuda")
        got = torch.full((1, m["N"]), float("nan"), dtype=torch.float32, device="cuda")
        tt.tetra_gemv_tail(d["codes"], d["sigma"], table, d["x"], want, m["N"], m["K"], 1, d["tail"])
        tt.tetra_gemv_noalloc(d["codes"], d["sigma"], table, d["x"], got, m["N"], m["K"], d["tail"])
        torch.cuda.synchronize()
        a, b = want.cpu().numpy()[0].astype(np.float64), got.cpu().numpy()[0].astype(np.float64)
        assert np.isfinite(b).all()
        # the two entry points sum in different orders: equal up to float32 rounding
        assert np.linalg.norm(a - b) <= 1e-5 * np.linalg.norm(a)
        assert np.max(np.abs(a - b)) <= 1e-4 * np.max(np.abs(a))
        # and each against the FP64 oracle, within the tolerance of the GEMV tests
        ref = oracle_product(orc, m, synth.DEFAULT_GAIN)
        assert_gemv_close(b, ref, "noalloc %dx%d" % (m["N"], m["K"]))
        assert_gemv_close(a, ref, "ordinary %dx%d" % (m["N"], m["K"]))


def test_noalloc_rejects_sizes_beyond_its_fixed_scratch():
    from paper_2609_35465_b200 import tetra as tt
    table = tt.tetra_build_table(synth.DEFAULT_GAIN)
    buf = torch.zeros(64, dtype=torch.uint8, device="cuda")
    rc = tt.lib().tetra_gemv_noalloc(C.c_void_p(buf.data_ptr()), C.c_void_p(buf.data_ptr()),
                                     C.c_void_p(table.data_ptr()), C.c_void_p(buf.data_ptr()),
                                     C.c_void_p(buf.data_ptr()), 8, tt.NOALLOC_MAX_K + 24, None, None)
    assert rc == -6
    # a tail pointer with K < 24 leaves no whole word in a row: rejected like tetra_gemv_tail does
    rc = tt.lib().tetra_gemv_noalloc(C.c_void_p(buf.data_ptr()), C.c_void_p(buf.data_ptr()),
                                     C.c_void_p(table.data_ptr()), C.c_void_p(buf.data_ptr()),
                                     C.c_void_p(buf.data_ptr()), 8, 16, C.c_void_p(buf.data_ptr()), None)
    assert rc == -2
