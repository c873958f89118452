"""tetra_gemv_batched (decode once, tensor-core contraction per block) against the FP64 oracle."""
import numpy as np
import pytest
import torch

from paper_2609_35465_b200 import shapes, synth
from helpers import assert_gemv_close, make_matrix, oracle_product

pytestmark = pytest.mark.gpu
GAIN = synth.DEFAULT_GAIN


@pytest.fixture(scope="module")
def tt():
    from paper_2609_35465_b200 import tetra
    return tetra


@pytest.fixture(scope="module")
def table(tt):
    return tt.tetra_build_table(GAIN)


def run(tt, table, m):
    batch = m["x"].shape[0]
    codes = tt.tetra_pack_codes(torch.from_numpy(m["codes"]).cuda(), table, m["N"], m["B"])
    sigma = torch.from_numpy(m["sigma"]).cuda()
    x = torch.from_numpy(m["x"]).cuda()
    tail = torch.from_numpy(m["tail"]).cuda() if m["tail"] is not None else None
    y = torch.full((batch, m["N"]), float("nan"), dtype=torch.float32, device="cuda")
    tt.tetra_gemv_batched(codes, sigma, table, x, y, m["N"], m["K"], batch, tail)
    torch.cuda.synchronize()
    return y.cpu().numpy()


@pytest.mark.parametrize("N,K,tail_mode,batch", [
    (256, 2560, True, 2), (256, 2560, True, 5), (256, 2560, True, 8), (256, 2560, True, 16),
    (520, 4096, True, 16), (33, 24 * 31 + 5, True, 3), (33, 24 * 31 + 5, False, 9), (7, 48, True, 16),
    (1, 24, True, 1), (72, 17408, True, 12), (2048, 2304, True, 4), (40, 49152, True, 3), (24, 49152, True, 16),
])
def test_batched_matches_oracle(tt, table, orc, N, K, tail_mode, batch):
    m = make_matrix(51, N * 3 + K + batch, N, K, tail_mode, batch=batch)
    y = run(tt, table, m)
    assert np.isfinite(y).all()
    for b in range(batch):
        ref = oracle_product(orc, m, GAIN, batch_index=b)
        assert_gemv_close(y[b], ref, "batched %dx%d vector %d/%d" % (N, K, b, batch))
        assert np.max(np.abs(y[b] - ref["y"]) / ref["abssum"]) < 1e-5


def test_batched_agrees_with_the_batch1_path(tt, table):
    m = make_matrix(52, 1, 512, 4096, True, batch=6)
    yb = run(tt, table, m)
    codes = tt.tetra_pack_codes(torch.from_numpy(m["codes"]).cuda(), table, m["N"], m["B"])
    y1 = torch.empty((6, m["N"]), dtype=torch.float32, device="cuda")
    tt.tetra_gemv_tail(codes, torch.from_numpy(m["sigma"]).cuda(), table, torch.from_numpy(m["x"]).cuda(), y1,
                       m["N"], m["K"], 6, torch.from_numpy(m["tail"]).cuda())
    torch.cuda.synchronize()
    y1 = y1.cpu().numpy()
    assert np.linalg.norm(yb - y1) <= 1e-5 * np.linalg.norm(y1)


def test_batched_vectors_with_very_different_magnitudes(tt, table, orc):
    """Every vector has its own fixed-point step per block column: a vector 4096 times smaller than its
    neighbour keeps full precision."""
    m = make_matrix(53, 2, 128, 1200, True, batch=4)
    m["x"][1] = (m["x"][1].astype(np.float32) / 4096).astype(np.float16)
    m["x"][2] = (m["x"][2].astype(np.float32) * 512).astype(np.float16)
    y = run(tt, table, m)
    for b in range(4):
        ref = oracle_product(orc, m, GAIN, batch_index=b)
        assert_gemv_close(y[b], ref, "vector %d" % b)
        assert np.max(np.abs(y[b] - ref["y"]) / ref["abssum"]) < 1e-5


def test_batched_argument_checks(tt, table):
    import ctypes as C
    buf = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    p = C.c_void_p(buf.data_ptr())
    L = tt.lib()
    assert L.tetra_gemv_batched(p, p, C.c_void_p(table.data_ptr()), p, p, 8, 24, 17, None, p, 4096, None) == -4
    assert L.tetra_gemv_batched(p, p, C.c_void_p(table.data_ptr()), p, p, 8, 24, 2, None, None, 0, None) == -1
    assert L.tetra_gemv_batched(p, p, C.c_void_p(table.data_ptr()), p, p, 8, 24, 2, None, p, 16, None) == -6
    assert tt.tetra_batched_workspace_bytes(4096, 12288) >= 512 * 1600
