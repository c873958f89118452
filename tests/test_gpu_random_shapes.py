"""Seeded random shapes through every GEMV entry point against the FP64 oracle: sizes that no hand-picked
case names (odd row counts, K around multiples of 24 and of 32 words, one-row and one-word matrices, both
tail rules, random list compositions and batch sizes).  Each entry point sees the same matrices."""
import numpy as np
import pytest
import torch

from paper_2609_35465_b200 import synth
from helpers import assert_gemv_close, make_matrix, oracle_product
from test_gpu_gemv import upload

pytestmark = pytest.mark.gpu
GAIN = synth.DEFAULT_GAIN


@pytest.fixture(scope="module")
def tt():
    from paper_2609_35465_b200 import tetra
    return tetra


@pytest.fixture(scope="module")
def table(tt):
    return tt.tetra_build_table(GAIN)


def random_shape(rng):
    """(N, K, tail_mode): mostly small, sometimes wide or tall, K near the boundaries that matter."""
    kind = rng.integers(0, 6)
    if kind == 0:
        N, words = int(rng.integers(1, 40)), int(rng.integers(1, 70))
    elif kind == 1:
        N, words = int(rng.integers(1, 600)), int(rng.integers(1, 200))
    elif kind == 2:
        N, words = int(rng.integers(1, 64)), int(rng.choice([31, 32, 33, 63, 64, 65, 127, 128, 129, 511, 512, 513]))
    elif kind == 3:
        N, words = int(rng.choice([7, 8, 9, 15, 16, 17, 31, 32, 33, 255, 256, 257, 511, 512, 513])), int(rng.integers(1, 90))
    elif kind == 4:
        N, words = int(rng.integers(1, 24)), int(rng.integers(600, 2048))
    else:
        N, words = int(rng.integers(600, 1500)), int(rng.integers(1, 48))
    extra = int(rng.choice([0, 0, 1, 5, 8, 16, 23]))
    tail_mode = bool(rng.integers(0, 2))
    K = 24 * words + extra
    if K > 49152:
        K = 49152
    return N, K, tail_mode


def check(m, y, orc, what, batch_index=0):
    ref = oracle_product(orc, m, GAIN, batch_index=batch_index)
    assert_gemv_close(y, ref, what)


@pytest.mark.parametrize("seed", range(12))
def test_random_single_matrices_on_every_entry_point(tt, table, orc, seed):
    rng = np.random.default_rng(1000 + seed)
    for case in range(5):
        N, K, tail_mode = random_shape(rng)
        batch = int(rng.choice([1, 1, 2, 3, 5, 8, 11, 16]))
        m = make_matrix(71, 97 * seed + case, N, K, tail_mode, batch=batch)
        d = upload(tt, table, m)
        what = "%dx%d tail_mode=%s batch %d" % (N, K, tail_mode, batch)
        # the spec call, all vectors
        if m["ntail"]:
            tt.tetra_gemv_tail(d["codes"], d["row_scales"], table, d["x"], d["y"], N, K, batch, d["tail"])
        else:
            tt.tetra_gemv(d["codes"], d["row_scales"], table, d["x"], d["y"], N, K, batch)
        torch.cuda.synchronize()
        y = d["y"].cpu().numpy()
        for b in range(batch):
            check(m, y[b], orc, "tetra_gemv " + what, b)
        # the batched call
        d["y"].fill_(float("nan"))
        tt.tetra_gemv_batched(d["codes"], d["row_scales"], table, d["x"], d["y"], N, K, batch, d["tail"])
        torch.cuda.synchronize()
        y = d["y"].cpu().numpy()
        for b in range(batch):
            check(m, y[b], orc, "tetra_gemv_batched " + what, b)
        # the planned list of one (first vector), the no-allocation call (first vector, K within its limit)
        d["y"].fill_(float("nan"))
        pr = tt.make_problems([d])
        ws = torch.empty(max(16, tt.tetra_grouped_workspace_bytes(pr)), dtype=torch.uint8, device="cuda")
        tt.tetra_gemv_grouped(pr, table, ws)
        torch.cuda.synchronize()
        check(m, d["y"].cpu().numpy()[0], orc, "tetra_gemv_grouped " + what)
        if K <= 24576:
            d["y"].fill_(float("nan"))
            tt.tetra_gemv_noalloc(d["codes"], d["row_scales"], table, d["x"], d["y"], N, K, d["tail"])
            torch.cuda.synchronize()
            check(m, d["y"].cpu().numpy()[0], orc, "tetra_gemv_noalloc " + what)


@pytest.mark.parametrize("seed", range(8))
def test_random_lists(tt, table, orc, seed):
    rng = np.random.default_rng(2000 + seed)
    for case in range(3):
        count = int(rng.integers(1, 9))
        shapes_list = [random_shape(rng) for _ in range(count)]
        mats = [make_matrix(72, 1000 * seed + 10 * case + i, N, K, tm) for i, (N, K, tm) in enumerate(shapes_list)]
        devs = [upload(tt, table, m) for m in mats]
        pr = tt.make_problems(devs)
        tt.tetra_gemv_list(pr, table)
        torch.cuda.synchronize()
        for m, d in zip(mats, devs):
            check(m, d["y"].cpu().numpy()[0], orc, "list of %d: %dx%d" % (count, m["N"], m["K"]))
            d["y"].fill_(float("nan"))
        ws = torch.empty(max(16, tt.tetra_grouped_workspace_bytes(pr)), dtype=torch.uint8, device="cuda")
        tt.tetra_gemv_grouped(pr, table, ws)
        torch.cuda.synchronize()
        for m, d in zip(mats, devs):
            check(m, d["y"].cpu().numpy()[0], orc, "planned list of %d: %dx%d" % (count, m["N"], m["K"]))
