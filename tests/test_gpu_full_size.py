"""Parity at the benchmark's full sizes, in the launch configuration bench.py
times (a planned list run by tetra_gemv_grouped_run), on sampled output rows
the oracle computes one by one; plus properties that hold at any size."""
import numpy as np
import pytest
import torch

from paper_2609_35465_b200 import shapes, synth
from helpers import assert_gemv_close, make_matrix, oracle_product

pytestmark = pytest.mark.gpu


def _check_sampled(dp, orc, picks, rows_per_matrix=6, seed=0):
    rng = np.random.default_rng(seed)
    y_all = dp.y_all.cpu().numpy()
    worst = 0.0
    for i in picks:
        it = dp.items[i]
        rows = np.unique(np.concatenate([[0, it["N"] - 1], rng.integers(0, it["N"], rows_per_matrix)]))
        m = dp.host_inputs(i, rows=rows)
        ref = oracle_product(orc, m, dp.gain, threads=1)
        y = y_all[it["yoff"]:it["yoff"] + it["N"]][rows]
        _, w = assert_gemv_close(y, ref, it["name"])
        worst = max(worst, w)
    return worst


def test_qwen3_8b_full_pass_sampled_rows(orc):
    """Config 2: all 252 matrices of the Qwen3-8B-shaped pass in one planned run."""
    from paper_2609_35465_b200.workload import DevicePass
    dp = DevicePass(shapes.QWEN3_8B.all_matrices(), seed=0)
    dp.y_all.fill_(float("nan"))
    dp.run_grouped()
    torch.cuda.synchronize()
    y = dp.y_all.cpu().numpy()
    used = np.zeros(len(y), dtype=bool)
    for it in dp.items:
        used[it["yoff"]:it["yoff"] + it["N"]] = True
    assert np.isfinite(y[used]).all()                     # every output row was written
    assert dp.algorithmic_bytes == 1785397248
    picks = list(range(7)) + [7 * 17 + k for k in range(7)] + list(range(245, 252))
    _check_sampled(dp, orc, picks)
    # rerun: bit-identical (fixed summation order, no atomics)
    dp.run_grouped()
    torch.cuda.synchronize()
    assert np.array_equal(dp.y_all.cpu().numpy()[used], y[used])
    # the host-buffer entry point gives the same bits
    dp.y_all.zero_()
    dp.run_grouped_hostio()
    torch.cuda.synchronize()
    assert np.array_equal(dp.y_host.numpy()[used], y[used])


def test_qwen3_14b_full_pass_sampled_rows(orc):
    """Config 3: all 280 matrices of the Qwen3-14B-shaped pass (hidden 5120, intermediate 17408: 213 and
    725 words per row, tails of 8; 3.35 GB) in one planned run, sampled rows of every matrix."""
    from paper_2609_35465_b200.workload import DevicePass
    dp = DevicePass(shapes.QWEN3_14B.all_matrices(), seed=3)
    assert len(dp.items) == 280
    dp.y_all.fill_(float("nan"))
    dp.run_grouped()
    torch.cuda.synchronize()
    y = dp.y_all.cpu().numpy()
    used = np.zeros(len(y), dtype=bool)
    for it in dp.items:
        used[it["yoff"]:it["yoff"] + it["N"]] = True
    assert np.isfinite(y[used]).all()                     # every output row was written
    _check_sampled(dp, orc, range(len(dp.items)), rows_per_matrix=4, seed=3)


def test_qwen3_4b_layer_zero_pad_rule(orc):
    """Config 1 with K zero-padded to a multiple of 24 instead of the tail rule."""
    from paper_2609_35465_b200.workload import DevicePass
    mats = shapes.QWEN3_4B.layer_matrices()
    dp = DevicePass(mats, seed=4, tail_mode=False)
    assert all(it["ntail"] == 0 and it["B"] == -(-it["K"] // 24) for it in dp.items)
    dp.run_grouped()
    torch.cuda.synchronize()
    _check_sampled(dp, orc, range(len(mats)), rows_per_matrix=8, seed=4)


@pytest.mark.parametrize("batch", shapes.CONFIG4_BATCHES)
def test_down_proj_batch_sweep_sampled_rows(orc, batch):
    """Config 4: N = 4096, K = 12288 with 1..16 activation vectors."""
    from paper_2609_35465_b200 import tetra as tt
    m = shapes.CONFIG4
    table = tt.tetra_build_table(synth.DEFAULT_GAIN)
    codes = synth.codes_torch(6, 1, m.N, m.blocks, device="cuda")
    packed = tt.tetra_pack_codes(codes, table, m.N, m.blocks)
    sigma = synth.row_scales(6, 1, m.N)
    x = synth.activations(6, 1, m.K, batch)
    y = torch.full((batch, m.N), float("nan"), dtype=torch.float32, device="cuda")
    tt.tetra_gemv(packed, torch.from_numpy(sigma).cuda(), table, torch.from_numpy(x).cuda(), y, m.N, m.K, batch)
    torch.cuda.synchronize()
    yh = y.cpu().numpy()
    assert np.isfinite(yh).all()
    rows = np.array([0, 1, 2047, 4095, 1234, 3001])
    host_codes = np.stack([synth.words_to_bytes(synth.words(6, 1, m.blocks, int(r) * m.blocks)) for r in rows])
    for b in sorted({0, batch - 1}):
        mm = dict(N=len(rows), K=m.K, B=m.blocks, ntail=0, codes=host_codes, sigma=sigma[rows], x=x, tail=None)
        ref = oracle_product(orc, mm, synth.DEFAULT_GAIN, batch_index=b, threads=1)
        assert_gemv_close(yh[b][rows], ref, "batch %d column %d" % (batch, b))


@pytest.mark.parametrize("batch", shapes.CONFIG4_BATCHES)
def test_down_proj_batched_sampled_rows(orc, batch):
    """Config 4 through tetra_gemv_batched (decode once, tensor-core contraction): the shape and the batch
    sizes the benchmark's sweep times.  Rows: first and last, the rows around the 16- and 32-row tile edges,
    around the boundaries of the 16-warp tile groups (512 rows) and around the CTA ranges' cuts, and random
    ones; every vector of the batch."""
    from paper_2609_35465_b200 import tetra as tt
    m = shapes.CONFIG4
    table = tt.tetra_build_table(synth.DEFAULT_GAIN)
    codes = synth.codes_torch(6, 2, m.N, m.blocks, device="cuda")
    packed = tt.tetra_pack_codes(codes, table, m.N, m.blocks)
    sigma = synth.row_scales(6, 2, m.N)
    x = synth.activations(6, 2, m.K, batch)
    y = torch.full((batch, m.N), float("nan"), dtype=torch.float32, device="cuda")
    tt.tetra_gemv_batched(packed, torch.from_numpy(sigma).cuda(), table, torch.from_numpy(x).cuda(), y, m.N, m.K,
                          batch, None)
    torch.cuda.synchronize()
    yh = y.cpu().numpy()
    assert np.isfinite(yh).all()
    edges = [0, 1, 15, 16, 31, 32, 33, 511, 512, 513, 1023, 1024, 2047, 2048, 3071, 3072, 3583, 3584, 4094, 4095]
    rows = np.unique(np.concatenate([edges, np.random.default_rng(batch).integers(0, m.N, 12)]))
    host_codes = np.stack([synth.words_to_bytes(synth.words(6, 2, m.blocks, int(r) * m.blocks)) for r in rows])
    for b in range(batch):
        mm = dict(N=len(rows), K=m.K, B=m.blocks, ntail=0, codes=host_codes, sigma=sigma[rows], x=x, tail=None)
        ref = oracle_product(orc, mm, synth.DEFAULT_GAIN, batch_index=b, threads=4)
        assert_gemv_close(yh[b][rows], ref, "batched, batch %d vector %d" % (batch, b))


@pytest.mark.parametrize("batch,words", [(5, 384), (16, 384), (2, 640), (4, 640)])
def test_batched_long_cta_ranges_sampled_rows(orc, batch, words):
    """8192 x 9232 through tetra_gemv_batched: 16 tile groups x 96 column groups are more than ten cells per
    CTA, so every CTA rebuilds its activation image in the middle of its range (after eight passes with five
    to eight vectors, after four with more) and most CTAs cross a tile-group boundary; K leaves a float16
    tail of 16.  With two to four vectors (another kernel, whose image holds sixteen passes) 8192 x 15376:
    160 column groups, seventeen cells per CTA.  Rows around the tile-group boundaries and random ones, every
    vector."""
    from paper_2609_35465_b200 import tetra as tt
    N, K = 8192, 24 * words + 16
    m = make_matrix(23, 7 + batch, N, K, True, batch=batch)
    table = tt.tetra_build_table(synth.DEFAULT_GAIN)
    packed = tt.tetra_pack_codes(torch.from_numpy(m["codes"]).cuda(), table, N, m["B"])
    y = torch.full((batch, N), float("nan"), dtype=torch.float32, device="cuda")
    tt.tetra_gemv_batched(packed, torch.from_numpy(m["sigma"]).cuda(), table, torch.from_numpy(m["x"]).cuda(), y, N, K,
                          batch, torch.from_numpy(m["tail"]).cuda())
    torch.cuda.synchronize()
    yh = y.cpu().numpy()
    assert np.isfinite(yh).all()
    edges = [0, 31, 32, 511, 512, 513, 1023, 1024, 4095, 4096, 7679, 7680, 8190, 8191]
    rows = np.unique(np.concatenate([edges, np.random.default_rng(batch).integers(0, N, 18)]))
    for b in range(batch):
        ref = oracle_product(orc, m, synth.DEFAULT_GAIN, rows=rows, batch_index=b, threads=4)
        assert_gemv_close(yh[b][rows], ref, "long ranges, batch %d vector %d" % (batch, b))


def test_tall_matrix_sampled_rows(orc):
    """151,936 x 4096 (the row count of the model's vocabulary; 155 MB of codes, 18,992 row groups): the index
    arithmetic of every path far beyond the projection shapes.  One launch, the planned list, three vectors
    through the tensor-core kernel; rows at both ends, around the tile-group edges and random ones."""
    from paper_2609_35465_b200 import tetra as tt
    N, K, batch = 151936, 4096, 3
    B, ntail = K // 24, K % 24
    table = tt.tetra_build_table(synth.DEFAULT_GAIN)
    codes = synth.codes_torch(31, 4, N, B, device="cuda")
    packed = tt.tetra_pack_codes(codes, table, N, B)
    del codes
    sigma = synth.row_scales(31, 4, N)
    x = synth.activations(31, 4, K, batch)
    tail = synth.tails(31, 4, sigma, ntail)
    d = dict(codes=packed, row_scales=torch.from_numpy(sigma).cuda(), x=torch.from_numpy(x).cuda(),
             tail=torch.from_numpy(tail).cuda(), N=N, K=K)
    edges = [0, 7, 8, 511, 512, 75967, 75968, 151424, 151934, 151935]
    rows = np.unique(np.concatenate([edges, np.random.default_rng(9).integers(0, N, 22)]))
    host_codes = np.stack([synth.words_to_bytes(synth.words(31, 4, B, int(r) * B)) for r in rows])

    def check(y, b, what):
        mm = dict(N=len(rows), K=K, B=B, ntail=ntail, codes=host_codes, sigma=sigma[rows], x=x, tail=tail[rows])
        ref = oracle_product(orc, mm, synth.DEFAULT_GAIN, batch_index=b, threads=4)
        assert_gemv_close(y[rows], ref, what)

    y = torch.full((batch, N), float("nan"), dtype=torch.float32, device="cuda")
    d["y"] = y
    tt.tetra_gemv_tail(packed, d["row_scales"], table, d["x"], y, N, K, 1, d["tail"])
    torch.cuda.synchronize()
    y0 = y[0].cpu().numpy()
    assert np.isfinite(y0).all()
    check(y0, 0, "tall matrix, one launch")
    y.fill_(float("nan"))
    pr = tt.make_problems([d])
    ws = torch.empty(tt.tetra_grouped_workspace_bytes(pr), dtype=torch.uint8, device="cuda")
    tt.tetra_gemv_grouped(pr, table, ws)
    torch.cuda.synchronize()
    y1 = y[0].cpu().numpy()
    assert np.isfinite(y1).all()
    check(y1, 0, "tall matrix, planned list")
    y.fill_(float("nan"))
    tt.tetra_gemv_batched(packed, d["row_scales"], table, d["x"], y, N, K, batch, d["tail"])
    torch.cuda.synchronize()
    yb = y.cpu().numpy()
    assert np.isfinite(yb).all()
    for b in range(batch):
        check(yb[b], b, "tall matrix, batched vector %d" % b)
