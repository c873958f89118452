"""GPU GEMV parity against the FP64 oracle on the same seeded inputs, within
rel-L2 <= 1e-3 and |delta_n| <= 1e-3 sqrt(sum_k (s_n w_nk x_k)^2) + 1e-6."""
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


def upload(tt, table, m):
    d = dict(N=m["N"], K=m["K"])
    codes = torch.from_numpy(m["codes"]).cuda()
    d["codes_file"] = codes
    d["codes"] = tt.tetra_pack_codes(codes, table, m["N"], m["B"])
    d["row_scales"] = torch.from_numpy(m["sigma"]).cuda()
    d["x"] = torch.from_numpy(m["x"]).cuda()
    d["tail"] = torch.from_numpy(m["tail"]).cuda() if m["tail"] is not None else None
    d["y"] = torch.full((m["x"].shape[0], m["N"]), float("nan"), dtype=torch.float32, device="cuda")
    return d


def run_fast(tt, table, m, d):
    batch = m["x"].shape[0]
    if m["ntail"]:
        tt.tetra_gemv_tail(d["codes"], d["row_scales"], table, d["x"], d["y"], m["N"], m["K"], batch, d["tail"])
    else:
        tt.tetra_gemv(d["codes"], d["row_scales"], table, d["x"], d["y"], m["N"], m["K"], batch)
    torch.cuda.synchronize()
    return d["y"].cpu().numpy()


CASES = [
    # N, K, tail_mode                      (config 0; ragged tails; tiny; wide; zero-pad)
    (2048, 2304, True),
    (1024, 2560, True),
    (1024, 2560, False),
    (520, 4096, True),
    (264, 12288, True),
    (72, 17408, True),
    (1, 24, True),
    (7, 48, True),
    (9, 24 * 33, True),
    (33, 24 * 31 + 5, True),
    (33, 24 * 31 + 5, False),
    (300, 24 * 513, True),
    (40, 49152, True),          # the largest K the library takes (2048 blocks per row)
    (17, 49152 - 7, False),
]


@pytest.mark.parametrize("N,K,tail_mode", CASES)
def test_fast_gemv_matches_oracle(tt, table, orc, N, K, tail_mode):
    m = make_matrix(31, N * 7 + K, N, K, tail_mode)
    d = upload(tt, table, m)
    y = run_fast(tt, table, m, d)
    assert np.isfinite(y).all()
    ref = oracle_product(orc, m, GAIN)
    rel, worst = assert_gemv_close(y[0], ref, "fast %dx%d" % (N, K))
    # the paper's own check (Sec. 5.1): every row within 1e-5 * sum |w x|
    assert np.max(np.abs(y[0] - ref["y"]) / ref["abssum"]) < 1e-5


@pytest.mark.parametrize("N,K,tail_mode", [(2048, 2304, True), (96, 2560, True), (33, 24 * 31 + 5, False), (5, 24, True)])
def test_paper_design_gemv_matches_oracle(tt, table, orc, N, K, tail_mode):
    m = make_matrix(32, N * 7 + K, N, K, tail_mode)
    d = upload(tt, table, m)
    tt.tetra_gemv_paper_design(d["codes_file"], 6 * m["B"], d["row_scales"], table, d["x"], d["y"], N, K, 1,
                               d["tail"])
    torch.cuda.synchronize()
    ref = oracle_product(orc, m, GAIN)
    assert_gemv_close(d["y"].cpu().numpy()[0], ref, "paper design %dx%d" % (N, K))


@pytest.mark.parametrize("batch", [2, 5, 16])
def test_batched_activations(tt, table, orc, batch):
    m = make_matrix(33, batch, 256, 2560, True, batch=batch)
    d = upload(tt, table, m)
    y = run_fast(tt, table, m, d)
    for b in range(batch):
        assert_gemv_close(y[b], oracle_product(orc, m, GAIN, batch_index=b), "batch column %d" % b)


def test_grouped_launch_one_layer(tt, table, orc):
    """One Qwen3-4B-shaped layer (config 1) in a single persistent launch, every row checked."""
    mats = [make_matrix(34, i, mm.N, mm.K, True) for i, mm in enumerate(shapes.QWEN3_4B.layer_matrices())]
    devs = [upload(tt, table, m) for m in mats]
    problems = tt.make_problems(devs)
    ws = torch.empty(tt.tetra_grouped_workspace_bytes(problems), dtype=torch.uint8, device="cuda")
    tt.tetra_gemv_grouped(problems, table, ws)
    torch.cuda.synchronize()
    first = [d["y"].cpu().numpy().copy() for d in devs]
    tt.tetra_gemv_grouped_run(ws, table)                   # the plan can be run again: same bits
    torch.cuda.synchronize()
    for m, d, f in zip(mats, devs, first):
        y = d["y"].cpu().numpy()[0]
        assert np.array_equal(y, f[0])
        assert_gemv_close(y, oracle_product(orc, m, GAIN), "grouped %dx%d" % (m["N"], m["K"]))
        # the single-matrix entry point sums in another order: equal up to float32 rounding
        d["y"].fill_(float("nan"))
        y1 = run_fast(tt, table, m, d)[0]
        assert np.linalg.norm(y - y1) <= 1e-5 * np.linalg.norm(y)



@pytest.mark.parametrize("shapes_list", [
    [(512, 2560, True), (264, 12288, True), (72, 17408, True), (9, 24 * 33, True)],   # a few matrices
    [(1024, 4096, True)],                                                             # a single one
    [(33, 24 * 31 + 5, False), (7, 48, True), (1, 24, True)],                         # tiny and ragged
    [(40, 49152, True), (3000, 24 * 64, True), (16, 49152 - 24, True)],               # the largest K, coarse mode
])
def test_grouped_small_lists(tt, table, orc, shapes_list):
    """Small lists run in the planned path's fine mode (one row group x a slice of the column
    groups per unit, slices summed in fixed order by the last one to finish): every row checked,
    and a second run of the same plan gives the same bits."""
    mats = [make_matrix(38, 100 * i + N, N, K, tm) for i, (N, K, tm) in enumerate(shapes_list)]
    devs = [upload(tt, table, m) for m in mats]
    problems = tt.make_problems(devs)
    ws = torch.empty(tt.tetra_grouped_workspace_bytes(problems), dtype=torch.uint8, device="cuda")
    tt.tetra_gemv_grouped(problems, table, ws)
    torch.cuda.synchronize()
    first = [d["y"].cpu().numpy().copy() for d in devs]
    for d in devs:
        d["y"].fill_(float("nan"))
    tt.tetra_gemv_grouped_run(ws, table)
    torch.cuda.synchronize()
    for m, d, f in zip(mats, devs, first):
        y = d["y"].cpu().numpy()[0]
        assert np.array_equal(y, f[0])
        assert_gemv_close(y, oracle_product(orc, m, GAIN), "small list %dx%d" % (m["N"], m["K"]))


def test_special_inputs(tt, table, orc):
    N, K = 64, 240
    m = make_matrix(35, 1, N, K, True)
    m["codes"][:] = 0                                      # origin blocks: y = 0 exactly
    d = upload(tt, table, m)
    assert not run_fast(tt, table, m, d).any()
    m = make_matrix(35, 2, N, K, True)
    m["x"][:] = 0                                          # zero activations
    d = upload(tt, table, m)
    assert not run_fast(tt, table, m, d).any()
    m = make_matrix(35, 3, N, K, True)                     # unit vectors pick single weights
    for k in (0, 23, 24, 239):
        m["x"][:] = 0
        m["x"][0, k] = 1.0
        d = upload(tt, table, m)
        assert_gemv_close(run_fast(tt, table, m, d)[0], oracle_product(orc, m, GAIN), "unit %d" % k)
    # outlier channels: activations are held exactly down to 2^-12 of their block's largest,
    # so a block mixing 1000x outliers with ordinary values loses nothing
    m = make_matrix(35, 4, N, K, True)
    m["x"][0, 5::24] = (m["x"][0, 5::24].astype(np.float32) * 1000).astype(np.float16)
    m["x"][0, 30] = np.float16(60000.0)
    m["x"][0, 31] = np.float16(60000.0 / 4096)
    d = upload(tt, table, m)
    y = run_fast(tt, table, m, d)[0]
    ref = oracle_product(orc, m, GAIN)
    assert_gemv_close(y, ref, "outlier channels")
    assert np.max(np.abs(y - ref["y"]) / ref["abssum"]) < 1e-5   # float32 rounding of outlier-sized sums
    # below that the error is bounded by the step, 2^-23 of the block's largest, per coordinate
    m = make_matrix(35, 5, N, K, True)
    m["x"][0, :24:2] = np.float16(6.0e-5)
    m["x"][0, 5] = np.float16(60000.0)
    d = upload(tt, table, m)
    y = run_fast(tt, table, m, d)[0]
    ref = oracle_product(orc, m, GAIN)
    Y, mm, g = orc.decode_blocks(m["codes"][:, 0])
    bound = m["sigma"].astype(np.float64) * GAIN[g] / np.sqrt(16.0 * np.maximum(mm, 1)) * np.abs(Y).sum(axis=1) \
        * 60000.0 * 2.0 ** -23
    assert np.all(np.abs(y - ref["y"]) <= bound + 1e-6 * ref["abssum"])


def test_reruns_are_bit_identical(tt, table):
    m = make_matrix(36, 1, 1024, 4096, True)
    d = upload(tt, table, m)
    a = run_fast(tt, table, m, d).copy()
    d["y"].fill_(0)
    b = run_fast(tt, table, m, d)
    assert np.array_equal(a, b)


def test_hostio_entry_point(tt, table, orc):
    m = make_matrix(37, 1, 512, 2560, True)
    d = upload(tt, table, m)
    xh = torch.from_numpy(m["x"]).pin_memory()
    yh = torch.empty((1, m["N"]), dtype=torch.float32).pin_memory()
    xs = torch.empty_like(d["x"])
    tt.tetra_gemv_hostio(d["codes"], d["row_scales"], table, xh, yh, xs, d["y"], m["N"], m["K"], 1, d["tail"])
    torch.cuda.synchronize()
    assert_gemv_close(yh.numpy()[0], oracle_product(orc, m, GAIN), "hostio")


def test_hostio_mapped_results(tt, table, orc):
    """Results stored straight into pinned host memory (the plan's y pointers aim there): same bits as the
    staged copy, and within tolerance of the oracle."""
    from paper_2609_35465_b200 import shapes
    from paper_2609_35465_b200.workload import DevicePass
    dp = DevicePass([shapes.Matrix("a", 520, 4096), shapes.Matrix("b", 264, 2560), shapes.Matrix("c", 33, 749)], seed=61)
    dp.run_grouped_hostio()
    torch.cuda.synchronize()
    staged = dp.y_host.numpy().copy()
    dp.plan_mapped_results()
    dp.run_grouped_mapped()
    torch.cuda.synchronize()
    assert np.array_equal(dp.y_mapped.numpy(), staged)
    for i, it in enumerate(dp.items):
        ref = oracle_product(orc, dp.host_inputs(i), dp.gain)
        assert_gemv_close(dp.y_mapped.numpy()[it["yoff"]:it["yoff"] + it["N"]], ref, it["name"])


# ---------------------------------------------------------------------------
# tetra_gemv_list: a short list in one launch, no plan and no scratch memory
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("shapes_list", [
    [(1024, 4096, True), (256, 4096, True), (256, 4096, True)],                        # q, k, v of a layer, scaled down
    [(520, 2560, True)],                                                               # one matrix, ragged rows
    [(33, 24 * 31 + 5, False), (7, 48, True), (1, 24, True), (9, 24 * 33, True)],      # tiny: several matrices per CTA
    [(40, 49152, True), (300, 24 * 64, True)],                                         # more columns than the image holds
    [(300, 24 * 513, True), (264, 12288, True)],                                       # the sixteen-warp configuration
    [(8 * i + 3, 24 * (i + 1) + i, i % 2 == 0) for i in range(8)],                     # the longest list, every rule
])
def test_gemv_list_matches_oracle(tt, table, orc, shapes_list):
    mats = [make_matrix(39, 100 * i + N, N, K, tm) for i, (N, K, tm) in enumerate(shapes_list)]
    devs = [upload(tt, table, m) for m in mats]
    problems = tt.make_problems(devs)
    tt.tetra_gemv_list(problems, table)
    torch.cuda.synchronize()
    first = [d["y"].cpu().numpy().copy() for d in devs]
    for d in devs:
        d["y"].fill_(float("nan"))
    tt.tetra_gemv_list(problems, table)                    # the same bits on a second run
    torch.cuda.synchronize()
    for m, d, f in zip(mats, devs, first):
        y = d["y"].cpu().numpy()[0]
        assert np.array_equal(y, f[0])
        ref = oracle_product(orc, m, GAIN)
        assert_gemv_close(y, ref, "list %dx%d" % (m["N"], m["K"]))
        assert np.max(np.abs(y - ref["y"]) / np.maximum(ref["abssum"], 1e-30)) < 1e-5


def test_gemv_list_rejects_long_lists(tt, table):
    m = make_matrix(39, 1, 8, 24, True)
    devs = [upload(tt, table, m) for _ in range(tt.LIST_MAX + 1)]
    problems = tt.make_problems(devs)
    assert tt.lib().tetra_gemv_list(problems, len(problems), table.data_ptr(), None) == -2
    assert tt.lib().tetra_gemv_list(problems, 0, table.data_ptr(), None) == -2


# ---------------------------------------------------------------------------
# a plan describes itself: the workspace can be moved
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("shapes_list", [
    [(1024, 4096, True), (33, 749, False)],                                            # fine mode
    [(40, 49152, True), (3000, 24 * 64, True), (16, 49152 - 24, True)],                # coarse mode
])
def test_planned_workspace_can_be_copied_to_another_address(tt, table, orc, shapes_list):
    mats = [make_matrix(40, 100 * i + N, N, K, tm) for i, (N, K, tm) in enumerate(shapes_list)]
    devs = [upload(tt, table, m) for m in mats]
    problems = tt.make_problems(devs)
    ws = torch.empty(tt.tetra_grouped_workspace_bytes(problems), dtype=torch.uint8, device="cuda")
    tt.tetra_gemv_grouped_plan(problems, ws)
    torch.cuda.synchronize()
    moved = torch.empty(ws.numel() + 4096, dtype=torch.uint8, device="cuda")[2048:2048 + ws.numel()]
    moved.copy_(ws)
    ws.fill_(0xA5)                                         # the place where the plan was made is gone
    del ws
    tt.tetra_gemv_grouped_run(moved, table)
    torch.cuda.synchronize()
    for m, d in zip(mats, devs):
        assert_gemv_close(d["y"].cpu().numpy()[0], oracle_product(orc, m, GAIN), "moved plan %dx%d" % (m["N"], m["K"]))


# ---------------------------------------------------------------------------
# non-finite activations
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("bad", [float("nan"), float("inf"), -float("inf")])
def test_non_finite_activations_give_nan_rows_on_every_entry_point(tt, table, bad):
    """A NaN or an infinity among the activations of a block column must not come out as a finite number:
    every row reads every column, so every row is NaN (documented in the header)."""
    N, K = 264, 24 * 40 + 16
    m = make_matrix(41, 7, N, K, True, batch=3)
    m["x"][1, 24 * 17 + 5] = np.float16(bad)               # vector 1 only
    d = upload(tt, table, m)

    def check(y, what):
        assert np.isfinite(y[0]).all() and np.isfinite(y[2]).all(), what
        assert np.isnan(y[1]).all(), what

    check(run_fast(tt, table, m, d), "tetra_gemv_tail")
    ws = torch.empty(tt.tetra_batched_workspace_bytes(N, K), dtype=torch.uint8, device="cuda")
    yb = torch.zeros((3, N), dtype=torch.float32, device="cuda")
    tt.tetra_gemv_batched(d["codes"], d["row_scales"], table, d["x"], yb, N, K, 3, d["tail"], ws)
    torch.cuda.synchronize()
    check(yb.cpu().numpy(), "tetra_gemv_batched")
    # one vector at a time: list, planned list, no-allocation entry point
    ys = {name: torch.zeros((3, N), dtype=torch.float32, device="cuda") for name in ("list", "grouped", "noalloc")}
    for v in range(3):
        item = dict(d, x=d["x"][v], y=ys["list"][v])
        tt.tetra_gemv_list(tt.make_problems([item]), table)
        item = dict(d, x=d["x"][v], y=ys["grouped"][v])
        pr = tt.make_problems([item])
        wsg = torch.empty(tt.tetra_grouped_workspace_bytes(pr), dtype=torch.uint8, device="cuda")
        tt.tetra_gemv_grouped(pr, table, wsg)
        tt.tetra_gemv_noalloc(d["codes"], d["row_scales"], table, d["x"][v], ys["noalloc"][v], N, K, d["tail"])
        torch.cuda.synchronize()
    for name, y in ys.items():
        check(y.cpu().numpy(), name)


def test_non_finite_tail_activation_follows_ieee(tt, table):
    N, K = 64, 24 * 10 + 16
    m = make_matrix(41, 8, N, K, True)
    m["x"][0, 24 * 10 + 3] = np.float16("inf")             # multiplies tail weights only
    d = upload(tt, table, m)
    y = run_fast(tt, table, m, d)[0]
    w = m["tail"][:, 3].astype(np.float32)
    assert np.all(np.isinf(y[w != 0])) and np.all(np.sign(y[w != 0]) == np.sign(w[w != 0]))
    assert np.all(np.isnan(y[w == 0]))
