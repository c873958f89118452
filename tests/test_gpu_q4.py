"""GPU parity of the 4-bit group-quantised kernels against the FP64 oracle, through the C ABI
(Sec. 4.1, 4.4, 5.1).  Tolerances as for the Tetra product: relative L2 <= 1e-3 and, per element,
|delta| <= 1e-3 * sqrt(sum_k (w x)^2) + 1e-6; dequantised rows are bit-exact."""
import numpy as np
import pytest

from paper_2609_35465_b200 import synth

pytestmark = pytest.mark.gpu

REL_L2, ABS_COEF, ABS_FLOOR = 1e-3, 1e-3, 1e-6


def _device_matrix(seed, stream, N, K, G, scale=None, offset=None, q=None):
    import torch
    from paper_2609_35465_b200 import tetra
    q = synth.q4_nibbles(seed, stream, N, K) if q is None else q
    s, o = synth.q4_scales_offsets(seed, stream, N, K // G)
    scale = s if scale is None else scale
    offset = o if offset is None else offset
    packed = tetra.tetra_q4_pack(torch.from_numpy(q).cuda(), torch.from_numpy(scale).cuda(),
                                 torch.from_numpy(offset).cuda(), N, K, G)
    return q, scale, offset, packed


def _check_gemv(q, scale, offset, packed, x, N, K, G, batch):
    import torch
    from oracle import q4 as oq
    from paper_2609_35465_b200 import tetra
    y = torch.full((batch, N), float("nan"), dtype=torch.float32, device="cuda")
    tetra.tetra_q4_gemv(packed, torch.from_numpy(x).cuda(), y, N, K, G, batch)
    got = y.cpu().numpy().astype(np.float64)
    want, tn = oq.gemv(q, scale, offset, x, N, K, G, batch)
    assert np.isfinite(got).all()
    rel = np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-300)
    assert rel <= REL_L2, rel
    bound = ABS_COEF * tn + ABS_FLOOR
    worst = np.max(np.abs(got - want) / bound)
    assert worst <= 1.0, worst
    return rel, worst


@pytest.mark.parametrize("N,K,G,batch", [
    (16, 128, 128, 1), (16, 64, 64, 1), (64, 1024, 128, 1), (37, 1152, 128, 1), (1, 256, 64, 1),
    (1024, 4096, 128, 1), (2560, 9728, 128, 1), (300, 4096, 64, 1), (512, 17408, 128, 1),
    (129, 2560, 64, 3), (256, 4096, 128, 8), (2048, 5120, 64, 5),
    (64, 32768, 64, 1), (48, 65536, 128, 2), (40, 65536, 64, 1),   # the largest K the library takes
])
def test_q4_gemv_matches_oracle(N, K, G, batch):
    q, s, o, packed = _device_matrix(21, N + K, N, K, G)
    x = synth.activations(21, 5, K, batch)
    _check_gemv(q, s, o, packed, x, N, K, G, batch)


def test_q4_gemv_extreme_nibbles_and_scales():
    """All-15 and all-0 weights, large offsets against small scales, float16-subnormal scales."""
    N, K, G = 48, 1024, 128
    x = synth.activations(22, 1, K, 2)
    for fill in (0x00, 0xFF, 0x0F, 0xF0):
        q = np.full((N, K // 2), fill, dtype=np.uint8)
        q_, s, o, packed = _device_matrix(22, 2, N, K, G, q=q)
        _check_gemv(q, s, o, packed, x, N, K, G, 2)
    s = np.full((N, K // G), 6e-8, dtype=np.float16)  # subnormal
    o = np.full((N, K // G), 0.75, dtype=np.float16)
    q, s, o, packed = _device_matrix(22, 3, N, K, G, scale=s, offset=o)
    _check_gemv(q, s, o, packed, x, N, K, G, 2)


def test_q4_gemv_is_deterministic_and_ignores_other_vectors():
    import torch
    from paper_2609_35465_b200 import tetra
    N, K, G = 700, 4096, 128
    q, s, o, packed = _device_matrix(23, 1, N, K, G)
    x = torch.from_numpy(synth.activations(23, 1, K, 4)).cuda()
    y1 = torch.empty((4, N), dtype=torch.float32, device="cuda")
    y2 = torch.empty((4, N), dtype=torch.float32, device="cuda")
    tetra.tetra_q4_gemv(packed, x, y1, N, K, G, 4)
    tetra.tetra_q4_gemv(packed, x, y2, N, K, G, 4)
    assert torch.equal(y1, y2)
    y3 = torch.empty((1, N), dtype=torch.float32, device="cuda")
    tetra.tetra_q4_gemv(packed, x[2:3].contiguous(), y3, N, K, G, 1)
    assert torch.equal(y3[0], y1[2])  # a vector's result does not depend on its neighbours in the batch


@pytest.mark.parametrize("N,K,G", [(100, 256, 64), (151936, 1024, 64), (50, 2560, 128)])
def test_q4_rows_bit_exact(N, K, G):
    import torch
    from oracle import q4 as oq
    from paper_2609_35465_b200 import tetra
    rows = min(N, 4096)  # the oracle side only needs the rows that are looked up
    ids = synth.token_ids(24, 1, 33, N)
    ids[0], ids[1] = 0, N - 1
    q = synth.q4_nibbles(24, N, N, K)
    s, o = synth.q4_scales_offsets(24, N, N, K // G)
    s[ids[2], 0] = np.float16(6e-8)  # a subnormal scale on a row that is looked up
    packed = tetra.tetra_q4_pack(torch.from_numpy(q).cuda(), torch.from_numpy(s).cuda(), torch.from_numpy(o).cuda(),
                                 N, K, G)
    out = torch.full((len(ids), K), float("nan"), dtype=torch.float16, device="cuda")
    tetra.tetra_q4_rows(packed, torch.from_numpy(ids).cuda(), out, N, K, G)
    del rows
    want = oq.rows(q, s, o, ids, N, K, G)
    assert np.array_equal(out.cpu().numpy().view(np.uint16), want.view(np.uint16))


def test_q4_argument_checks():
    import torch
    from paper_2609_35465_b200 import tetra
    N, K, G = 32, 256, 64
    q, s, o, packed = _device_matrix(25, 1, N, K, G)
    x = torch.zeros((1, K), dtype=torch.float16, device="cuda")
    y = torch.zeros((1, N), dtype=torch.float32, device="cuda")
    with pytest.raises(tetra.TetraError):
        tetra.tetra_q4_gemv(packed, x, y, N, K, 96, 1)  # group size
    with pytest.raises(tetra.TetraError):
        tetra.tetra_q4_gemv(packed, x, y, N, 200, 64, 1)  # K not a multiple of G
    with pytest.raises(tetra.TetraError):
        tetra.tetra_q4_gemv(packed, x, y, N, K, G, 9)  # batch
    with pytest.raises(tetra.TetraError):
        tetra.tetra_q4_packed_bytes(0, K, G)
    out = torch.zeros((0, K), dtype=torch.float16, device="cuda")
    tetra.tetra_q4_rows(packed, torch.zeros(0, dtype=torch.int32, device="cuda"), out, N, K, G)  # empty: no launch
    ids = torch.tensor([5, -1, N], dtype=torch.int32, device="cuda")  # ids outside the table give zero rows
    out = torch.full((3, K), 1.0, dtype=torch.float16, device="cuda")
    tetra.tetra_q4_rows(packed, ids, out, N, K, G)
    assert torch.count_nonzero(out[1:]) == 0 and torch.count_nonzero(out[0]) > 0


def test_q4_head_full_size_sampled_rows():
    """The output-head shape the bench times (151,936 x 4096, groups of 64), batch 1 and 8: rows sampled over
    the whole table (first, last, strip and CTA-range boundaries included) against the oracle."""
    import torch
    from oracle import q4 as oq
    from paper_2609_35465_b200 import tetra
    N, K, G = 151936, 4096, 64
    q = synth.q4_nibbles(26, 1, N, K)
    s, o = synth.q4_scales_offsets(26, 1, N, K // G)
    packed = tetra.tetra_q4_pack(torch.from_numpy(q).cuda(), torch.from_numpy(s).cuda(), torch.from_numpy(o).cuda(),
                                 N, K, G)
    rng = np.random.default_rng(26)
    rows = np.unique(np.concatenate([[0, 1, 31, 32, 33, 1023, 1024, 1056, N - 33, N - 32, N - 1],
                                     rng.integers(0, N, 300)]))
    for batch in (1, 8):
        x = synth.activations(26, 2, K, batch)
        y = torch.full((batch, N), float("nan"), dtype=torch.float32, device="cuda")
        tetra.tetra_q4_gemv(packed, torch.from_numpy(x).cuda(), y, N, K, G, batch)
        got = y.cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        want, tn = oq.gemv(q[rows], s[rows], o[rows], x, len(rows), K, G, batch)
        d = got[:, rows] - want
        assert np.linalg.norm(d) / np.linalg.norm(want) <= REL_L2
        assert np.max(np.abs(d) / (ABS_COEF * tn + ABS_FLOOR)) <= 1.0


# ---------------------------------------------------------------------------
# tetra_q4_list_*: a list of matrices from one persistent grid
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("G,shapes_list", [
    (128, [(1024, 4096), (4096, 4096), (4096, 12288)]),                 # v, o, down of a Qwen3-8B-shaped layer
    (128, [(37, 1152), (16, 128), (300, 2560), (1, 256), (64, 1024)]),  # ragged rows, tiny matrices
    (64, [(129, 2560), (2048, 5120)]),                                  # groups of 64
    (128, [(32, 65536)]),                                               # one strip cut across hundreds of warps
    (64, [(40, 65536), (33, 64)]),
])
def test_q4_list_matches_oracle(G, shapes_list):
    import torch
    from oracle import q4 as oq
    from paper_2609_35465_b200 import tetra
    mats, items = [], []
    for i, (N, K) in enumerate(shapes_list):
        q, s, o, packed = _device_matrix(24, 100 * i + N + K, N, K, G)
        x = synth.activations(24, i, K, 1)
        y = torch.full((N,), float("nan"), dtype=torch.float32, device="cuda")
        mats.append((q, s, o, x, N, K))
        items.append(dict(packed=packed, x=torch.from_numpy(x[0]).cuda(), y=y, N=N, K=K))
    problems = tetra.make_q4_problems(items)
    ws = tetra.tetra_q4_list_plan(problems, G)
    tetra.tetra_q4_list_run(ws, G)
    torch.cuda.synchronize()
    first = [it["y"].cpu().numpy().copy() for it in items]
    for it in items:
        it["y"].fill_(float("nan"))
    moved = torch.empty(ws.numel() + 1024, dtype=torch.uint8, device="cuda")[512:512 + ws.numel()]
    moved.copy_(ws)                                          # the plan describes itself: run it from a copy
    ws.fill_(0x5A)
    tetra.tetra_q4_list_run(moved, G)
    torch.cuda.synchronize()
    for (q, s, o, x, N, K), it, f in zip(mats, items, first):
        got = it["y"].cpu().numpy()
        assert np.array_equal(got, f)                        # bit-identical from run to run
        want, tn = oq.gemv(q, s, o, x, N, K, G, 1)
        assert np.isfinite(got).all()
        rel = np.linalg.norm(got - want[0]) / max(np.linalg.norm(want[0]), 1e-300)
        assert rel <= REL_L2, rel
        assert np.max(np.abs(got - want[0]) / (ABS_COEF * tn[0] + ABS_FLOOR)) <= 1.0
        # and the single-matrix entry point gives the same values up to float32 summation order
        y1 = torch.empty((1, N), dtype=torch.float32, device="cuda")
        tetra.tetra_q4_gemv(it["packed"], it["x"].reshape(1, -1), y1, N, K, G, 1)
        torch.cuda.synchronize()
        assert np.linalg.norm(y1.cpu().numpy()[0] - got) <= 1e-5 * max(np.linalg.norm(got), 1e-30)


def test_q4_list_rejects_bad_lists():
    import torch
    from paper_2609_35465_b200 import tetra
    q, s, o, packed = _device_matrix(25, 1, 64, 256, 128)
    x = torch.zeros(256, dtype=torch.float16, device="cuda")
    y = torch.zeros(64, dtype=torch.float32, device="cuda")
    ok = tetra.make_q4_problems([dict(packed=packed, x=x, y=y, N=64, K=256)])
    assert tetra.lib().tetra_q4_list_workspace_bytes(ok, 1, 128) > 0
    assert tetra.lib().tetra_q4_list_workspace_bytes(ok, 1, 96) == 0          # group size
    assert tetra.lib().tetra_q4_list_workspace_bytes(ok, 0, 128) == 0         # empty list
    bad = tetra.make_q4_problems([dict(packed=packed, x=x, y=y, N=64, K=192)])
    assert tetra.lib().tetra_q4_list_workspace_bytes(bad, 1, 128) == 0        # K not a multiple of G
    ws = torch.empty(16, dtype=torch.uint8, device="cuda")
    assert tetra.lib().tetra_q4_list_plan(ok, 1, 128, ws.data_ptr(), 16, None) == -6


def test_binding_rejects_tensors_that_are_too_small():
    """The C ABI takes plain pointers; the Python binding knows the tensors' sizes and refuses a call whose
    tensors are smaller than what the call would read or write, before anything is launched."""
    import torch
    from paper_2609_35465_b200 import tetra
    N, K, G = 64, 256, 64
    q = torch.zeros((N // 2, K // 2), dtype=torch.uint8, device="cuda")          # half the rows
    sc = torch.ones((N, K // G), dtype=torch.float16, device="cuda")
    with pytest.raises(tetra.TetraError, match="needs"):
        tetra.tetra_q4_pack(q, sc, sc, N, K, G)
    q = torch.zeros((N, K // 2), dtype=torch.uint8, device="cuda")
    packed = tetra.tetra_q4_pack(q, sc, sc, N, K, G)
    x = torch.zeros(K, dtype=torch.float16, device="cuda")
    y = torch.zeros(N, dtype=torch.float32, device="cuda")
    with pytest.raises(tetra.TetraError, match="needs"):
        tetra.tetra_q4_gemv(packed[:-16], x, y, N, K, G, 1)
    with pytest.raises(tetra.TetraError, match="needs"):
        tetra.tetra_q4_gemv(packed, x, y, N, K, G, 2)                           # two vectors, tensors for one
    table = tetra.tetra_build_table()
    codes = torch.zeros(tetra.tetra_codes_bytes(N, 4), dtype=torch.uint8, device="cuda")
    rs = torch.ones(N, dtype=torch.float32, device="cuda")
    x = torch.zeros(96, dtype=torch.float16, device="cuda")
    for call in (lambda: tetra.tetra_gemv(codes, rs, table, x, y, N, 24 * 5),     # five words per row, codes hold four
                 lambda: tetra.tetra_gemv(codes, rs[:10], table, x, y, N, 96),
                 lambda: tetra.tetra_gemv_batched(codes, rs, table, x, y, N, 96, 3),
                 lambda: tetra.tetra_gemv_noalloc(codes, rs, table, x, y[:8], N, 96),
                 lambda: tetra.make_problems([dict(codes=codes, row_scales=rs, x=x[:50], y=y, N=N, K=96)])):
        with pytest.raises(tetra.TetraError, match="needs"):
            call()
    tetra.tetra_gemv(codes, rs, table, x, y, N, 96)                             # the right sizes pass
    torch.cuda.synchronize()
