"""GPU decode parity: both decoders of the CUDA library against the CPU oracle,
bit for bit (Sec. 3.4: every 48-bit value is a legal word)."""
import numpy as np
import pytest
import torch

from paper_2609_35465_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tt():
    from paper_2609_35465_b200 import tetra
    return tetra


@pytest.fixture(scope="module")
def table(tt):
    return tt.tetra_build_table()


def _oracle(orc, words):
    return orc.decode_blocks(synth.words_to_bytes(words))


def _gpu_file(tt, table, words):
    codes = torch.from_numpy(synth.words_to_bytes(words)).cuda()
    y, mg = tt.tetra_decode_blocks(codes, table)
    torch.cuda.synchronize()
    return y.cpu().numpy(), mg.cpu().numpy()


def _gpu_packed(tt, table, words, N, B):
    codes = torch.from_numpy(synth.words_to_bytes(words)).cuda().reshape(N, B, 6)
    packed = tt.tetra_pack_codes(codes, table, N, B)
    assert packed.numel() == -(-N // 8) * 48 * B
    y, mg = tt.tetra_decode_packed(packed, table, N, B)
    torch.cuda.synchronize()
    return y.cpu().numpy().reshape(-1, 24), mg.cpu().numpy().reshape(-1, 2)


def test_device_table_holds_the_paper_blob(tt, table, orc):
    blob = bytes(table[:18816].cpu().numpy())
    assert blob == orc.table_blob()


def test_random_words_file_order(tt, table, orc):
    w = synth.words(21, 0, 2_000_000)
    y, mg = _gpu_file(tt, table, w)
    Y, m, g = _oracle(orc, w)
    assert np.array_equal(y, Y)
    assert np.array_equal(mg[:, 0], m) and np.array_equal(mg[:, 1], g)


@pytest.mark.parametrize("N,B", [(2048, 96), (13, 37), (1, 1), (8, 32), (9, 33), (64, 725)])
def test_random_words_packed(tt, table, orc, N, B):
    w = synth.words(22, N * 1000 + B, N * B)
    y, mg = _gpu_packed(tt, table, w, N, B)
    Y, m, g = _oracle(orc, w)
    assert np.array_equal(y, Y)
    assert np.array_equal(mg[:, 0], m) and np.array_equal(mg[:, 1], g)


def test_field_sweeps_both_decoders(tt, table, orc):
    """Every value of every field (all 4096 rows in sections 1 and 3, the whole
    middle list, every trellis path), others fixed at random."""
    fields = [(0, 11), (11, 11), (22, 11), (33, 12), (45, 1), (46, 1), (47, 1)]
    ws = []
    for b in synth.words(23, 0, 8).tolist():
        for lo, wd in fields:
            rng = np.arange(1 << wd, dtype=np.uint64)
            ws.append((np.uint64(b) & ~np.uint64(((1 << wd) - 1) << lo)) | (rng << np.uint64(lo)))
    w = np.concatenate(ws)
    w = np.concatenate([w, np.array([0, 1, (1 << 48) - 1, 1 << 45, 1 << 46, 1 << 47], dtype=np.uint64)])
    pad = (-len(w)) % 40
    w = np.concatenate([w, np.zeros(pad, dtype=np.uint64)])
    Y, m, g = _oracle(orc, w)
    y, mg = _gpu_file(tt, table, w)
    assert np.array_equal(y, Y) and np.array_equal(mg[:, 0], m) and np.array_equal(mg[:, 1], g)
    y, mg = _gpu_packed(tt, table, w, len(w) // 40, 40)
    assert np.array_equal(y, Y) and np.array_equal(mg[:, 0], m) and np.array_equal(mg[:, 1], g)


def test_rank4_rows_and_every_pattern(tt, table, orc):
    """The rows that hold a coordinate of rank 4 (|y| up to 10) take the fix-up
    path of the fast decoder: all of them, in sections 1 and 3, with every
    trellis path through a few states and both parities."""
    rows = orc.rows
    r4 = [i for i in range(4096) if any(((int(rows[i]) >> (4 * j)) & 15) == 4 for j in range(8))]
    assert len(r4) == 32
    ws = []
    for idx in r4:
        cls, i = divmod(idx, 2048)
        for path in range(0, 4096, 7):
            for p in (0, 1):
                for i2 in (0, 1300):
                    delta = int(i2 >= 1240)
                    # section 1 reads row idx when r = cls; section 3 when p ^ r ^ delta = cls
                    ws.append(i | (i2 << 11) | (5 << 22) | (path << 33) | (p << 45) | (cls << 46))
                    r = cls ^ p ^ delta
                    ws.append(9 | (i2 << 11) | (i << 22) | (path << 33) | (p << 45) | (r << 46))
    w = np.array(ws, dtype=np.uint64)
    pad = (-len(w)) % 64
    w = np.concatenate([w, np.zeros(pad, dtype=np.uint64)])
    Y, m, g = _oracle(orc, w)
    assert np.abs(Y).max() == 10
    y, mg = _gpu_file(tt, table, w)
    assert np.array_equal(y, Y) and np.array_equal(mg[:, 0], m)
    y, mg = _gpu_packed(tt, table, w, len(w) // 64, 64)
    assert np.array_equal(y, Y) and np.array_equal(mg[:, 0], m)


def test_empty_input_is_a_no_op(tt, table):
    codes = torch.empty((0, 6), dtype=torch.uint8, device="cuda")
    y, mg = tt.tetra_decode_blocks(codes, table)
    assert y.shape == (0, 24)
