"""Pins of the encoder-search oracle (Sec. 3.1, 3.5, Eq. (2)) against the definition and the paper's figures.

The oracle finds the codebook point of largest cosine with a staged search (per-section tables joined over
the trellis).  Its pins: brute force over the WHOLE codebook restricted to the first rows of every list,
every candidate produced by the word decoder; decode -> encode round trips; never worse than sampled
codewords; the gain rule against a direct evaluation of the error; the retention on Gaussian blocks between
the paper's figure for its own non-exhaustive search (88.80 %) and that of the 24-dimensional ball (91.98 %).
"""
import numpy as np
import pytest

from oracle import encode
from paper_2609_35465_b200 import synth

MASK48 = np.uint64((1 << 48) - 1)


def _cosines(orc, words, w):
    Y, m, g = orc.decode_blocks(synth.words_to_bytes(np.asarray(words, dtype=np.uint64) & MASK48))
    Y = Y.astype(np.float64)
    n = np.linalg.norm(Y, axis=1)
    with np.errstate(invalid="ignore", divide="ignore"):
        c = (Y @ w) / (n * np.linalg.norm(w))
    c[n == 0] = -np.inf
    return c, Y


def _restricted_codebook(orc, L):
    """Every 47-bit index whose three row fields lie in the first L entries of their class lists."""
    n0 = orc.n0
    i13 = np.arange(L, dtype=np.uint64)
    i2 = np.concatenate([np.arange(min(L, n0)), n0 + np.arange(min(L, 2048 - n0))]).astype(np.uint64)
    path = np.arange(4096, dtype=np.uint64)  # s8 (6) b1 (1) b2 (4) b3 (1) are contiguous fields at bit 33
    pr = np.arange(4, dtype=np.uint64)       # p at bit 45, r at bit 46
    grid = np.meshgrid(i13, i2, i13, path, pr, indexing="ij")
    return (grid[0] | (grid[1] << np.uint64(11)) | (grid[2] << np.uint64(22)) | (grid[3] << np.uint64(33)) |
            (grid[4] << np.uint64(45))).reshape(-1)


@pytest.mark.parametrize("L", [1, 2])
def test_brute_force_on_restricted_codebook(orc, L):
    book = _restricted_codebook(orc, L)
    assert len(book) == L * (2 * L) * L * 4096 * 4
    rng = np.random.default_rng(3)
    blocks = [rng.standard_normal(24) for _ in range(4)]
    blocks.append(np.r_[np.ones(8), np.zeros(16)])          # mass in one section
    blocks.append(-np.abs(rng.standard_normal(24)))         # all negative
    blocks.append(np.r_[0.0, 0.0, 5.0, np.zeros(21)])       # one coordinate
    for w in blocks:
        c, _ = _cosines(orc, book, w)
        words, cos = encode.encode_blocks(w[None, :], row_limit=L)
        assert abs(cos[0] - c.max()) <= 1e-12, (cos[0], c.max())
        got, _ = _cosines(orc, words, w)                     # the word it returns attains that cosine
        assert abs(got[0] - c.max()) <= 1e-12
        assert int(words[0] & MASK48) in set(book[np.abs(c - c.max()) <= 1e-12].tolist())


def test_round_trip_of_codebook_points(orc):
    w = synth.words(31, 0, 24)
    Y, m, g = orc.decode_blocks(synth.words_to_bytes(w))
    keep = m > 0
    words, cos = encode.encode_blocks(Y[keep].astype(np.float64))
    assert np.all(cos >= 1 - 1e-12)
    Y2, _, _ = orc.decode_blocks(synth.words_to_bytes(words & MASK48))
    # cosine 1: the result is a positive multiple of the point (usually the point itself)
    a, b = Y[keep].astype(np.float64), Y2.astype(np.float64)
    assert np.allclose(a / np.linalg.norm(a, axis=1, keepdims=True), b / np.linalg.norm(b, axis=1, keepdims=True),
                       atol=1e-12)


def test_never_worse_than_sampled_codewords(orc):
    rng = np.random.default_rng(8)
    sample = synth.words(32, 1, 200000)
    for k in range(3):
        w = rng.standard_normal(24)
        c, _ = _cosines(orc, sample, w)
        words, cos = encode.encode_blocks(w[None, :])
        assert cos[0] >= c.max() - 1e-12
        assert 0.9 < cos[0] <= 1.0


def test_zero_block_and_gain_rule():
    words, cos = encode.encode_blocks(np.zeros((1, 24)))
    assert words[0] == 0 and cos[0] == 0.0
    rng = np.random.default_rng(9)
    gain = np.array([4.3, 5.4])
    for _ in range(200):
        c, sigma = rng.uniform(2, 8), rng.uniform(0.5, 2.0)
        # |w - u gain sigma|^2 for a unit vector u with <w, u> = c is |w|^2 - 2 gain sigma c + (gain sigma)^2
        err = (gain * sigma) ** 2 - 2 * gain * sigma * c
        assert encode.choose_gain(c, sigma, gain) == int(np.argmin(err))


def test_retention_on_gaussian_blocks(orc):
    """Sec. 3.5: 88.80 % for the paper's own (non-exhaustive) search on this codebook, 91.98 % for the
    24-dimensional ball; the exact search on this codebook lies between them."""
    n = 2048
    w = synth.normal(11, 0, 20, n * 24).reshape(n, 24).astype(np.float64)
    gain = synth.DEFAULT_GAIN.astype(np.float64)
    words, cos = encode.encode_blocks(w, sigma=1.0, gain=gain)
    Y, m, g = orc.decode_blocks(synth.words_to_bytes(words))
    assert np.array_equal(g, (words >> np.uint64(47)).astype(np.uint8))
    what = Y / np.linalg.norm(Y, axis=1, keepdims=True) * gain[g][:, None]
    D = ((w - what) ** 2).mean()
    retention = 0.5 * np.log2(1.0 / D) / 2.0 * 100.0
    assert 88.80 <= retention <= 91.98, retention


# ---------------------------------------------------------------------------
# Pins that do not share the search's decomposition (per-section tables joined over the trellis): both go
# through the word decoder only.
# ---------------------------------------------------------------------------
def test_planted_optima_deep_in_the_lists(orc):
    """Codebook points from deep rows (ranks 2-4, the class-1 half of the middle list, the last entries of the
    lists, both parities), turned by 3 degrees: any two codebook directions are at least 15.9 degrees apart,
    so the search must come back with the planted direction."""
    from encode_cases import deep_words, direction_cosines, planted_blocks
    words = deep_words(orc, 2000, seed=5)
    rows = np.asarray(orc.rows, dtype=np.uint32)
    assert ((words >> np.uint64(11)) & np.uint64(2047) >= np.uint64(orc.n0)).sum() >= 900
    w, Y = planted_blocks(orc, words, seed=6)
    found, cos = encode.encode_blocks(w)
    assert np.all(np.abs(cos - np.cos(np.deg2rad(3.0))) <= 1e-9)          # the value of the optimum
    c, Y2 = direction_cosines(orc, found & MASK48, Y)                     # direction of the word it returns
    assert np.all(c >= 1 - 1e-12)
    ranks = np.stack([(rows >> np.uint32(4 * j)) & np.uint32(15) for j in range(8)], axis=1).max(axis=1)
    i1 = (words & np.uint64(2047)).astype(np.int64) + 2048 * ((words >> np.uint64(46)) & np.uint64(1)).astype(np.int64)
    assert {2, 3, 4} <= set(ranks[i1].tolist())                           # the planted rows do reach ranks 2, 3, 4


def test_no_single_field_neighbour_beats_the_search(orc):
    """Brute force through the word decoder around the search's answer: every word that differs from it in one
    field (all 2048 values of each row index, all 4096 trellis paths, the other parity/class pairs), about
    10,000 words per block, over a million in all; none may have a larger cosine."""
    from encode_cases import direction_cosines, single_field_neighbours
    n = 104
    w = synth.normal(12, 3, 20, n * 24).reshape(n, 24).astype(np.float64)
    w[0, 8:] = 0
    w[1] = np.abs(w[1])
    found, cos = encode.encode_blocks(w)
    total = 0
    for k in range(n):
        nb = single_field_neighbours(found[k])
        c, _ = direction_cosines(orc, nb, w[k])
        assert c.max() <= cos[k] + 1e-12, (k, c.max(), cos[k])
        total += len(nb)
    assert total >= 1_000_000
