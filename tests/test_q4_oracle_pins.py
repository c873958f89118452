"""Pins of the 4-bit group-quantisation oracle against numpy and closed forms (Sec. 4.1, 4.4, 5.1).

Each test is chosen so that a plausible mistake in the oracle (nibble order, transposed scale table, group
index off by one, dropped offset, wrong half conversion or rounding) fails it.
"""
import numpy as np
import pytest

from oracle import q4
from paper_2609_35465_b200 import synth


def test_half_to_double_every_pattern():
    bits = np.arange(65536, dtype=np.uint16)
    want = bits.view(np.float16).astype(np.float64)
    got = np.array([q4.half_to_double(int(b)) for b in bits])
    finite = np.isfinite(want)
    assert np.array_equal(got[finite], want[finite])
    assert np.array_equal(np.isnan(got), np.isnan(want))
    assert np.array_equal(np.isinf(got), np.isinf(want)) and np.array_equal(np.sign(got[~finite & ~np.isnan(want)]),
                                                                            np.sign(want[~finite & ~np.isnan(want)]))


def test_float_to_half_against_numpy():
    rng = np.random.default_rng(5)
    # every representable half, the midpoints between neighbours (ties), and points just off the midpoints
    halves = np.arange(0x7C00, dtype=np.uint16).view(np.float16).astype(np.float64)
    mids = (halves[:-1] + halves[1:]) / 2
    cases = np.concatenate([halves, mids, mids * (1 + 2.0 ** -20), mids * (1 - 2.0 ** -20),
                            rng.standard_normal(20000) * np.exp(rng.uniform(-20, 12, 20000)),
                            [65504.0, 65519.9, 65520.0, 70000.0, 2.0 ** -25, 2.0 ** -25 * 1.0001, 0.0]])
    cases = np.concatenate([cases, -cases]).astype(np.float32)
    with np.errstate(over="ignore"):
        want = cases.astype(np.float16).view(np.uint16)
    got = np.array([q4.float_to_half(float(c)) for c in cases], dtype=np.uint16)
    assert np.array_equal(got, want)


def _unpack(q, N, K):
    """numpy's view of the nibble order: weight 2b low, 2b+1 high."""
    out = np.empty((N, K), dtype=np.int64)
    out[:, 0::2] = q & 15
    out[:, 1::2] = q >> 4
    return out


@pytest.mark.parametrize("G", [64, 128])
def test_single_nibble_matrices(G):
    """One nonzero weight: y_n = q * scale * x_k and nothing else (nibble, row, column and group order)."""
    N, K = 5, 3 * G
    x = synth.activations(3, 0, K)
    xd = x.astype(np.float64).reshape(-1)
    for n, k, v in [(0, 0, 1), (0, 1, 1), (2, 1, 15), (4, K - 1, 9), (3, G, 7), (1, G - 1, 3), (2, 2 * G + 17, 12)]:
        q = np.zeros((N, K // 2), dtype=np.uint8)
        q[n, k // 2] = v << (4 * (k & 1))
        scale = np.zeros((N, K // G), dtype=np.float16)
        scale[n, k // G] = 0.5
        offset = np.zeros((N, K // G), dtype=np.float16)
        y, tn = q4.gemv(q, scale, offset, x, N, K, G)
        want = np.zeros(N)
        want[n] = 0.5 * v * xd[k]
        assert np.array_equal(y[0], want)
        assert tn[0, n] == abs(want[n])
        # a scale in any OTHER group, or on any other row, must not matter
        scale2 = np.full((N, K // G), 3.0, dtype=np.float16)
        scale2[n, k // G] = 0.5
        y2, _ = q4.gemv(q, scale2, offset, x, N, K, G)
        assert np.array_equal(y2[0], want)


def test_offset_only_and_scale_ramp():
    N, K, G = 3, 512, 128
    x = synth.activations(4, 0, K)
    xd = x.astype(np.float64).reshape(-1)
    groups = K // G
    # q = 0: y_n = sum_g offset[n, g] * sum_{k in g} x_k
    offset = (np.arange(N * groups).reshape(N, groups) * 0.25 - 1).astype(np.float16)
    y, _ = q4.gemv(np.zeros((N, K // 2), np.uint8), np.ones((N, groups), np.float16), offset, x, N, K, G)
    gs = xd.reshape(groups, G)
    want = np.array([sum(float(offset[n, g]) * gs[g].sum() for g in range(groups)) for n in range(N)])
    assert np.allclose(y[0], want, rtol=0, atol=1e-12)
    # q = 1 everywhere, scale[n, g] = g + 1, x = 1: y_n = G * (1 + 2 + ... + groups)
    ones = np.ones(K, dtype=np.float16)
    scale = np.tile(np.arange(1, groups + 1, dtype=np.float16), (N, 1))
    y, tn = q4.gemv(np.full((N, K // 2), 0x11, np.uint8), scale, np.zeros((N, groups), np.float16), ones, N, K, G)
    assert np.array_equal(y[0], np.full(N, G * groups * (groups + 1) / 2))
    assert np.allclose(tn[0], np.sqrt(G * sum((g + 1) ** 2 for g in range(groups))))


@pytest.mark.parametrize("G,N,K,batch", [(128, 37, 1024, 1), (64, 19, 448, 3), (128, 8, 128, 2)])
def test_dense_product_of_numpy(G, N, K, batch):
    q = synth.q4_nibbles(7, 1, N, K)
    scale, offset = synth.q4_scales_offsets(7, 1, N, K // G)
    x = synth.activations(7, 1, K, batch)
    W = (np.repeat(scale.astype(np.float64), G, axis=1) * _unpack(q, N, K) +
         np.repeat(offset.astype(np.float64), G, axis=1))
    want = x.astype(np.float64).reshape(batch, K) @ W.T
    y, tn = q4.gemv(q, scale, offset, x, N, K, G, batch)
    assert np.allclose(y, want, rtol=1e-12, atol=1e-12)
    want_tn = np.sqrt(((x.astype(np.float64).reshape(batch, 1, K) * W[None]) ** 2).sum(-1))
    assert np.allclose(tn, want_tn, rtol=1e-12)
    for n, k in [(0, 0), (N - 1, K - 1), (N // 2, min(G, K - 1)), (1, G - 1)]:
        assert q4.weight(q, scale, offset, K, G, n, k) == W[n, k]


def test_rows_against_numpy_float32_then_float16():
    N, K, G = 50, 256, 64
    q = synth.q4_nibbles(8, 2, N, K)
    scale, offset = synth.q4_scales_offsets(8, 2, N, K // G)
    ids = np.array([0, 49, 7, 7, 23], dtype=np.int32)
    W = (np.repeat(scale.astype(np.float64), G, axis=1) * _unpack(q, N, K) +
         np.repeat(offset.astype(np.float64), G, axis=1))  # exact in float64
    want = W[ids].astype(np.float32).astype(np.float16)
    got = q4.rows(q, scale, offset, ids, N, K, G)
    assert np.array_equal(got.view(np.uint16), want.view(np.uint16))
    with pytest.raises(IndexError):
        q4.rows(q, scale, offset, np.array([50], np.int32), N, K, G)
    with pytest.raises(ValueError):  # K is not a multiple of the group size
        q4.gemv(q, scale[:, :2], offset[:, :2], synth.activations(1, 1, K), N, K, 96)
