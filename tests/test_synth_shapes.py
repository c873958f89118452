"""Host logic: the seeded generators and the byte accounting of the workloads."""
import numpy as np
import torch

from paper_2609_35465_b200 import shapes, synth


def test_generators_are_deterministic_and_distinct():
    a = synth.codes(3, 5, 16, 9)
    assert np.array_equal(a, synth.codes(3, 5, 16, 9))
    assert not np.array_equal(a, synth.codes(3, 6, 16, 9))
    assert not np.array_equal(a, synth.codes(4, 5, 16, 9))
    w = synth.words(1, 2, 100000)
    assert w.max() < (1 << 48)
    bits = ((w[:, None] >> np.arange(48, dtype=np.uint64)[None, :]) & np.uint64(1)).mean(axis=0)
    assert np.all(np.abs(bits - 0.5) < 0.01)               # every field uniform over its range
    assert np.array_equal(synth.bytes_to_words(synth.words_to_bytes(w)), w)
    # chunked draws agree with one draw
    assert np.array_equal(synth.words(1, 2, 1000, start=500), w[500:1500])


def test_torch_generator_matches_numpy():
    a = synth.codes(9, 4, 33, 21)
    b = synth.codes_torch(9, 4, 33, 21).numpy()
    assert np.array_equal(a, b)


def test_input_distributions():
    s = synth.row_scales(0, 1, 200000).astype(np.float64)
    assert abs(np.log(s).mean() + 4.0) < 0.01 and abs(np.log(s).std() - 0.3) < 0.01
    x = synth.activations(0, 1, 200000)[0].astype(np.float64)
    assert x.dtype == np.float64 and abs(x.mean()) < 0.01 and abs(x.std() - 1.0) < 0.01
    t = synth.tails(0, 1, s[:1000].astype(np.float32), 16)
    assert t.shape == (1000, 16) and t.dtype == np.float16


def test_paper_byte_accounting():
    """Sec. 5.2, Table 'bench': the 216 lattice matrices of the 4B shapes read 0.95 GB,
    2.148 bits per weight with float32 tails and scales; padding rows to 8 bytes adds 4.1 MB."""
    ms = [m for m in shapes.QWEN3_4B.all_matrices() if not m.name.endswith(".v")]
    assert len(ms) == 216 and len(shapes.QWEN3_4B.all_matrices()) == 252
    total = sum(shapes.file_bytes(m) for m in ms)
    w = sum(shapes.weights(m) for m in ms)
    assert round(total / 1e9, 2) == 0.95
    assert round(total * 8 / w, 3) == 2.148
    pad = sum(shapes.file_bytes(m, row_pad=8) for m in ms) - total
    assert round(pad / 1e6, 1) == 4.1
    assert len(shapes.QWEN3_14B.all_matrices()) == 280


def test_layer_shapes():
    q, k, v, o, gate, up, down = shapes.QWEN3_8B.layer_matrices()
    assert (q.N, q.K) == (4096, 4096) and (k.N, k.K) == (1024, 4096) and (down.N, down.K) == (4096, 12288)
    assert q.blocks == 170 and q.ntail == 16 and down.blocks == 512 and down.ntail == 0
    q14 = shapes.QWEN3_14B.layer_matrices()[0]
    assert (q14.N, q14.K, q14.blocks, q14.ntail) == (5120, 5120, 213, 8)
