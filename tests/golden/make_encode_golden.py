"""Writes tests/golden/encode_retention.txt from the CPU oracle alone.

Sec. 3.5 measures the format on 20,000 Gaussian blocks at 2 bits per weight: 88.80 % retention for the
paper's own non-exhaustive search on this codebook, 91.98 % for the codebook that searches one
24-dimensional ball.  Neither the blocks nor the two gains are printed, so the figures are not reproducible
digit for digit; this script records what the exact search of oracle/tetra_encode_oracle.c attains on the
seeded blocks the tests use (the same recipe, 20,000 blocks, the library's default gains), which the GPU
path is then compared with at full size.
Run:  python tests/golden/make_encode_golden.py        (about two minutes on 16 cores)
"""
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle  # noqa: E402
from oracle import encode  # noqa: E402
from paper_2609_35465_b200 import synth  # noqa: E402

N = 20000


def main():
    orc = oracle.get()
    w = synth.normal(11, 0, 20, N * 24).reshape(N, 24).astype(np.float32).astype(np.float64)
    gain = synth.DEFAULT_GAIN.astype(np.float64)
    words, cos = encode.encode_blocks(w, sigma=1.0, gain=gain)
    Y, m, g = orc.decode_blocks(synth.words_to_bytes(words))
    what = Y / np.linalg.norm(Y, axis=1, keepdims=True) * gain[g][:, None]
    D = ((w - what) ** 2).mean()
    retention = 0.5 * np.log2(1.0 / D) / 2.0 * 100.0
    out = ["# written by tests/golden/make_encode_golden.py from oracle/ only",
           "# blocks = synth.normal(11, 0, 20, 24 n) rounded to float32, sigma = 1, gains = synth.DEFAULT_GAIN",
           "# paper, Sec. 3.5 (its own search / the 24-dimensional ball): 88.80 91.98",
           "blocks %d" % N,
           "mean_cosine %.9f" % cos.mean(),
           "min_cosine %.9f" % cos.min(),
           "mse_per_weight %.9f" % D,
           "retention_percent %.4f" % retention,
           "gain_bit_ones %d" % int(g.sum()),
           "mean_shell %.6f" % m.mean()]
    with open(os.path.join(HERE, "encode_retention.txt"), "w") as f:
        f.write("\n".join(out) + "\n")
    print("\n".join(out))


if __name__ == "__main__":
    main()
