"""Word lists for the encoder pins that share nothing with the encoder's own decomposition: words that reach
deep into the row lists (for planted optima), and the single-field neighbourhood of a word (for a brute-force
local check through the word decoder).  Pure bookkeeping on the 48-bit word of Sec. 3.3-3.4; no arithmetic of
the search."""
import numpy as np

from paper_2609_35465_b200 import synth

# field positions of the file-order word, from the least significant bit
I1, I2, I3, PATH, P, R = 0, 11, 22, 33, 45, 46


def make_word(i1, i2, i3, path, p, r):
    return (np.uint64(i1) | (np.uint64(i2) << np.uint64(I2)) | (np.uint64(i3) << np.uint64(I3)) |
            (np.uint64(path) << np.uint64(PATH)) | (np.uint64(p) << np.uint64(P)) | (np.uint64(r) << np.uint64(R)))


def deep_words(orc, count, seed):
    """`count` words whose rows lie deep in the lists: rows holding ranks 2, 3 and 4, the class-1 half of the
    middle list (i2 >= N0), the last entries of every list, both parities and both classes."""
    rows = np.asarray(orc.rows, dtype=np.uint32)
    ranks = np.stack([(rows >> np.uint32(4 * j)) & np.uint32(15) for j in range(8)], axis=1)
    maxrank = ranks.max(axis=1)
    n0 = orc.n0
    rng = np.random.default_rng(seed)
    by_class = []
    for cls in range(2):
        mr = maxrank[2048 * cls:2048 * (cls + 1)]
        pools = [np.nonzero(mr == k)[0] for k in (2, 3, 4)] + [np.arange(2040, 2048)]
        assert all(len(q) for q in pools), "every class has rows of ranks 2, 3 and 4"
        by_class.append(pools)
    words = []
    while len(words) < count:
        p, r = int(rng.integers(2)), int(rng.integers(2))
        kind = len(words) % 4
        i1 = int(rng.choice(by_class[r][kind]))
        i2 = int(rng.integers(n0, 2048)) if len(words) % 2 else int(rng.integers(n0 - 300, n0))
        r3 = p ^ r ^ int(i2 >= n0)                           # Eq. (3): the class the third index is read in
        i3 = int(rng.choice(by_class[r3][(kind + 1 + len(words) // 4) % 4]))
        words.append(make_word(i1, i2, i3, int(rng.integers(4096)), p, r))
    return np.array(words, dtype=np.uint64)


def single_field_neighbours(word):
    """Every word that differs from `word` in exactly one field (gain bit cleared): all i1, all i2, all i3,
    all trellis paths, and the other three (p, r) pairs."""
    w = int(word) & ((1 << 47) - 1)

    def with_field(pos, width, values):
        mask = ((1 << width) - 1) << pos
        return [(w & ~mask) | (int(v) << pos) for v in values]
    out = (with_field(I1, 11, range(2048)) + with_field(I2, 11, range(2048)) + with_field(I3, 11, range(2048)) +
           with_field(PATH, 12, range(4096)) + with_field(P, 2, range(4)))
    return np.array(sorted(set(out) - {w}), dtype=np.uint64)


def direction_cosines(orc, words, w):
    """FP64 cosine between block(s) w and the decoded points of `words` (-inf for the origin)."""
    Y, m, g = orc.decode_blocks(synth.words_to_bytes(np.asarray(words, dtype=np.uint64)))
    Y = Y.astype(np.float64)
    n = np.linalg.norm(Y, axis=1)
    w = np.asarray(w, dtype=np.float64)
    with np.errstate(invalid="ignore", divide="ignore"):
        c = (Y * w).sum(axis=1) / (n * (np.linalg.norm(w, axis=-1)))
    c[n == 0] = -np.inf
    return c, Y


def planted_blocks(orc, words, seed, angle_deg=3.0):
    """The decoded points of `words`, each turned by `angle_deg` degrees in a random direction.  Distinct
    lattice points differ by a vector of squared norm >= 32, so two codebook directions of squared norm
    <= 416 are at least acos(1 - 16/416) = 15.9 degrees apart: within 3 degrees of a point, that point's
    direction is the unique closest one."""
    _, Y = direction_cosines(orc, words, np.ones(24))
    rng = np.random.default_rng(seed)
    e = rng.standard_normal(Y.shape)
    u = Y / np.linalg.norm(Y, axis=1, keepdims=True)
    e -= (e * u).sum(axis=1, keepdims=True) * u              # orthogonal to the point
    e /= np.linalg.norm(e, axis=1, keepdims=True)
    t = np.deg2rad(angle_deg)
    scale = rng.uniform(0.25, 4.0, size=(len(Y), 1))         # the objective is scale-free
    return scale * np.linalg.norm(Y, axis=1, keepdims=True) * (np.cos(t) * u + np.sin(t) * e), Y
