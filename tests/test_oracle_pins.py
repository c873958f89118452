"""Pins for the CPU oracle: each test checks it against something the paper or
the mathematics fixes, computed here without the oracle's own code path."""
import hashlib
import os

import numpy as np
import pytest

from paper_2609_35465_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def popcount(a):
    a = np.asarray(a, dtype=np.uint64)
    n = np.zeros(a.shape, dtype=np.int64)
    for k in range(24):
        n += ((a >> np.uint64(k)) & np.uint64(1)).astype(np.int64)
    return n


def ranks_of(rows):
    rows = np.asarray(rows, dtype=np.uint32)
    return np.stack([(rows >> np.uint32(4 * j)) & np.uint32(15) for j in range(8)], axis=-1).astype(np.int64)


def val_table(orc):
    return np.array([[orc.rank_value(o, r) for r in range(8)] for o in range(4)], dtype=np.int64)


# ---------------------------------------------------------------- Golay code
def test_golay_weight_enumerator_and_linearity(orc):
    """A binary [24,12] code with weights 0/8/12/16/24 in numbers 1/759/2576/759/1
    is the extended Golay code (Sec. 3.2 needs nothing more of it)."""
    g = orc.golay.astype(np.uint64)
    assert len(np.unique(g)) == 4096 and int(g.max()) < (1 << 24)
    w, cnt = np.unique(popcount(g), return_counts=True)
    assert dict(zip(w.tolist(), cnt.tolist())) == {0: 1, 8: 759, 12: 2576, 16: 759, 24: 1}
    gs = set(g.tolist())
    rng = np.random.default_rng(1)
    a = g[rng.integers(0, 4096, 20000)]
    b = g[rng.integers(0, 4096, 20000)]
    assert all(int(v) in gs for v in (a ^ b))            # closed under addition
    assert np.all(popcount(a & b) % 2 == 0)              # self-orthogonal
    for octad in (0x0000FF, 0x00FF00, 0xFF0000):         # three disjoint octads, Sec. 3.2
        assert octad in gs


def test_trellis_has_64_states_per_cut(orc):
    """Sec. 3.2: the cuts after coordinates 8 and 16 each have 64 states.  A
    state is a set of codewords sharing their futures; count those directly."""
    g = orc.golay
    c1, c2, c3 = g & 0xFF, (g >> 8) & 0xFF, (g >> 16) & 0xFF
    fut = {}
    for a, b, c in zip(c1.tolist(), c2.tolist(), c3.tolist()):
        fut.setdefault(a, set()).add((b, c))
    assert len(fut) == 128                                # pattern bytes of section 1
    assert len({frozenset(v) for v in fut.values()}) == 64
    past = {}
    for a, b, c in zip(c1.tolist(), c2.tolist(), c3.tolist()):
        past.setdefault(c, set()).add((a, b))
    assert len(past) == 128
    assert len({frozenset(v) for v in past.values()}) == 64
    assert len(set(c2.tolist())) == 128
    for sec in (c1, c2, c3):                              # all even weight
        assert np.all(popcount(sec) % 2 == 0)


def test_trellis_tables_spell_the_code(orc):
    """64 x 2 x 16 x 2 = 4096 paths, one per codeword (Sec. 3.2, Fig. geom)."""
    pre, br, suf = orc.prefixes, orc.branches, orc.suffixes
    assert pre.nbytes + br.nbytes + suf.nbytes == 2304    # Sec. 3.4
    words = set()
    for s8 in range(64):
        reached = {}
        for b2 in range(16):
            c2, s16 = int(br[16 * s8 + b2]) & 0xFF, int(br[16 * s8 + b2]) >> 8
            assert s16 < 64
            reached.setdefault(s16, []).append(c2)
            for b1 in range(2):
                for b3 in range(2):
                    words.add(int(pre[2 * s8 + b1]) | (c2 << 8) | (int(suf[2 * s16 + b3]) << 16))
        assert len(reached) == 8                          # 8 next states, 2 parallel branches each
        assert all(len(v) == 2 and v[0] ^ v[1] == 0xFF for v in reached.values())
    assert words == set(orc.golay.tolist())
    # two prefixes of a state share their futures: same state
    g = orc.golay
    fut = {}
    for w in g.tolist():
        fut.setdefault(w & 0xFF, set()).add(w >> 8)
    for s8 in range(64):
        assert fut[int(pre[2 * s8])] == fut[int(pre[2 * s8 + 1])]


# ---------------------------------------------------------------- rank rows
def test_rank_value_lists(orc):
    """Sec. 3.3 prints the lists for o = 0 and o = 1; every list is o + 4Z in
    order of distance from zero."""
    v = val_table(orc)
    assert v[0, :4].tolist() == [0, 4, -4, 8]
    assert v[1, :3].tolist() == [1, -3, 5]
    for o in range(4):
        assert np.all((v[o] - o) % 4 == 0)
        assert np.all(np.diff(np.abs(v[o])) >= 0)
        assert len(set(v[o].tolist())) == 8
        lo, hi = v[o].min(), v[o].max()                   # no gaps: the 8 nearest values
        assert set(v[o].tolist()) == {x for x in range(lo, hi + 1) if (x - o) % 4 == 0}


def test_rows_are_the_cheapest_per_class(orc):
    """Independent enumeration (numpy): the cost multiset of each half equals that of
    the 2048 cheapest vectors of its class; N0 = 1240 and 808 (Sec. 3.3)."""
    grids = np.stack(np.meshgrid(*[np.arange(6)] * 8, indexing="ij"), axis=-1).reshape(-1, 8)
    cost = ((2 * grids + 1) ** 2).sum(axis=1)
    cls = np.isin(grids, (1, 2, 5, 6)).sum(axis=1) % 2
    rows = orc.rows
    rk = ranks_of(rows)
    assert rk.max() <= 4
    tcost = ((2 * rk + 1) ** 2).sum(axis=1)
    tcls = np.isin(rk, (1, 2, 5, 6)).sum(axis=1) % 2
    assert np.all(tcls[:2048] == 0) and np.all(tcls[2048:] == 1)
    assert len(np.unique(rows)) == 4096
    for c in (0, 1):
        best = np.sort(cost[cls == c])[:2048]
        assert best.max() < 121 + 7                       # ranks >= 5 can never enter
        assert np.array_equal(np.sort(tcost[2048 * c:2048 * (c + 1)]), best)
        assert np.all(np.diff(tcost[2048 * c:2048 * (c + 1)]) >= 0)   # sorted by cost
    assert [orc.row_cost(int(r)) for r in rows[:50]] == tcost[:50].tolist()
    assert [orc.row_cls(int(r)) for r in rows[2040:2056]] == tcls[2040:2056].tolist()
    # middle list = 2048 cheapest overall
    best_all = np.sort(cost)[:2048]
    assert orc.n0 == 1240 and 2048 - orc.n0 == 808
    mid = np.array([orc.mix(i)[0] for i in range(2048)])
    dl = np.array([orc.mix(i)[1] for i in range(2048)])
    assert np.array_equal(np.sort(tcost[mid]), best_all)
    assert np.array_equal(dl, tcls[mid]) and dl[:1240].sum() == 0 and dl[1240:].all()
    assert len(np.unique(mid)) == 2048
    # the cut between classes in the middle list falls exactly where Sec. 3.3 says
    assert (cost[cls == 0] < 72).sum() == 499 and (cost[cls == 1] < 72).sum() == 808
    assert ((cost == 72) & (cls == 1)).sum() == 0


def test_class_is_k_parity_and_cost_is_norm(orc):
    """Sec. 3.3: cls(rho) is the parity of sum k_j for every pattern byte and
    parity p; cost is the squared norm when p = 1."""
    v = val_table(orc)
    rk = ranks_of(orc.rows)                               # [4096, 8]
    tcls = np.array([orc.row_cls(int(r)) for r in orc.rows])
    tcost = np.array([orc.row_cost(int(r)) for r in orc.rows])
    bytes_ = sorted(set((orc.golay & 0xFF).tolist()))
    assert len(bytes_) == 128
    for p in (0, 1):
        for c in bytes_:
            cj = (c >> np.arange(8)) & 1
            o = p + 2 * cj
            y = v[o[None, :], rk]
            k = (y - o[None, :]) // 4
            assert np.all(4 * k + o[None, :] == y)
            assert np.array_equal(k.sum(axis=1) % 2, tcls)
            if p == 1:
                assert np.array_equal((y * y).sum(axis=1), tcost)
    # the scalar section decoder agrees with that reading on a sample
    rng = np.random.default_rng(2)
    for _ in range(3000):
        p, c, i = int(rng.integers(2)), bytes_[int(rng.integers(128))], int(rng.integers(4096))
        cj = (c >> np.arange(8)) & 1
        want = v[p + 2 * cj, rk[i]]
        assert np.array_equal(orc.decode_section(p, c, int(orc.rows[i])), want)


# ---------------------------------------------------------------- the whole codebook
def _section_histograms(orc):
    v = val_table(orc)
    rk = ranks_of(orc.rows)
    mid0 = np.arange(0, orc.n0)
    mid1 = np.arange(2048, 2048 + 2048 - orc.n0)
    hist = {}
    maxabs = 0
    for p in (0, 1):
        for c in sorted(set((orc.golay & 0xFF).tolist())):
            o = p + 2 * ((c >> np.arange(8)) & 1)
            y = v[o[None, :], rk]
            maxabs = max(maxabs, int(np.abs(y).max()))
            n = (y * y).sum(axis=1)
            for key, idx in (("h0", np.arange(2048)), ("h1", np.arange(2048, 4096)),
                             ("m0", mid0), ("m1", mid1)):
                hist[(p, c, key)] = np.bincount(n[idx], minlength=256)
    return hist, maxabs


def test_codebook_shells_match_leech_theta_series(orc):
    """Count the points of the whole codebook per shell by convolving section
    histograms over all codewords, parities and classes.  Sec. 3.4: m <= 26,
    max |y_j| = 10.  The lattice's theta series 1 + 196560 q^4 + 16773120 q^6 +
    398034000 q^8 + ... bounds every shell and the codebook holds the first two
    shells completely; 47 bits of index give 2^47 points."""
    hist, maxabs = _section_histograms(orc)
    assert maxabs == 10
    total = np.zeros(1024, dtype=object)
    cache = {}
    for w in orc.golay.tolist():
        c1, c2, c3 = w & 0xFF, (w >> 8) & 0xFF, (w >> 16) & 0xFF
        for p in (0, 1):
            for r in (0, 1):
                for d in (0, 1):
                    r3 = p ^ r ^ d
                    key = (p, c1, r, c2, d, c3, r3)
                    a = hist[(p, c1, "h%d" % r)]
                    b = hist[(p, c2, "m%d" % d)]
                    c = hist[(p, c3, "h%d" % r3)]
                    ab = cache.get((p, c1, r, c2, d))
                    if ab is None:
                        ab = np.convolve(a, b)
                        cache[(p, c1, r, c2, d)] = ab
                    abc = np.convolve(ab, c)
                    total[:len(abc)] += abc.astype(object)
    counts = {i: int(n) for i, n in enumerate(total) if n}
    assert sum(counts.values()) == 2 ** 47
    assert all(norm % 16 == 0 for norm in counts)
    shells = {norm // 16: n for norm, n in counts.items()}
    assert max(shells) == 26
    assert shells[0] == 1 and 1 not in shells
    assert shells[2] == 196560 and shells[3] == 16773120
    theta = {4: 398034000, 5: 4629381120, 6: 34417656000}
    for m, n in theta.items():
        assert 0 < shells[m] <= n


def test_origin_and_hand_decoded_words(orc):
    """Sec. 3.4: the all-zero word is the origin.  i1 = 1 picks the second
    cheapest class-0 row, two coordinates at rank 1, i.e. +4 (Sec. 3.3 lists)."""
    y, m, g = orc.decode_word(0)
    assert not y.any() and m == 0 and g == 0
    y, m, g = orc.decode_word(1)
    assert sorted(y.tolist()) == [0] * 22 + [4, 4] and m == 2 and g == 0
    y, m, g = orc.decode_word(1 << 47)
    assert not y.any() and g == 1
    # p = 1 on the cheapest rows: every coordinate is +-1 (norm 24 is not a
    # lattice norm, so Eq. (3) must have moved section 3 to class 1: one +-3)
    y, m, g = orc.decode_word(1 << 45)
    assert sorted(np.abs(y).tolist()) == [1] * 23 + [3] and m == 2


def _membership_numpy(orc, Y):
    """Eq. (1), vectorised here independently of the oracle's C test."""
    Y = Y.astype(np.int64)
    p = Y[:, 0] & 1
    ok = np.all((Y & 1) == p[:, None], axis=1)
    half = (Y - p[:, None]) // 2
    cj = half & 1
    c = (cj << np.arange(24)[None, :]).sum(axis=1)
    ok &= np.isin(c, orc.golay.astype(np.int64))
    rest = Y - p[:, None] - 2 * cj
    ok &= np.all(rest % 4 == 0, axis=1)
    ok &= ((rest // 4).sum(axis=1) & 1) == p
    return ok


def test_random_words_decode_into_the_lattice(orc):
    """Sec. 3.4: any 48-bit value decodes to a point of the lattice."""
    w = synth.words(7, 0, 400000)
    Y, m, g = orc.decode_blocks(synth.words_to_bytes(w))
    assert _membership_numpy(orc, Y).all()
    assert np.array_equal((Y.astype(np.int64) ** 2).sum(axis=1), 16 * m.astype(np.int64))
    assert np.array_equal(g, (w >> np.uint64(47)).astype(np.uint8))
    assert m.max() <= 26 and np.abs(Y).max() <= 10
    for i in range(0, 400000, 997):                       # the C membership test agrees
        assert orc.in_leech(Y[i])
    # rescaled Leech lattice: inner products are multiples of 8, norms of 16
    Z = Y[:3000].astype(np.int64)
    assert np.all((Z @ Z.T) % 8 == 0)
    # the membership test itself rejects near misses
    bad = Y[5].copy(); bad[3] += 2
    assert not orc.in_leech(bad) and not _membership_numpy(orc, bad[None])[0]
    bad = Y[5].copy(); bad[0] += 4
    assert not orc.in_leech(bad) and not _membership_numpy(orc, bad[None])[0]


def test_field_sweeps_stay_in_the_lattice(orc):
    """Sweep every field over its whole range with the others fixed."""
    fields = [(0, 11), (11, 11), (22, 11), (33, 6), (39, 1), (40, 4), (44, 1), (45, 1), (46, 1), (47, 1)]
    assert sum(wd for _, wd in fields) == 48
    base = synth.words(11, 0, 6)
    for b in base.tolist():
        for lo, wd in fields:
            rng = np.arange(1 << wd, dtype=np.uint64)
            w = (np.uint64(b) & ~np.uint64(((1 << wd) - 1) << lo)) | (rng << np.uint64(lo))
            Y, m, g = orc.decode_blocks(synth.words_to_bytes(w))
            assert _membership_numpy(orc, Y).all()
            if lo != 47:                                   # the gain bit does not move the point
                assert len({bytes(r) for r in Y}) == len(w)


def test_distinct_words_give_distinct_points(orc):
    """Brute force on sub-cubes of the code space (gain bit aside)."""
    def word(i1, i2, i3, s8, b1, b2, b3, p, r):
        return (i1 | i2 << 11 | i3 << 22 | s8 << 33 | b1 << 39 | b2 << 40 | b3 << 44 | p << 45 | r << 46)
    ws = [word(i1, i2, i3, s8, b1, b2, b3, p, r)
          for i1 in (0, 1, 2047) for i2 in (0, 5, 1239, 1240, 2047) for i3 in (0, 3)
          for s8 in (0, 37) for b1 in (0, 1) for b2 in (0, 9) for b3 in (0, 1)
          for p in (0, 1) for r in (0, 1)]
    Y, _, _ = orc.decode_blocks(synth.words_to_bytes(np.array(ws, dtype=np.uint64)))
    assert len({bytes(r) for r in Y}) == len(ws) == 1920
    # a dense corner: all of i1 x 8 values of i3, one trellis path
    ws = np.array([word(i1, 0, i3, 0, 0, 0, 0, 0, 0) for i1 in range(2048) for i3 in range(8)], dtype=np.uint64)
    Y, _, _ = orc.decode_blocks(synth.words_to_bytes(ws))
    assert len({bytes(r) for r in Y}) == len(ws)


# ---------------------------------------------------------------- blob
def test_table_blob_layout(orc):
    blob = orc.table_blob()
    assert len(blob) == 18816                             # Sec. 3.4
    rows = np.frombuffer(blob[:16384], dtype="<u4")
    assert np.array_equal(rows, orc.rows)
    assert blob[16384:16512] == orc.prefixes.tobytes()
    assert np.array_equal(np.frombuffer(blob[16512:18560], dtype="<u2"), orc.branches)
    assert blob[18560:18688] == orc.suffixes.tobytes()
    rs = np.frombuffer(blob[18688:], dtype="<f4")
    assert rs[0] == 0.0                                   # the origin needs no special case
    m = np.arange(1, 32, dtype=np.float64)
    assert np.array_equal(rs[1:], (1.0 / np.sqrt(16.0 * m)).astype(np.float32))


def test_golden_regression(orc):
    """Freeze the readings: hashes and decodes written by tests/golden/make_golden.py
    (which calls the oracle only)."""
    lines = [l.split() for l in open(os.path.join(GOLDEN, "oracle_freeze.txt")) if l.strip() and l[0] != "#"]
    blob = orc.table_blob()
    for kind, *rest in lines:
        if kind == "sha256":
            name, lo, hi, digest = rest
            assert hashlib.sha256(blob[int(lo):int(hi)]).hexdigest() == digest, name
        elif kind == "decode":
            word, m, g, *ys = rest
            y, mm, gg = orc.decode_word(int(word, 16))
            assert (y.tolist(), mm, gg) == ([int(v) for v in ys], int(m), int(g))


# ---------------------------------------------------------------- product
def _dense_from_blocks(orc, codes, sigma, gain):
    N, B, _ = codes.shape
    Y, m, g = orc.decode_blocks(codes.reshape(-1, 6))
    scale = np.where(m > 0, gain.astype(np.float64)[g] / np.sqrt(16.0 * np.maximum(m, 1)), 0.0)
    W = (Y.astype(np.float64) * scale[:, None]).reshape(N, B * 24)
    return W * sigma.astype(np.float64)[:, None]


@pytest.mark.parametrize("N,B,ntail", [(5, 3, 0), (16, 7, 16), (33, 10, 8)])
def test_gemv_equals_generic_dense_product(orc, N, B, ntail):
    """Eq. (2) + Sec. 5.1 against numpy's dense product on the decoded matrix."""
    codes = synth.codes(3, N, N, B)
    sigma = synth.row_scales(3, N, N)
    gain = synth.DEFAULT_GAIN
    x = synth.activations(3, N, 24 * B + ntail)[0]
    tail = synth.tails(3, N, sigma, ntail) if ntail else None
    res = orc.gemv(codes.reshape(N, -1), sigma, gain, x, tail)
    W = _dense_from_blocks(orc, codes, sigma, gain)
    if ntail:
        W = np.concatenate([W, tail.astype(np.float64)], axis=1)
    xd = x.astype(np.float64)
    want = W @ xd
    assert np.allclose(res["y"], want, rtol=1e-12, atol=1e-15)
    assert np.allclose(res["termnorm"], np.sqrt(((W * xd) ** 2).sum(axis=1)), rtol=1e-12)
    assert np.allclose(res["abssum"], np.abs(W * xd).sum(axis=1), rtol=1e-12)
    # threads do not change the result
    res2 = orc.gemv(codes.reshape(N, -1), sigma, gain, x, tail, threads=4)
    assert np.array_equal(res["y"], res2["y"])


def test_gemv_special_cases(orc):
    N, B = 6, 4
    codes = synth.codes(5, 1, N, B)
    sigma = synth.row_scales(5, 1, N)
    gain = np.array([2.0, 3.0], dtype=np.float32)
    W = _dense_from_blocks(orc, codes, sigma, gain)
    for k in (0, 23, 24, 95):                             # unit vectors pick single weights
        x = np.zeros(24 * B); x[k] = 1.0
        assert np.allclose(orc.gemv(codes.reshape(N, -1), sigma, gain, x)["y"], W[:, k], rtol=1e-13)
    zero = np.zeros((N, B * 6), dtype=np.uint8)           # origin blocks contribute nothing
    x = synth.activations(5, 1, 24 * B)[0]
    assert not orc.gemv(zero, sigma, gain, x)["y"].any()
    # |w| of a block is gain * sigma (Eq. (2)): check through row norms
    Y, m, g = orc.decode_blocks(codes.reshape(-1, 6))
    blocknorm = np.sqrt((W.reshape(N, B, 24) ** 2).sum(axis=2))
    want = gain.astype(np.float64)[g].reshape(N, B) * sigma.astype(np.float64)[:, None]
    assert np.allclose(blocknorm, np.where(m.reshape(N, B) > 0, want, 0.0), rtol=1e-12)
    # padded rows: bytes beyond 6 B of a row are ignored
    padded = np.zeros((N, 32), dtype=np.uint8); padded[:, :24] = codes.reshape(N, -1); padded[:, 24:] = 0xAB
    assert np.array_equal(orc.gemv(padded, sigma, gain, x)["y"], orc.gemv(codes.reshape(N, -1), sigma, gain, x)["y"])
