"""Seeded synthetic inputs for the Tetra decode-and-multiply path.

This module holds no arithmetic of the method: it only draws numbers.  Both
the CPU oracle's callers and the CUDA path's callers take their inputs from
here, so the two sides see identical bytes.

Recipe (the inputs stand in for the paper's Qwen3 projection matrices, which
are not available; shapes follow the Qwen3 dense models, Sec. 4.1):
  * codes: every 48-bit value is a legal word (Sec. 3.4), so a word is 48
    uniform random bits -- each field uniform over its range, the trellis
    path a uniform walk.  Word k of stream (seed, matrix) is the top 48 bits
    of splitmix64 applied to a counter; stored as six little-endian bytes.
  * row scales: float32 exp(-4 + 0.3 z), z ~ N(0, 1).
  * activations x: float16 N(0, 1).
  * unquantized tail (K mod 24 weights per row, Sec. 4.1): float16(sigma_n z),
    the magnitude of a scaled decoded weight.
Normal variates are Box-Muller over the same counter-based generator.
"""
import numpy as np

_MASK = np.uint64(0xFFFFFFFFFFFFFFFF)


def splitmix64(x: np.ndarray) -> np.ndarray:
    """The splitmix64 output function applied elementwise to uint64 counters."""
    with np.errstate(over="ignore"):
        z = (x + np.uint64(0x9E3779B97F4A7C15)) & _MASK
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        return z ^ (z >> np.uint64(31))


def _stream_base(seed: int, stream: int, purpose: int) -> np.uint64:
    """A well-mixed 64-bit offset for (seed, stream, purpose)."""
    key = np.array([(seed & 0xFFFFFFFF) | ((stream & 0xFFFFFF) << 32) | ((purpose & 0xFF) << 56)],
                   dtype=np.uint64)
    return splitmix64(splitmix64(key))[0]


def raw_u64(seed: int, stream: int, purpose: int, n: int, start: int = 0) -> np.ndarray:
    """n uint64 draws, counters start..start+n-1 of the given stream."""
    base = _stream_base(seed, stream, purpose)
    with np.errstate(over="ignore"):
        ctr = (np.arange(start, start + n, dtype=np.uint64) + base) & _MASK
    return splitmix64(ctr)


def words(seed: int, stream: int, n: int, start: int = 0) -> np.ndarray:
    """n uniform 48-bit Tetra words as uint64."""
    return raw_u64(seed, stream, 0, n, start) >> np.uint64(16)


def words_to_bytes(w: np.ndarray) -> np.ndarray:
    """uint64 words -> uint8 [n, 6], little-endian."""
    w = np.ascontiguousarray(w, dtype="<u8")
    return np.ascontiguousarray(w.view(np.uint8).reshape(-1, 8)[:, :6])


def bytes_to_words(b: np.ndarray) -> np.ndarray:
    """uint8 [n, 6] -> uint64 words."""
    b = np.ascontiguousarray(b, dtype=np.uint8).reshape(-1, 6)
    out = np.zeros((b.shape[0], 8), dtype=np.uint8)
    out[:, :6] = b
    return out.view("<u8").reshape(-1)


def codes(seed: int, stream: int, N: int, B: int) -> np.ndarray:
    """File-order codes of an N x (24 B) matrix: uint8 [N, B, 6]."""
    out = np.empty((N * B, 6), dtype=np.uint8)
    step = 1 << 22
    for s in range(0, N * B, step):
        n = min(step, N * B - s)
        out[s:s + n] = words_to_bytes(words(seed, stream, n, s))
    return out.reshape(N, B, 6)


def normal(seed: int, stream: int, purpose: int, n: int) -> np.ndarray:
    """n standard normal float64 draws (Box-Muller)."""
    u = raw_u64(seed, stream, purpose, 2 * n)
    u1 = ((u[:n] >> np.uint64(11)).astype(np.float64) + 1.0) * (1.0 / 9007199254740992.0)  # (0, 1]
    u2 = (u[n:] >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def row_scales(seed: int, stream: int, N: int) -> np.ndarray:
    """float32 lognormal(mu = -4, sigma = 0.3) row scales."""
    return np.exp(-4.0 + 0.3 * normal(seed, stream, 1, N)).astype(np.float32)


def activations(seed: int, stream: int, K: int, batch: int = 1) -> np.ndarray:
    """float16 N(0, 1) activations, shape [batch, K]."""
    return normal(seed, stream, 2, batch * K).astype(np.float16).reshape(batch, K)


def tails(seed: int, stream: int, sigma: np.ndarray, ntail: int) -> np.ndarray:
    """float16 unquantized tail weights, shape [N, ntail]."""
    N = sigma.shape[0]
    z = normal(seed, stream, 3, N * ntail).reshape(N, ntail)
    return (sigma.astype(np.float64)[:, None] * z).astype(np.float16)


# Two-level Lloyd-Max quantiser of the length of a standard normal vector in
# 24 dimensions; the paper does not print its two gain values, and both the
# oracle and the CUDA path simply read whatever pair they are given.
DEFAULT_GAIN = np.array([4.3156, 5.4415], dtype=np.float32)


# ---------------------------------------------------------------------------
# The same code stream generated with torch ops (on any device), for workloads
# too large to draw on the host in reasonable time.  Bit-identical to codes().
# ---------------------------------------------------------------------------
def _s64(v: int) -> int:
    v &= 0xFFFFFFFFFFFFFFFF
    return v - (1 << 64) if v >= (1 << 63) else v


def codes_torch(seed: int, stream: int, N: int, B: int, device="cpu"):
    """File-order codes uint8 [N, B, 6] as a torch tensor on `device`."""
    import torch

    def lsr(z, k):  # logical shift right of int64 bit patterns
        return (z >> k) & ((1 << (64 - k)) - 1)

    base = int(_stream_base(seed, stream, 0))
    n = N * B
    z = torch.arange(n, dtype=torch.int64, device=device) + _s64(base)
    z = z + _s64(0x9E3779B97F4A7C15)
    z = (z ^ lsr(z, 30)) * _s64(0xBF58476D1CE4E5B9)
    z = (z ^ lsr(z, 27)) * _s64(0x94D049BB133111EB)
    z = z ^ lsr(z, 31)
    w = lsr(z, 16)
    return w.view(torch.uint8).reshape(n, 8)[:, :6].contiguous().reshape(N, B, 6)


# ---------------------------------------------------------------------------
# 4-bit group-quantised matrices (int4 projections, embedding table, output head)
# ---------------------------------------------------------------------------
def q4_nibbles(seed: int, stream: int, N: int, K: int) -> np.ndarray:
    """uint8 [N, K/2]: two uniform 4-bit weights per byte (weight 2b in the low nibble)."""
    n = N * (K // 2)
    w = raw_u64(seed, stream, 11, (n + 7) // 8)
    return w.view(np.uint8)[:n].reshape(N, K // 2).copy()


def q4_scales_offsets(seed: int, stream: int, N: int, groups: int):
    """float16 [N, groups] each: scale = exp(-5 + 0.3 z) (about a weight range of 0.1 over 15 steps),
    offset = -scale * (7.5 + 0.5 z'), so that the weights of a group straddle zero."""
    z = normal(seed, stream, 12, N * groups)
    z2 = normal(seed, stream, 13, N * groups)
    scale = np.exp(-5.0 + 0.3 * z).astype(np.float16)
    offset = (-(scale.astype(np.float64)) * (7.5 + 0.5 * z2)).astype(np.float16)
    return scale.reshape(N, groups), offset.reshape(N, groups)


def token_ids(seed: int, stream: int, count: int, vocab: int) -> np.ndarray:
    """int32 [count]: uniform row numbers."""
    return (raw_u64(seed, stream, 14, count) % np.uint64(vocab)).astype(np.int32)
