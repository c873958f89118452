"""Workload shapes and byte accounting for the Tetra projections.

Shapes are those of the dense Qwen3 models' seven projections per layer
(Sec. 4.1); a matrix is N output rows by K inputs, stored as floor(K/24)
48-bit words per row plus a tail of K mod 24 unquantized weights (Sec. 4.1),
or, in zero-pad mode, as ceil(K/24) words with x read as zero beyond K.
"""
from dataclasses import dataclass
from typing import List

BLOCK = 24          # weights per 48-bit word
WORD_BYTES = 6


@dataclass(frozen=True)
class Matrix:
    name: str
    N: int
    K: int

    @property
    def blocks(self) -> int:          # tail mode
        return self.K // BLOCK

    @property
    def ntail(self) -> int:
        return self.K % BLOCK

    @property
    def blocks_padded(self) -> int:   # zero-pad mode
        return -(-self.K // BLOCK)


@dataclass(frozen=True)
class Model:
    name: str
    layers: int
    hidden: int
    intermediate: int
    q_heads: int
    kv_heads: int
    head_dim: int = 128

    def layer_matrices(self) -> List[Matrix]:
        q = self.q_heads * self.head_dim
        kv = self.kv_heads * self.head_dim
        h, i = self.hidden, self.intermediate
        return [Matrix("q", q, h), Matrix("k", kv, h), Matrix("v", kv, h), Matrix("o", h, q),
                Matrix("gate", i, h), Matrix("up", i, h), Matrix("down", h, i)]

    def all_matrices(self) -> List[Matrix]:
        out = []
        for layer in range(self.layers):
            for m in self.layer_matrices():
                out.append(Matrix("L%d.%s" % (layer, m.name), m.N, m.K))
        return out


QWEN3_4B = Model("qwen3-4b", 36, 2560, 9728, 32, 8)
QWEN3_8B = Model("qwen3-8b", 36, 4096, 12288, 32, 8)
QWEN3_14B = Model("qwen3-14b", 40, 5120, 17408, 40, 8)
MODELS = {m.name: m for m in (QWEN3_4B, QWEN3_8B, QWEN3_14B)}

CONFIG0 = Matrix("config0", 2048, 2304)
CONFIG4 = Matrix("down8b", 4096, 12288)
CONFIG4_BATCHES = (1, 2, 4, 8, 16)


def file_bytes(m: Matrix, tail_bytes: int = 4, scale_bytes: int = 4, row_pad: int = 1) -> int:
    """Bytes one matrix occupies: words + tail + one scale per row, each row of
    words padded to a multiple of row_pad bytes."""
    row = -(-(m.blocks * WORD_BYTES) // row_pad) * row_pad
    return m.N * (row + m.ntail * tail_bytes + scale_bytes)


def weights(m: Matrix) -> int:
    return m.N * m.K
