"""Checks of GPU results against the CPU oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.

The tolerance of the decode-and-multiply outputs, the seeded inputs of one
product, and the oracle's FP64 reference for them.  Imported by the tests, by
the smoke check and by the bench harness's in-run verification; the CUDA
library and its Python binding never import it.  The input generators come
from the package's synth module, which holds no arithmetic of the method.
"""
import numpy as np

from paper_2609_35465_b200 import synth

# Tolerance of a GEMV output vector y against the FP64 oracle:
#   relative L2 error <= REL_L2, and for every row n
#   |delta_n| <= ABS_COEF * sqrt(sum_k (s_n w_nk x_k)^2) + ABS_FLOOR.
REL_L2 = 1e-3
ABS_COEF = 1e-3
ABS_FLOOR = 1e-6


def make_matrix(seed, stream, N, K, tail_mode, batch=1):
    """Host-side inputs of one product.  tail_mode: the paper's rule (floor(K/24)
    words + float16 tail, Sec. 4.1); otherwise ceil(K/24) words and x zero-extended."""
    ntail = K % 24 if tail_mode else 0
    B = K // 24 if tail_mode else -(-K // 24)
    codes = synth.codes(seed, stream, N, B)
    sigma = synth.row_scales(seed, stream, N)
    x = synth.activations(seed, stream, K, batch)
    tail = synth.tails(seed, stream, sigma, ntail) if ntail else None
    return dict(N=N, K=K, B=B, ntail=ntail, codes=codes, sigma=sigma, x=x, tail=tail)


def oracle_product(orc, m, gain, rows=None, batch_index=0, threads=8):
    """FP64 reference (Eq. (2), Sec. 5.1) for all rows, or for the listed rows only."""
    codes = m["codes"].reshape(m["N"], -1)
    sigma, tail = m["sigma"], m["tail"]
    if rows is not None:
        codes, sigma = codes[rows], sigma[rows]
        tail = tail[rows] if tail is not None else None
    x = m["x"][batch_index].astype(np.float64)
    xpad = np.zeros(24 * m["B"] + m["ntail"])
    xpad[:min(len(x), len(xpad))] = x[:len(xpad)]
    return orc.gemv(codes, sigma, gain, xpad, tail, threads=threads)


def gemv_errors(y_gpu, ref):
    """(relative L2 error, largest |delta_n| as a fraction of its bound)."""
    y_gpu = np.asarray(y_gpu, dtype=np.float64)
    d = y_gpu - ref["y"]
    rel = np.linalg.norm(d) / max(np.linalg.norm(ref["y"]), 1e-300)
    bound = ABS_COEF * ref["termnorm"] + ABS_FLOOR
    return float(rel), float(np.max(np.abs(d) / bound))


def assert_gemv_close(y_gpu, ref, what=""):
    rel, worst = gemv_errors(y_gpu, ref)
    assert rel <= REL_L2, "%s: relative L2 error %.3e" % (what, rel)
    assert worst <= 1.0, "%s: worst element at %.3f of its bound" % (what, worst)
    return rel, worst
