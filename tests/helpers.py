"""Shared pieces of the GPU parity tests: seeded inputs for one matrix and the
tolerance check of the GEMV outputs against the FP64 oracle."""
import numpy as np

from paper_2609_35465_b200 import synth

REL_L2 = 1e-3          # relative L2 error of a whole output vector
ABS_COEF = 1e-3        # |delta_n| <= ABS_COEF * sqrt(sum_k (s_n w_nk x_k)^2) + ABS_FLOOR
ABS_FLOOR = 1e-6


def make_matrix(seed, stream, N, K, tail_mode, batch=1):
    """Host-side inputs of one product.  tail_mode: the paper's rule (floor(K/24)
    words + float16 tail); otherwise ceil(K/24) words and x zero-extended."""
    ntail = K % 24 if tail_mode else 0
    B = K // 24 if tail_mode else -(-K // 24)
    codes = synth.codes(seed, stream, N, B)
    sigma = synth.row_scales(seed, stream, N)
    x = synth.activations(seed, stream, K, batch)
    tail = synth.tails(seed, stream, sigma, ntail) if ntail else None
    return dict(N=N, K=K, B=B, ntail=ntail, codes=codes, sigma=sigma, x=x, tail=tail)


def oracle_product(orc, m, gain, rows=None, batch_index=0, threads=8):
    """FP64 reference for all rows, or for the listed rows only."""
    codes = m["codes"].reshape(m["N"], -1)
    sigma, tail = m["sigma"], m["tail"]
    if rows is not None:
        codes, sigma = codes[rows], sigma[rows]
        tail = tail[rows] if tail is not None else None
    x = m["x"][batch_index].astype(np.float64)
    xpad = np.zeros(24 * m["B"] + m["ntail"])
    xpad[:min(len(x), len(xpad))] = x[:len(xpad)]
    return orc.gemv(codes, sigma, gain, xpad, tail, threads=threads)


def assert_gemv_close(y_gpu, ref, what=""):
    y_gpu = np.asarray(y_gpu, dtype=np.float64)
    d = y_gpu - ref["y"]
    rel = np.linalg.norm(d) / max(np.linalg.norm(ref["y"]), 1e-300)
    bound = ABS_COEF * ref["termnorm"] + ABS_FLOOR
    worst = float(np.max(np.abs(d) / bound))
    assert rel <= REL_L2, "%s: relative L2 error %.3e" % (what, rel)
    assert worst <= 1.0, "%s: worst element at %.3f of its bound" % (what, worst)
    return rel, worst
