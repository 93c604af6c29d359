"""Comparison helpers for the CUDA-vs-oracle parity tests."""
import math

import numpy as np


def assert_codes_match(gpu_codes, ref_codes, x, mult, what):
    """Codes must be identical except where x*mult lies within 1e-6 of a rounding tie.

    mult is the per-row float64 multiplier of the quantiser (sqrt7/(beta+eps) or 127/(gamma+eps)).
    """
    gpu_codes = np.asarray(gpu_codes)
    bad = np.argwhere(gpu_codes != ref_codes)
    for m, j in bad:
        v = float(x[m, j]) * float(mult[m])
        assert abs(abs(v - math.floor(v)) - 0.5) < 1e-6 and abs(int(gpu_codes[m, j]) - int(ref_codes[m, j])) == 1, (
            f"{what}: code mismatch at {(m, j)}: gpu {gpu_codes[m, j]} ref {ref_codes[m, j]} v={v!r}")
    return len(bad)


def max_rel_err(y_gpu, y_ref):
    """Element-wise |a-b|/|b| with exact zeros required to match exactly."""
    y_gpu = np.asarray(y_gpu, np.float64)
    zero = y_ref == 0
    assert (y_gpu[zero] == 0).all(), "an exact-zero output is non-zero on the GPU"
    nz = ~zero
    if not nz.any():
        return 0.0
    return float((np.abs(y_gpu[nz] - y_ref[nz]) / np.abs(y_ref[nz])).max())


def unpack_mask_bits(bits, K):
    """uint32 [M, ceil(K/32)] bitmap -> uint8 [M, K]."""
    b = np.asarray(bits).view(np.uint32)
    M = b.shape[0]
    out = ((b[:, :, None] >> np.arange(32, dtype=np.uint32)[None, None, :]) & 1).astype(np.uint8)
    return out.reshape(M, -1)[:, :K]
