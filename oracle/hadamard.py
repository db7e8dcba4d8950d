"""Random Hadamard transform + NVFP4 with stochastic rounding: the comparison recipe of Section 4 and of the
appendix on the implementation of NVFP4 and the vendor's recipe (the paper compares Metis with "a random Hadamard
transform alongside SR"; it gives neither the transform size nor the sign source).

Test infrastructure: a slow restatement used to check the CUDA library; never on the product path.

Reading used here: the transform acts on blocks of 16 consecutive elements along the contraction axis - the NVFP4
block - as  y = H16 (s * x) / 4  with H16 the Sylvester Hadamard matrix and s a vector of random signs, one per
position along the contraction axis, shared by every row and by both operands of a product, so that
(x H D)(w H D)^T = x w^T.  Sign of position c: bit 15 of the 16-bit Philox draw of index c, stream 0x300.
The transform is evaluated as four butterfly stages in binary32 (distance 1, 2, 4, 8; (a, b) -> (a + b, a - b)),
then one exact multiplication by 1/4: this order is the definition, so the bytes can be compared bit for bit.
"""
import numpy as np

from . import nvfp4, philox

STREAM_SIGNS = 0x300
F32 = np.float32


def signs(n, seed):
    """+-1 per position along the contraction axis."""
    u = philox.draw_u16(np.arange(n, dtype=np.uint64), seed, STREAM_SIGNS)
    return np.where((u >> 15) & 1, F32(-1.0), F32(1.0)).astype(F32)


def rht(x, seed):
    """Random Hadamard transform of every 16-block of the last axis (binary32 butterflies)."""
    x = np.asarray(x, dtype=F32)
    rows, cols = x.shape
    assert cols % 16 == 0
    v = (x * signs(cols, seed)[None, :]).reshape(rows, cols // 16, 16).copy()
    for h in (1, 2, 4, 8):
        w = v.reshape(rows, cols // 16, 16 // (2 * h), 2, h)
        a, b = w[:, :, :, 0, :].copy(), w[:, :, :, 1, :].copy()
        w[:, :, :, 0, :] = a + b
        w[:, :, :, 1, :] = a - b
    return (v * F32(0.25)).reshape(rows, cols)


def rht_inverse(y, seed):
    """Inverse of rht in float64 (H16/4 is symmetric and orthogonal: the inverse is the same butterfly, then the signs)."""
    y = np.asarray(y, dtype=np.float64)
    rows, cols = y.shape
    v = y.reshape(rows, cols // 16, 16).copy()
    for h in (1, 2, 4, 8):
        w = v.reshape(rows, cols // 16, 16 // (2 * h), 2, h)
        a, b = w[:, :, :, 0, :].copy(), w[:, :, :, 1, :].copy()
        w[:, :, :, 0, :] = a + b
        w[:, :, :, 1, :] = a - b
    return (v * 0.25).reshape(rows, cols) * signs(cols, seed).astype(np.float64)[None, :]


def quantize_rht(x, rounding=nvfp4.ROUND_SR, seed=0, stream=philox.STREAM_RESIDUAL):
    """NVFP4 (blocks along the columns, own amax/2688 tensor scale) of the transformed tensor; stochastic rounding by default."""
    return nvfp4.quantize(rht(x, seed), nvfp4.AXIS_COLS, rounding, seed, stream)


def fake_quantize_rht(x, rounding=nvfp4.ROUND_SR, seed=0):
    """Quantize in the rotated basis and come back: what the recipe makes of x, in x's own coordinates (float64)."""
    return rht_inverse(nvfp4.dequantize(*quantize_rht(x, rounding, seed)), seed)
