"""Gaussian test matrix of the random projection (Section 3.1, "Subspace Preservation via Random Projection").

Test infrastructure: a slow restatement used to check the CUDA library; never on the product path.

The paper asks for a Gaussian matrix Omega with (hidden dim) rows and k+s columns.  To make it
reproducible bit for bit, entry (i, j) is the standard normal quantile at one of 65536 equally
likely levels chosen by the 16-bit Philox draw of the entry's index, rounded to bfloat16:

    Omega[i, j] = bf16( Phi^-1( (u + 0.5) / 65536 ) ),   u = draw_u16(i*q + j, seed, stream 0x100)
"""
import numpy as np
from scipy.special import ndtri

from . import philox


def round_to_bf16(x):
    """Round float64/float32 values to the nearest bfloat16 (ties to even); returns float32."""
    f = np.asarray(x, dtype=np.float32)
    # the float64 -> float32 step above is exact for every value this module produces only if it
    # does not sit on a bf16 tie after rounding; the quantile table is checked for that in tests
    b = f.view(np.uint32).astype(np.uint64)
    lsb = (b >> np.uint64(16)) & np.uint64(1)
    b = (b + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    return b.astype(np.uint32).view(np.float32).reshape(f.shape)


def quantile_level(u16):
    """bf16-rounded standard normal quantile of level (u + 0.5)/65536, as float32."""
    p = (np.asarray(u16, dtype=np.float64) + 0.5) / 65536.0
    return round_to_bf16(ndtri(p))


def omega(n, q, seed, stream=philox.STREAM_OMEGA):
    """The n x q test matrix as float32 holding bf16-representable values."""
    idx = np.arange(n, dtype=np.uint64)[:, None] * np.uint64(q) + np.arange(q, dtype=np.uint64)[None, :]
    return quantile_level(philox.draw_u16(idx, seed, stream))
