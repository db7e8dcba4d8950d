"""NVFP4 encoder / decoder of the oracle (Section 2.3, "Quantization Bias"; Appendix C.1).

Test infrastructure: a slow restatement used to check the CUDA library; never on the product path.

Format as the paper states it: values are partitioned into blocks of 16; each block gets one
E4M3 scale derived from the largest magnitude in the block and rounded UP to the next
representable E4M3 value, so the block is always covered; each element becomes round(e/s)*s
with round() onto the E2M1 set +-{0, 0.5, 1, 1.5, 2, 3, 4, 6}.  Added on top (the paper has block scales only): one FP32 scale
per tensor, s_T = amax/(6*448), so the E4M3 block scales use their whole range.

The defined arithmetic is IEEE binary32, round to nearest even, no fused multiply-add, denormals
kept, in exactly this order (numpy float32 scalar/array ops satisfy it):

  1. s_T = amax_T / 2688          (1.0 if amax_T == 0), or a given value
  2. per block: t = amax_b / (6 * s_T); t = min(t, 448)
  3. s_b = smallest non-negative finite E4M3 value >= t
  4. s_b == 0: magnitudes 0, signs kept.  Else r = 1 / (s_b * s_T); y = x * r
  5. code = sign(y) | E2M1 magnitude of |y| by round-to-nearest-even (ties to the even code,
     |y| > 6 saturates) or by stochastic rounding (below)

Stochastic rounding (Section 4 applies it by default; mechanics are this build's reading):
a = min(|y|, 6); lo/hi = E2M1 neighbours with lo <= a < hi; f = (a - lo)/(hi - lo), exact in
binary32; with a 16-bit draw u the element goes up iff f*65536 > u.  Representable values never
move, P(up) = ceil(f*65536)/65536.  Scales are never stochastic.

A quantized tensor is always returned "K-major": the block axis is the last axis of the stored
arrays.  Blocks along the rows of x are therefore stored as the quantization of x transposed.
"""
import numpy as np

from . import philox

F32 = np.float32
BLOCK = 16
AXIS_COLS = 1      # blocks of 16 consecutive elements inside a row
AXIS_ROWS = 2      # blocks of 16 consecutive elements inside a column
ROUND_RNE = 0
ROUND_SR = 1

E2M1_GRID = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0], dtype=F32)
_E2M1_MID = ((E2M1_GRID[:-1].astype(np.float64) + E2M1_GRID[1:].astype(np.float64)) / 2).astype(F32)


def e4m3_value(code):
    """Value of a non-negative E4M3FN byte 0x00..0x7E (4 exponent bits, bias 7, 3 mantissa bits)."""
    e, f = (code >> 3) & 0xF, code & 7
    if e == 0:
        return f * 2.0 ** -9
    return 2.0 ** (e - 7) * (1.0 + f / 8.0)


E4M3_POS = np.array([e4m3_value(c) for c in range(127)], dtype=F32)   # strictly increasing, 0 .. 448


def e4m3_ceil_code(t):
    """Byte of the smallest E4M3 value >= t (t already clamped to <= 448)."""
    return np.searchsorted(E4M3_POS, np.asarray(t, dtype=F32), side="left").astype(np.uint8)


def e2m1_encode_rne(y):
    """4-bit codes (sign in bit 3) of float32 y, nearest E2M1 value, ties to the even code, saturating."""
    y = np.asarray(y, dtype=F32)
    a = np.abs(y)
    mag = np.zeros(y.shape, dtype=np.uint8)
    for j, mid in enumerate(_E2M1_MID):
        # midpoint j lies between codes j and j+1; a tie goes to whichever of the two is even
        above = (a > mid) | ((a == mid) & (j % 2 == 1))
        mag += above.astype(np.uint8)
    return mag | (np.signbit(y).astype(np.uint8) << 3)


def e2m1_encode_sr(y, u16):
    """Stochastically rounded 4-bit codes of float32 y given one 16-bit draw per element."""
    y = np.asarray(y, dtype=F32)
    a = np.minimum(np.abs(y), F32(6.0))
    lo_idx = np.zeros(y.shape, dtype=np.int64)
    for g in E2M1_GRID[1:]:
        lo_idx += (a >= g)
    top = lo_idx == 7
    lo_c = np.minimum(lo_idx, 6)
    lo = E2M1_GRID[lo_c]
    step = E2M1_GRID[lo_c + 1] - lo
    f = (a - lo) / step                                   # exact: Sterbenz + power-of-two divisor
    up = (f * F32(65536.0)) > np.asarray(u16).astype(F32)
    mag = np.where(top, 7, lo_c + up.astype(np.int64)).astype(np.uint8)
    return mag | (np.signbit(y).astype(np.uint8) << 3)


def tensor_scale_from_amax(amax):
    amax = F32(amax)
    return F32(1.0) if amax == 0 else F32(amax / F32(2688.0))


def quantize(x, axis=AXIS_COLS, rounding=ROUND_RNE, seed=0, stream=philox.STREAM_RESIDUAL, tensor_scale=None,
             index=None):
    """Quantize a 2-D float32 array.  Returns (codes, scales, s_T) in K-major storage.

    codes  uint8 [R, K]     one 4-bit code per byte (pack() halves it)
    scales uint8 [R, K/16]  E4M3 bytes
    s_T    float32
    (R, K) = x.shape for AXIS_COLS and x.T.shape for AXIS_ROWS.  The stochastic-rounding draw of
    an element is keyed by its index in x (row*cols + col) whatever the block axis.  `index` (uint64,
    x's shape) replaces those keys: it lets a slice of a larger tensor be quantized with the draws its
    elements have inside that tensor (addressing only; the arithmetic is the same).
    """
    x = np.asarray(x, dtype=F32)
    rows, cols = x.shape
    if index is None:
        index = np.arange(rows, dtype=np.uint64)[:, None] * np.uint64(cols) + np.arange(cols, dtype=np.uint64)[None, :]
    else:
        index = np.asarray(index, dtype=np.uint64)
        if index.shape != x.shape:
            raise ValueError("index must have the shape of x")
    if axis == AXIS_ROWS:
        x, index = x.T, index.T
    elif axis != AXIS_COLS:
        raise ValueError("axis")
    R, K = x.shape
    if K % BLOCK:
        raise ValueError("block axis length must be a multiple of 16")
    if tensor_scale is None:
        s_T = tensor_scale_from_amax(np.max(np.abs(x)) if x.size else 0.0)
    else:
        s_T = F32(tensor_scale)
    xb = x.reshape(R, K // BLOCK, BLOCK)
    amax_b = np.max(np.abs(xb), axis=2)
    t = amax_b / F32(F32(6.0) * s_T)
    t = np.minimum(t, F32(448.0))
    sc = e4m3_ceil_code(t)
    s_b = E4M3_POS[sc]
    with np.errstate(divide="ignore", invalid="ignore", over="ignore"):
        r = F32(1.0) / (s_b * s_T)
        y = xb * r[:, :, None]
    y = np.where((s_b == 0)[:, :, None], np.copysign(F32(0.0), xb), y).astype(F32)
    y = y.reshape(R, K)
    if rounding == ROUND_RNE:
        codes = e2m1_encode_rne(y)
    elif rounding == ROUND_SR:
        codes = e2m1_encode_sr(y, philox.draw_u16(index, seed, stream))
    else:
        raise ValueError("rounding")
    return codes, sc, s_T


def dequantize(codes, scales, s_T):
    """Exact float64 value E2M1(code) * E4M3(scale) * s_T of every element (K-major storage)."""
    mag = E2M1_GRID.astype(np.float64)[codes & 7]
    val = np.where(codes & 8, -mag, mag)
    sb = E4M3_POS.astype(np.float64)[scales]
    return val * np.repeat(sb, BLOCK, axis=1) * float(s_T)


def pack(codes):
    """Two codes per byte: element 2j in the low nibble, 2j+1 in the high nibble."""
    return (codes[:, 0::2] | (codes[:, 1::2] << 4)).astype(np.uint8)


def unpack(packed):
    out = np.empty((packed.shape[0], packed.shape[1] * 2), dtype=np.uint8)
    out[:, 0::2] = packed & 0xF
    out[:, 1::2] = packed >> 4
    return out


def fake_quantize(x, axis=AXIS_COLS, **kw):
    """Quantize then dequantize, returned in the orientation of x (float64)."""
    c, s, st = quantize(x, axis=axis, **kw)
    d = dequantize(c, s, st)
    return d.T if axis == AXIS_ROWS else d
