"""Philox4x32-10 counter-based generator (Salmon et al., SC'11) and the per-element draw rule.

Test infrastructure: a slow restatement used to check the CUDA library; never on the product path.

The paper applies stochastic rounding (Section 4, "FP4 Training") and a Gaussian test matrix
(Section 3.1, "Subspace Preservation via Random Projection") without fixing a random source.
The reading taken here: every random quantity is a pure function of (seed, stream, logical
element index), so that both sides of a parity test can reproduce it.
"""
import numpy as np

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = 0x9E3779B9
_W1 = 0xBB67AE85
_MASK = np.uint64(0xFFFFFFFF)
_S32 = np.uint64(32)

# stream identifiers (third counter word) of the library's default draws
STREAM_RESIDUAL = 0x10
STREAM_LEFT = 0x11
STREAM_RIGHT = 0x12
STREAM_OMEGA = 0x100
STREAM_SAMPLING = 0x200


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Ten Philox rounds on arrays of 32-bit words held in uint64.  Returns four uint64 arrays (< 2**32)."""
    c0, c1, c2, c3 = (np.asarray(c, dtype=np.uint64) & _MASK for c in (c0, c1, c2, c3))
    c0, c1, c2, c3 = np.broadcast_arrays(c0, c1, c2, c3)
    k0 = int(k0) & 0xFFFFFFFF
    k1 = int(k1) & 0xFFFFFFFF
    for rnd in range(10):
        p0 = _M0 * c0                      # 64-bit products of 32-bit words cannot overflow uint64
        p1 = _M1 * c2
        hi0, lo0 = p0 >> _S32, p0 & _MASK
        hi1, lo1 = p1 >> _S32, p1 & _MASK
        n0 = hi1 ^ c1 ^ np.uint64(k0)
        n2 = hi0 ^ c3 ^ np.uint64(k1)
        c0, c1, c2, c3 = n0, lo1, n2, lo0
        k0 = (k0 + _W0) & 0xFFFFFFFF       # key schedule: bumped between rounds
        k1 = (k1 + _W1) & 0xFFFFFFFF
    return c0, c1, c2, c3


def draw_u16(index, seed, stream):
    """16 random bits for each logical element index.

    counter = (lo32(e>>3), hi32(e>>3), stream, 0), key = (lo32(seed), hi32(seed)); the eight
    elements that share e>>3 take the eight 16-bit halves of the four output words in order
    (word h>>1, low half first), h = e & 7.
    """
    e = np.asarray(index, dtype=np.uint64)
    blk = e >> np.uint64(3)
    w = philox4x32_10(blk & _MASK, blk >> _S32, np.uint64(stream), np.uint64(0),
                      int(seed) & 0xFFFFFFFF, (int(seed) >> 32) & 0xFFFFFFFF)
    h = e & np.uint64(7)
    word = np.choose((h >> np.uint64(1)).astype(np.int64), w)
    shift = (h & np.uint64(1)) * np.uint64(16)
    return ((word >> shift) & np.uint64(0xFFFF)).astype(np.uint32)


def draw_word0(counter0, seed, stream):
    """First output word for counter (counter0, 0, stream, 0); used by the row sampler."""
    w = philox4x32_10(np.asarray(counter0, dtype=np.uint64), np.uint64(0), np.uint64(stream), np.uint64(0),
                      int(seed) & 0xFFFFFFFF, (int(seed) >> 32) & 0xFFFFFFFF)
    return w[0].astype(np.uint64)
