"""Philox4x32-10, the counter-based generator of Salmon, Moraes, Dror and Shaw ("Parallel random
numbers: as easy as 1, 2, 3", SC'11), written out from its published definition.
TEST INFRASTRUCTURE ONLY.

Stochastic rounding (second rounding mode of the Methodology section) needs one uniform number
per tensor element; the paper does not say where they come from.  Here element number i of
an operand takes word (i mod 4) of philox4x32_10(counter = (i div 4 as two 32-bit words,
stream, 0), key = the seed's two 32-bit words), and u = (word >> 8) / 2^24, so that any
implementation reproduces the same draw from (seed, stream, i) alone.
"""
import numpy as np

_M0, _M1 = np.uint64(0xD2511F53), np.uint64(0xCD9E8D57)
_W0, _W1 = np.uint32(0x9E3779B9), np.uint32(0xBB67AE85)
_LO = np.uint64(0xFFFFFFFF)


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Ten rounds on arrays of uint32 counter words with scalar (or array) uint32 key words.
    One round: (hi0, lo0) = M0 * c0, (hi1, lo1) = M1 * c2 as 64-bit products;
    c <- (hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0); then the key is bumped by the Weyl constants."""
    c0, c1, c2, c3 = (np.asarray(c, dtype=np.uint32) for c in (c0, c1, c2, c3))
    k0, k1 = np.uint32(k0), np.uint32(k1)
    with np.errstate(over="ignore"):
        for _ in range(10):
            p0 = _M0 * c0.astype(np.uint64)
            p1 = _M1 * c2.astype(np.uint64)
            hi0, lo0 = (p0 >> np.uint64(32)).astype(np.uint32), (p0 & _LO).astype(np.uint32)
            hi1, lo1 = (p1 >> np.uint64(32)).astype(np.uint32), (p1 & _LO).astype(np.uint32)
            c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
            k0, k1 = np.uint32(k0 + _W0), np.uint32(k1 + _W1)
    return c0, c1, c2, c3


def element_uniforms(shape, seed, stream):
    """u in [0, 1) with 24 bits for every element of an array of this shape, numbered in C order."""
    n = int(np.prod(shape, dtype=np.int64))
    i = np.arange(n, dtype=np.uint64)
    blk = i >> np.uint64(2)
    words = philox4x32_10((blk & _LO).astype(np.uint32), (blk >> np.uint64(32)).astype(np.uint32),
                          np.full(n, stream, np.uint32), np.zeros(n, np.uint32),
                          np.uint32(seed & 0xFFFFFFFF), np.uint32((seed >> 32) & 0xFFFFFFFF))
    w = np.choose((i & np.uint64(3)).astype(np.int64), words)
    return ((w >> np.uint32(8)).astype(np.float64) / 2.0 ** 24).reshape(shape)
