"""Philox4x32-10, written from its published definition.

Source: J. Salmon, M. Moraes, R. Dror, D. Shaw, "Parallel random numbers: as
easy as 1, 2, 3", SC'11, Section 3.3 (the Philox S-P network) and the
constants of its Table 2 row "Philox4x32".

One call maps a 128-bit counter (c0, c1, c2, c3) and a 64-bit key (k0, k1) to
four 32-bit words.  Ten rounds; the key is bumped by the Weyl constants before
every round but the first.

This is test infrastructure (see the package docstring).
"""
import numpy as np

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = np.uint64(0x9E3779B9)   # golden ratio
_W1 = np.uint64(0xBB67AE85)   # sqrt(3) - 1
_MASK = np.uint64(0xFFFFFFFF)
_S32 = np.uint64(32)


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Return the four output words as uint64 arrays holding 32-bit values.

    All arguments broadcast against each other; each is taken modulo 2**32.
    """
    c0, c1, c2, c3, k0, k1 = (np.asarray(a, dtype=np.uint64) & _MASK
                              for a in (c0, c1, c2, c3, k0, k1))
    c0, c1, c2, c3, k0, k1 = np.broadcast_arrays(c0, c1, c2, c3, k0, k1)
    for r in range(10):
        if r > 0:
            k0 = (k0 + _W0) & _MASK
            k1 = (k1 + _W1) & _MASK
        p0 = _M0 * c0            # 32x32 -> 64 bit product, exact in uint64
        p1 = _M1 * c2
        hi0, lo0 = p0 >> _S32, p0 & _MASK
        hi1, lo1 = p1 >> _S32, p1 & _MASK
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
    return c0, c1, c2, c3


def philox_scalar(counter, key):
    """Pure-Python-int version of one block, for reading against the paper."""
    c = [int(w) & 0xFFFFFFFF for w in counter]
    k = [int(w) & 0xFFFFFFFF for w in key]
    for r in range(10):
        if r > 0:
            k[0] = (k[0] + 0x9E3779B9) & 0xFFFFFFFF
            k[1] = (k[1] + 0xBB67AE85) & 0xFFFFFFFF
        p0 = 0xD2511F53 * c[0]
        p1 = 0xCD9E8D57 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & 0xFFFFFFFF,
             (p0 >> 32) ^ c[3] ^ k[1], p0 & 0xFFFFFFFF]
    return tuple(c)
