"""Philox4xW-10 counter-based random number generator (oracle side).

Test infrastructure only.  Restates the algorithm of Salmon, Moraes, Dror and
Shaw, "Parallel random numbers: as easy as 1, 2, 3" (SC'11): a 4-word counter
is passed through 10 rounds; each round multiplies words 0 and 2 by two fixed
odd constants, takes the high and low halves of the double-width products,
xors the high halves with words 1 and 3 and with the two key words, and
permutes; the key is bumped by two Weyl constants after every round.

``philox4x32_10`` (vectorised, 32-bit words) is what the GRBS mask uses.
``philox4_generic`` (scalar Python integers, any word width) exists so that the
same round structure can be pinned against NumPy's Philox4x64 bit generator.
"""
import numpy as np

# multipliers and Weyl key increments published with the algorithm
_MULT = {32: (0xD2511F53, 0xCD9E8D57),
         64: (0xD2E7470EE14C6C93, 0xCA5A826395121157)}
_WEYL = {32: (0x9E3779B9, 0xBB67AE85),
         64: (0x9E3779B97F4A7C15, 0xBB67AE8584CAA73B)}


def philox4_generic(W, key, ctr, rounds=10):
    """One Philox4xW block with Python integers.

    key: 2 words, ctr: 4 words, each in [0, 2**W).  Returns the 4 output words.
    """
    mask = (1 << W) - 1
    M0, M1 = _MULT[W]
    W0, W1 = _WEYL[W]
    c0, c1, c2, c3 = (int(v) & mask for v in ctr)
    k0, k1 = (int(v) & mask for v in key)
    for _ in range(rounds):
        prod0 = M0 * c0
        prod1 = M1 * c2
        hi0, lo0 = prod0 >> W, prod0 & mask
        hi1, lo1 = prod1 >> W, prod1 & mask
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
        k0 = (k0 + W0) & mask
        k1 = (k1 + W1) & mask
    return [c0, c1, c2, c3]


def philox4x32_10(key0, key1, c0, c1, c2, c3):
    """Vectorised Philox4x32-10.

    All arguments broadcast against each other and are taken modulo 2**32.
    Returns a tuple of four uint32 arrays (the four output words).
    """
    u64 = np.uint64
    lo32 = u64(0xFFFFFFFF)
    sh = u64(32)
    c0, c1, c2, c3, k0, k1 = np.broadcast_arrays(
        *[np.asarray(v, dtype=np.uint64) & lo32 for v in (c0, c1, c2, c3, key0, key1)])
    M0, M1 = (u64(v) for v in _MULT[32])
    W0, W1 = (u64(v) for v in _WEYL[32])
    for _ in range(10):
        prod0 = M0 * c0          # < 2**64: both factors are below 2**32
        prod1 = M1 * c2
        hi0, lo0 = prod0 >> sh, prod0 & lo32
        hi1, lo1 = prod1 >> sh, prod1 & lo32
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
        k0 = (k0 + W0) & lo32
        k1 = (k1 + W1) & lo32
    return tuple(w.astype(np.uint32) for w in (c0, c1, c2, c3))
