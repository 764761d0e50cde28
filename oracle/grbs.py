"""Globally-randomized blockwise sparsifier (GRBS), Definition 2 (oracle side).

Test infrastructure only.  The flat vector of d elements is cut into
B = ceil(d / block_size) contiguous blocks (the last one may be short).  Every
worker derives the same selection from a shared seed, so the mask is a function
of (seed, step t, which compressor, block b) alone.  Reading taken where the
paper gives no sampling procedure: each block is selected independently with
probability 1/R, which makes C(v) = v * mask a 1/R-approximate compressor in
expectation exactly as Definition 2 states.

Draw: word 0 of Philox4x32-10 with key = (seed low 32 bits, seed high 32 bits)
and counter = (b, t low 32 bits, t high 32 bits, stream), stream 0 for the
per-step compressor of the update, 1 for the error-reset compressor.  Block b
is selected iff  word0 * R < 2**32  (R = 1 selects everything).  R = 0 stands for the
compressor C = 0 that keeps nothing (delta = 0, allowed by Definition 1 as extended in
Section 3): the special cases CSER-PL and CSEA of Appendix A.1.
"""
import numpy as np
from .philox import philox4x32_10

STREAM_GRAD = 0    # compressor applied to the update p every step (Algorithm 2 line 6)
STREAM_RESET = 1   # compressor applied to the error e every H steps (Algorithm 2 line 11)


def n_blocks(d, block_size):
    return (int(d) + int(block_size) - 1) // int(block_size)


def grbs_mask(seed, t, stream, B, R, block_begin=0):
    """uint8[B] selection flags of blocks block_begin .. block_begin+B-1 at step t."""
    if int(R) == 0:
        return np.zeros(B, np.uint8)
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    t = int(t) & 0xFFFFFFFFFFFFFFFF
    b = np.arange(block_begin, block_begin + B, dtype=np.uint64)
    word0 = philox4x32_10(seed & 0xFFFFFFFF, seed >> 32,
                          b, t & 0xFFFFFFFF, t >> 32, int(stream))[0]
    return (word0.astype(np.uint64) * np.uint64(R) < np.uint64(1 << 32)).astype(np.uint8)


def exact_count(B, R):
    """k of the exact-count reading of Definition 2: round(B / R), halves up; R = 0 gives 0."""
    if int(R) == 0:
        return 0
    return min(int(B), (2 * int(B) + int(R)) // (2 * int(R)))


def grbs_mask_exact(seed, t, stream, B, R):
    """Definition 2 read literally: exactly k = round(B / R) of the B blocks, the k with the
    smallest keys (word0, block id), word0 being the draw `grbs_mask` thresholds."""
    k = exact_count(B, R)
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    t = int(t) & 0xFFFFFFFFFFFFFFFF
    b = np.arange(B, dtype=np.uint64)
    word0 = philox4x32_10(seed & 0xFFFFFFFF, seed >> 32, b, t & 0xFFFFFFFF, t >> 32, int(stream))[0]
    order = np.lexsort((b, word0))                 # by word0, ties by block id
    mask = np.zeros(B, np.uint8)
    mask[order[:k]] = 1
    return mask
