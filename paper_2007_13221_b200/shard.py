"""Column-slab partition of the flat parameter vector across GPUs (host logic).

Given the masks, every column of the CSER step is independent of every other
column, and the GRBS masks depend only on (seed, step, global block id).  A GPU
that owns a slab of whole blocks, and draws its masks with the global ids of
those blocks, therefore computes exactly what a single GPU would compute for
those columns, with no exchange of data (Section 3.3: every worker picks the
same blocks from the synchronized seed).
"""


def slab_of_rank(d, block_size, rank, world_size):
    """(col_begin, col_end, block_begin) of `rank`'s slab: whole blocks, as even as possible."""
    B = (d + block_size - 1) // block_size
    base, extra = divmod(B, world_size)
    b0 = rank * base + min(rank, extra)
    b1 = b0 + base + (1 if rank < extra else 0)
    return min(b0 * block_size, d), min(b1 * block_size, d), b0


def workers_of_rank(n_total, rank, world_size):
    """(first, count) of the workers `rank` holds in the worker-sharded deployment."""
    base, extra = divmod(n_total, world_size)
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)
