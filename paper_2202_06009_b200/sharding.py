"""Scale-out across GPUs: contiguous chunk ranges.

Every operation of the method is elementwise or confined to one chunk (the l1
norm and the sign packing), and the only global quantities are host scalars
(learning rate, sum of learning rates, step index, policy bits).  A flat
parameter vector can therefore be cut at chunk boundaries and each piece given
to its own handle on its own GPU: no data ever crosses between the pieces.
"""
from typing import Tuple


def chunk_range(n_chunks: int, world: int, rank: int) -> Tuple[int, int]:
    """[first, last) chunk indices of `rank`: sizes differ by at most one chunk."""
    if not (0 <= rank < world):
        raise ValueError("rank outside the world")
    base, extra = divmod(n_chunks, world)
    first = rank * base + min(rank, extra)
    return first, first + base + (1 if rank < extra else 0)


def param_range(n_params: int, chunk: int, world: int, rank: int) -> Tuple[int, int]:
    """[first, last) parameter indices of `rank`; the ragged last chunk goes to the last non-empty rank."""
    n_chunks = -(-n_params // chunk)
    c0, c1 = chunk_range(n_chunks, world, rank)
    return min(c0 * chunk, n_params), min(c1 * chunk, n_params)
