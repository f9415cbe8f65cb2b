"""Partition of a matrix across ranks for the mask search: contiguous strips of M-row multiples.

Blocks are independent (Eq. 1 is stated per M x M block), so a strip needs no halo and no exchange;
mask and masked-weight outputs of different strips are disjoint and only the scalar objective is summed."""
from __future__ import annotations


def row_strip(rows: int, M: int, world_size: int, rank: int):
    """[r0, r1) of the rows owned by `rank`: block rows are dealt out as evenly as possible, in order."""
    if rows % M or world_size < 1 or not 0 <= rank < world_size:
        raise ValueError("rows must be a multiple of M and 0 <= rank < world_size")
    brows = rows // M
    base, extra = divmod(brows, world_size)
    b0 = rank * base + min(rank, extra)
    b1 = b0 + base + (1 if rank < extra else 0)
    return b0 * M, b1 * M
