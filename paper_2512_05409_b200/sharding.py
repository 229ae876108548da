"""Token sharding for more than one GPU.

Every call of the path works on token rows independently (per-token scales, per-token banks),
so M is split across ranks with the weights replicated and NO data-path collective: each rank
encodes and multiplies its own rows.  Only a consumer that wants the full [M, N] output on
one rank needs a gather.
"""
from __future__ import annotations


def row_shard(M: int, world_size: int, rank: int) -> tuple[int, int]:
    """Half-open row range [start, stop) of `rank`; sizes differ by at most one row."""
    if world_size < 1 or not (0 <= rank < world_size) or M < 0:
        raise ValueError("bad shard request")
    base, rem = divmod(M, world_size)
    start = rank * base + min(rank, rem)
    return start, start + base + (1 if rank < rem else 0)
