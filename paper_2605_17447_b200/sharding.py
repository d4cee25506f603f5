"""Sequence sharding for more than one GPU. Every sequence's caches, scores, selection and carried
fixation set are independent of every other sequence's, so ranks take disjoint contiguous slices of
the batch and exchange nothing on the data path."""
from __future__ import annotations

from typing import Tuple


def shard_sequences(num_sequences: int, rank: int, world_size: int) -> Tuple[int, int]:
    """[begin, end) of the sequences owned by `rank`; slices differ in size by at most one."""
    if world_size <= 0 or not (0 <= rank < world_size) or num_sequences < 0:
        raise ValueError("bad sharding arguments")
    base, extra = divmod(num_sequences, world_size)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)
