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


def shard_heads(num_q_heads: int, num_kv_heads: int, rank: int, world_size: int) -> Tuple[int, int, int, int]:
    """Head sharding inside a sequence (tensor-parallel caches): rank r holds KV heads
    [kv_begin, kv_end) and the query heads that read them, [q_begin, q_end) (query head h reads KV
    head h // (num_q_heads // num_kv_heads)). Every rank gets the same number of heads, which is what
    lets the ranks' local score means simply be added (see make_scores_exchange)."""
    if world_size <= 0 or not (0 <= rank < world_size) or num_kv_heads <= 0 or num_q_heads % num_kv_heads != 0:
        raise ValueError("bad sharding arguments")
    if num_kv_heads % world_size != 0:
        raise ValueError("the KV heads must divide evenly over the ranks")
    group = num_q_heads // num_kv_heads
    per = num_kv_heads // world_size
    return rank * per * group, (rank + 1) * per * group, rank * per, (rank + 1) * per


def make_scores_exchange(group=None):
    """The one exchange of a head-sharded decode step (Section 3.1.1: the focal score is the attention
    weight averaged over all heads): returns the callable for fastocr_decode_step's `scores_exchange`,
    an in-place all-reduce (sum) of the ranks' local score means over `group` (default: the world).
    The sum of the local means is world_size times the global mean: the same ranking, hence the same
    selection, and identical on every rank because every rank receives the same reduced values. With
    the NCCL backend the collective is enqueued behind the kernels already on the current stream."""
    import torch.distributed as dist

    def exchange(scores, layer):
        dist.all_reduce(scores, op=dist.ReduceOp.SUM, group=group)

    return exchange


def mean_ratio_over_ranks(ratio, group=None):
    """Warm-up with sharded heads: Eq. 1's image-attention ratio is a mean over heads, so the ranks'
    records [L][B] (equal head counts) are averaged in place before Focal Layer Selection."""
    import torch.distributed as dist

    dist.all_reduce(ratio, op=dist.ReduceOp.SUM, group=group)
    ratio /= dist.get_world_size(group)
    return ratio
