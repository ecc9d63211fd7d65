"""Head-sharded multi-GPU layout: which KV groups of one layer a rank owns.

Algorithm 1 of the paper is defined per head, and with grouped-query attention a KV head is shared by
the G query heads of its group, so the unit that can move to another GPU without any exchange inside
the path is a KV group (K, V of one KV head and the Q, O of its G query heads).  Rank r of N owns the
groups r, r + N, r + 2N, ...; it runs the unchanged C-ABI calls on its slice (H_kv' = groups owned,
H_q' = G * H_kv'), and the results are the single-GPU results of those heads bit for bit.  No
collective is needed in the data path; only the timing of a benchmark is reduced over ranks.
"""
from __future__ import annotations

from typing import List


def kv_groups_of_rank(n_kv_heads: int, rank: int, world: int) -> List[int]:
    """KV heads owned by `rank` (round robin).  Every KV head belongs to exactly one rank."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError(f"rank {rank} of {world}")
    if n_kv_heads < world:
        raise ValueError(f"{n_kv_heads} KV groups cannot be spread over {world} ranks")
    return list(range(rank, n_kv_heads, world))


def q_heads_of_groups(groups: List[int], group_size: int) -> List[int]:
    """Query heads of the given KV groups, in the order the rank's slice stores them."""
    return [g * group_size + i for g in groups for i in range(group_size)]
