"""Sharding of a region-level verification batch across replicas (host code only).

Stage 1 of the method verifies every region's draft independently (paper Eq. 2), so a batch splits across
GPUs by sequence with no exchange inside the step: every replica holds the full weights and the KV blocks of
its own regions, runs the same verify call on its share, and only the small integer results (accepted length
and emitted tokens per region) travel back, through the host.  The page-level stage (Eq. 4) is one sequence
and does not shard: replicas then work on different pages.

The partition balances a cost model of one verify step per region:
    rows * ROW_COST + pairs * PAIR_COST
where rows = draft length + 1 (the GEMM work grows with the rows) and pairs = attended (query, key) pairs
(the attention work).  The weight stream is the same on every replica and does not enter the balance.
"""
from __future__ import annotations

from typing import Dict, List, Sequence

# FLOP per query row through the projections / per attended pair, 24-layer decoder (ratio is what matters)
ROW_COST = 0.822e9
PAIR_COST = 98_304.0


def region_cost(context_len: int, draft_len: int) -> float:
    rows = int(draft_len) + 1
    pairs = rows * int(context_len) + rows * (rows + 1) // 2
    return rows * ROW_COST + pairs * PAIR_COST


def partition(context_lens: Sequence[int], draft_lens: Sequence[int], world: int) -> List[List[int]]:
    """Longest-processing-time greedy: regions by decreasing cost, each to the least-loaded replica (ties to
    the lowest rank).  Returns, per rank, the region indices it owns in increasing order.  Deterministic, so
    every rank computes the same partition without talking to the others."""
    if world <= 0:
        raise ValueError("world must be positive")
    if len(context_lens) != len(draft_lens):
        raise ValueError("context_lens and draft_lens differ in length")
    costs = [region_cost(L, k) for L, k in zip(context_lens, draft_lens)]
    order = sorted(range(len(costs)), key=lambda i: (-costs[i], i))
    load = [0.0] * world
    owned: List[List[int]] = [[] for _ in range(world)]
    for i in order:
        r = min(range(world), key=lambda j: (load[j], j))
        owned[r].append(i)
        load[r] += costs[i]
    return [sorted(o) for o in owned]


def imbalance(context_lens: Sequence[int], draft_lens: Sequence[int], owned: Sequence[Sequence[int]]) -> float:
    """max over ranks of the modelled cost divided by the mean (1.0 = perfectly balanced)."""
    loads = [sum(region_cost(context_lens[i], draft_lens[i]) for i in o) for o in owned]
    mean = sum(loads) / max(1, len(loads))
    return max(loads) / mean if mean > 0 else 1.0


def merge_results(per_rank: Sequence[Dict[int, object]], n_regions: int) -> List[object]:
    """Results keyed by region index from every rank -> one list in region order.  Every region must be
    reported exactly once."""
    out: List[object] = [None] * n_regions
    seen = [False] * n_regions
    for d in per_rank:
        for i, v in d.items():
            if not (0 <= i < n_regions) or seen[i]:
                raise ValueError(f"region {i} reported twice or out of range")
            out[i], seen[i] = v, True
    if not all(seen):
        raise ValueError(f"regions missing from the gathered results: {[i for i, s in enumerate(seen) if not s]}")
    return out


def gather_results(local: Dict[int, object], n_regions: int) -> List[object]:
    """Host-side gather over the default process group (any backend): every rank gets the merged list."""
    import torch.distributed as dist
    if not dist.is_initialized() or dist.get_world_size() == 1:
        return merge_results([local], n_regions)
    bucket: List[object] = [None] * dist.get_world_size()
    dist.all_gather_object(bucket, local)
    return merge_results(bucket, n_regions)
