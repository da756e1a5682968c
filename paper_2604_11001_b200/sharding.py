"""Replica sharding across ranks.

Replicas are independent (every draw is keyed by the replica's generator id), so several GPUs need no
data-path exchange: each rank simulates its own replicas and the per-group totals are plain int64 sums.
``shard_for_rank`` gives rank r the same groups with generator ids shifted by r x (span of ids in use),
so that the union over ranks is one larger simulation with distinct replicas (weak scaling).
``combine_group_totals`` adds per-group counter rows across ranks with torch.distributed (any backend).
"""
from __future__ import annotations

from dataclasses import replace

import torch

MAX_FIELDS = (0, 16, 18, 20)   # steps_done, max_lat, max_U, max_Q combine by maximum
OR_FIELDS = (1,)               # status combines by bitwise or


def id_span(cfg) -> int:
    return max(g.rng_replica_base + g.n_replicas for g in cfg.groups)


def shard_for_rank(cfg, rank: int):
    span = id_span(cfg)
    if (rank + 1) * span > 2 ** 32:
        raise ValueError("generator replica ids exceed 32 bits")
    groups = tuple(replace(g, rng_replica_base=g.rng_replica_base + rank * span) for g in cfg.groups)
    return cfg.with_(groups=groups)


def combine_group_totals(totals, dist=None):
    """totals: int64 tensor [n_groups, 28] of this rank.  Returns the combination over all ranks."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return totals
    out = totals.clone()
    dist.all_reduce(out, op=dist.ReduceOp.SUM)
    for f in MAX_FIELDS:
        col = totals[:, f].clone()
        dist.all_reduce(col, op=dist.ReduceOp.MAX)
        out[:, f] = col
    for f in OR_FIELDS:
        # bitwise or as a maximum per bit (status has two bits): every backend implements MAX, NCCL has no BOR
        bits = ((totals[:, f].unsqueeze(1) >> torch.arange(8, device=totals.device)) & 1).contiguous()
        dist.all_reduce(bits, op=dist.ReduceOp.MAX)
        out[:, f] = (bits << torch.arange(8, device=totals.device)).sum(dim=1)
    return out
