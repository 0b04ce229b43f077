"""Batch sharding for data-parallel inference: sequences are independent, so a batch splits across
ranks with no exchange step inside the forward.  The only communication is the optional gather of
the [B/G, H] embeddings afterwards.  Pure host logic (works with any torch.distributed backend)."""
from __future__ import annotations

from typing import List, Sequence

import torch
import torch.distributed as dist


def shard_indices(lengths: Sequence[int], world: int) -> List[List[int]]:
    """Partition sequence indices over `world` ranks balancing attention work (sum of length^2):
    sort by length descending and deal each sequence to the currently lightest rank.
    Deterministic; every index appears exactly once; shard sizes differ by at most one."""
    n = len(lengths)
    order = sorted(range(n), key=lambda i: (-int(lengths[i]), i))
    shards: List[List[int]] = [[] for _ in range(world)]
    load = [0] * world
    quota = [n // world + (1 if r < n % world else 0) for r in range(world)]
    for i in order:
        cands = [r for r in range(world) if len(shards[r]) < quota[r]]
        r = min(cands, key=lambda k: (load[k], k))
        shards[r].append(i)
        load[r] += int(lengths[i]) ** 2
    for s in shards:
        s.sort()
    return shards


def gather_embeddings(local: torch.Tensor, shards: List[List[int]], total: int) -> torch.Tensor:
    """All-gather the per-rank [len(shard), H] embeddings and scatter them back to batch order.
    Ranks with a shorter shard are padded to the longest one for the collective."""
    world = dist.get_world_size()
    cap = max(len(s) for s in shards)
    H = local.shape[1]
    padded = torch.zeros((cap, H), dtype=local.dtype, device=local.device)
    padded[: local.shape[0]] = local
    parts = [torch.empty_like(padded) for _ in range(world)]
    dist.all_gather(parts, padded)
    out = torch.zeros((total, H), dtype=local.dtype, device=local.device)
    for r, idx in enumerate(shards):
        if idx:
            out[torch.tensor(idx, device=local.device)] = parts[r][: len(idx)]
    return out
