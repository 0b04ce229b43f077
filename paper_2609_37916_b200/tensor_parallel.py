"""Tensor-parallel sharding of the encoder's parameters (Section 3.4: column / row sharding with an
all-reduce inside the layer) and the all-reduce adapters rlx_encoder_forward_tp's callback needs.
Pure host logic: slicing and torch.distributed calls; the arithmetic of the layer runs in the library.

Per layer, rank r of n with H' = H/n, F' = F/n and d = H / num_heads:
  column-parallel   wqkv [3H', H] = rows {q heads of r | k heads of r | v heads of r} of Wqkv, bqkv likewise;
                    w1 [F', H] = rows r*F' .. of W1, b1 likewise.           (no exchange)
  row-parallel      wo [H, H'] = columns r*H' .. of Wo;  w2 [H, F'] = columns r*F' .. of W2;
                    their outputs are partial sums, all-reduced over the ranks.
  bo, b2            the full vector on rank 0, zeros elsewhere (added once to the sum).
  LayerNorm vectors and embedding tables are replicated.
"""
from __future__ import annotations

from typing import Dict, List, Sequence, Tuple

import numpy as np
import torch
import torch.distributed as dist


def check_tp(num_heads: int, hidden: int, ffn: int, world: int) -> None:
    if world < 1 or num_heads % world or ffn % world or (hidden // world) % 64 or (ffn // world) % 64:
        raise ValueError(f"tensor-parallel size {world} does not divide heads={num_heads}, H={hidden}, F={ffn} "
                         "into whole heads and 64-wide contraction blocks")


def shard_layer_tp(lw: Dict[str, np.ndarray], rank: int, world: int, num_heads: int) -> Dict[str, np.ndarray]:
    """One layer's parameter shard for `rank` (numpy in, numpy out; see the module header for the layout)."""
    H = lw["wo"].shape[0]
    F = lw["w1"].shape[0]
    check_tp(num_heads, H, F, world)
    Hl, Fl = H // world, F // world
    rows = np.concatenate([np.arange(part * H + rank * Hl, part * H + (rank + 1) * Hl) for part in range(3)])
    out = dict(lw)
    out["wqkv"] = np.ascontiguousarray(lw["wqkv"][rows])
    out["bqkv"] = np.ascontiguousarray(lw["bqkv"][rows])
    out["wo"] = np.ascontiguousarray(lw["wo"][:, rank * Hl:(rank + 1) * Hl])
    out["w1"] = np.ascontiguousarray(lw["w1"][rank * Fl:(rank + 1) * Fl])
    out["b1"] = np.ascontiguousarray(lw["b1"][rank * Fl:(rank + 1) * Fl])
    out["w2"] = np.ascontiguousarray(lw["w2"][:, rank * Fl:(rank + 1) * Fl])
    if rank != 0:
        out["bo"] = np.zeros_like(lw["bo"])
        out["b2"] = np.zeros_like(lw["b2"])
    return out


def shard_weights_tp(layers: Sequence[Dict[str, np.ndarray]], rank: int, world: int,
                     num_heads: int) -> List[Dict[str, np.ndarray]]:
    return [shard_layer_tp(lw, rank, world, num_heads) for lw in layers]


def allreduce_on_group(group=None):
    """All-reduce for a backend that reduces device tensors in place, stream-ordered (NCCL)."""
    def fn(view: torch.Tensor) -> None:
        dist.all_reduce(view, op=dist.ReduceOp.SUM, group=group)
    return fn


def allreduce_through_host(group=None):
    """All-reduce for a CPU backend (gloo): the partial sums take a round trip through host memory.
    For tests and for boxes without a device-side collective; synchronises the stream."""
    def fn(view: torch.Tensor) -> None:
        host = view.float().cpu()
        dist.all_reduce(host, op=dist.ReduceOp.SUM, group=group)
        view.copy_(host.to(torch.bfloat16))
    return fn
