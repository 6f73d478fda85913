"""Host-side helpers for running the solver on several GPUs (one process per GPU).

The path shards without any exchange: layers -- and whole Transformer blocks -- are independent
units once their inputs exist, so every rank solves its own units and only timing is reduced.
"""
from __future__ import annotations

from typing import List, Sequence

import torch
import torch.distributed as dist

from .synth import workloads as WL


def rank_layers(layers: Sequence[WL.Layer], rank: int) -> List[WL.Layer]:
    """Weak scaling: rank r solves its own copy of the layer set, seeded as Transformer block (block_idx + r)."""
    return [WL.Layer(l.config_id, l.block_idx + rank, l.kind, l.R, l.C, l.n_tokens) for l in layers]


def shard_units(n_units: int, world: int, rank: int) -> range:
    """Strong scaling: contiguous, balanced share of n_units independent units (layers or row stripes)."""
    base, extra = divmod(n_units, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def max_over_ranks(value: float, device=None) -> float:
    """Slowest rank's time (the job's time); a no-op outside a process group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device=None) -> float:
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
