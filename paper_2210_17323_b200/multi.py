"""Host-side helpers for running the solver on several GPUs (one process per GPU).

The path shards without any exchange: layers -- and whole Transformer blocks -- are independent
units once their inputs exist, so every rank solves its own units and only timing is reduced.

One layer can also be split over ranks (strong scaling): the Hessian is a sum over calibration
tokens (Section 2: H = 2 X X^T), so each rank accumulates its token shard and ONE all-reduce of H
(a plain sum of local buffers) gives every rank the full matrix; the factor U is then computed
redundantly on every rank (it is needed everywhere and costs less than shipping it); the rows of W
are independent sub-problems given U (Section 2), so each rank quantizes its row stripe and the
outputs are disjoint row ranges.  The only exchange step is that all-reduce.
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


def all_reduce_sum_(t: torch.Tensor) -> torch.Tensor:
    """In-place sum of a local buffer over all ranks (NCCL for CUDA tensors, gloo for CPU tensors)."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return t


def token_shard(n_tokens: int, world: int, rank: int) -> range:
    """This rank's share of the calibration tokens (contiguous, balanced)."""
    return shard_units(n_tokens, world, rank)


def solve_layer_sharded(n_tokens, R, world, rank, hessian_of_tokens, factor_of, quantize_rows):
    """One layer over `world` ranks.  hessian_of_tokens(token_range) -> this rank's partial H (a tensor that supports
    all_reduce_sum_), factor_of(H) -> U, quantize_rows(row_range, U) -> that stripe's outputs.
    Returns (row_range, outputs, H, U)."""
    H = hessian_of_tokens(token_shard(n_tokens, world, rank))
    all_reduce_sum_(H)
    U = factor_of(H)
    rows = shard_units(R, world, rank)
    return rows, quantize_rows(rows, U), H, U
