"""Layer-level sharding across GPUs.

Layers of a model are independent quantization problems (each has its own H and W), so
N ranks simply take disjoint subsets of the layer list -- no collective is on the data path.
Only the timing / counting reductions below touch torch.distributed.
"""
from __future__ import annotations

from typing import List, Sequence

import torch
import torch.distributed as dist


def layer_cost(spec) -> float:
    """Rough relative cost of one layer: W-update products + factorisation + Hessian."""
    n, p = spec.d_in, spec.d_out
    return 12.0 * n * n * p * spec.T + 40.0 * float(n) ** 3 + 2.0 * spec.n_tokens * n * n


def shard_layers(layers: Sequence, rank: int, world: int) -> List:
    """Greedy longest-processing-time assignment; deterministic, identical on every rank."""
    order = sorted(range(len(layers)), key=lambda i: (-layer_cost(layers[i]), i))
    load = [0.0] * world
    owner = {}
    for i in order:
        r = min(range(world), key=lambda q: (load[q], q))
        owner[i] = r
        load[r] += layer_cost(layers[i])
    return [layers[i] for i in range(len(layers)) if owner[i] == rank]


def _reduce(value: float, op) -> float:
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=op)
    return float(t.item())


def max_over_ranks(value: float) -> float:
    return _reduce(value, dist.ReduceOp.MAX)


def sum_over_ranks(value: float) -> float:
    return _reduce(value, dist.ReduceOp.SUM)
