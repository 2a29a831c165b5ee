"""Sharding of the layer solver across GPUs, one process per GPU.

Two levels, neither of which puts a collective inside the ADMM loop:

* across layers -- the layers of a model are independent quantization problems (each has its own H and
  W), so N ranks take disjoint subsets of the layer list (`shard_layers`); only timing and counting
  reductions touch torch.distributed;
* inside a layer (`solve_layer_sharded`) -- H = X^T X is a sum over calibration rows (Sec. 3.1), so every
  rank accumulates the rows of its token shard and ONE all-reduce(sum) of the n x n fp32 accumulator gives
  every rank the whole Hessian; each rank then factorises it (replicated work) and runs the ADMM loop and
  the local search on its own slice of OUTPUT channels, which are independent problems given H (the
  projection of Sec. 3.3 and the local search of Sec. 3.5 act per channel).  The residual norms of
  Theorem 1 are combined from the shards' sums of squares after the loop.

The collectives run on caller-owned torch tensors through torch.distributed (NCCL on GPUs, gloo in the
CPU tests); no kernel of the library is handed another GPU's memory.
"""
from __future__ import annotations

import math
from typing import Callable, List, Sequence, Tuple

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


def _world() -> int:
    return dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1


def _reduce(value: float, op) -> float:
    if _world() == 1:
        return float(value)
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=op)
    return float(t.item())


def max_over_ranks(value: float) -> float:
    return _reduce(value, dist.ReduceOp.MAX)


def sum_over_ranks(value: float) -> float:
    return _reduce(value, dist.ReduceOp.SUM)


# ---------------------------------------------------------------------------------------------------
# inside one layer
# ---------------------------------------------------------------------------------------------------
def token_shard(n_chunks: int, rank: int, world: int) -> range:
    """Contiguous range of calibration chunks of this rank; the ranges of all ranks tile [0, n_chunks)."""
    lo = (n_chunks * rank) // world
    hi = (n_chunks * (rank + 1)) // world
    return range(lo, hi)


def channel_shard(d_out: int, rank: int, world: int, align: int = 128) -> Tuple[int, int]:
    """[j0, j1) of this rank's output channels.  Boundaries fall on multiples of `align` (one row tile of the
    product kernel) while every rank still gets channels; the slices of all ranks tile [0, d_out)."""
    units = d_out // align
    if units < world:                         # fewer tiles than ranks: split channel by channel
        align, units = 1, d_out
    j0 = (units * rank) // world * align
    j1 = (units * (rank + 1)) // world * align if rank + 1 < world else d_out
    return j0, j1


def allreduce_hessian(H_raw: torch.Tensor, n_tokens: int) -> int:
    """Sum of the ranks' accumulators, in place, and of their row counts (returned)."""
    if _world() > 1:
        dist.all_reduce(H_raw, op=dist.ReduceOp.SUM)
    return int(round(sum_over_ranks(float(n_tokens))))


def combine_residuals(resid_local: torch.Tensor) -> torch.Tensor:
    """[T, 2] residual norms of the whole layer from the norms over each rank's channels: Frobenius norms
    add in squares."""
    sq = resid_local.double() ** 2
    if _world() > 1:
        dist.all_reduce(sq, op=dist.ReduceOp.SUM)
    return sq.sqrt()


def gather_channels(local: torch.Tensor, d_out: int) -> torch.Tensor:
    """Concatenates the ranks' channel slices (dim 0) in rank order; every rank gets the whole array."""
    world = _world()
    if world == 1:
        return local
    rank = dist.get_rank()
    sizes = [channel_shard(d_out, r, world) for r in range(world)]
    width = max(j1 - j0 for j0, j1 in sizes)
    pad = torch.zeros((width,) + tuple(local.shape[1:]), dtype=local.dtype, device=local.device)
    pad[: local.shape[0]] = local
    parts = [torch.empty_like(pad) for _ in range(world)]
    dist.all_gather(parts, pad)
    assert sizes[rank][1] - sizes[rank][0] == local.shape[0]
    return torch.cat([parts[r][: sizes[r][1] - sizes[r][0]] for r in range(world)], dim=0)


def solve_layer_sharded(sol, spec, W: torch.Tensor, chunk: Callable[[int], torch.Tensor], resid=None,
                        local_search: bool = True):
    """One layer on all ranks: token-sharded Hessian, one all-reduce, replicated factorisation, channel-sharded
    ADMM loop and local search.

    sol: a solver with the methods of binding.Solver; spec: the layer (n_chunks, rho(), bits, group_size,
    symmetric); W: the whole [d_out, d_in] weight on this rank's device; chunk(c): calibration chunk c.
    Returns (codes, scale, zero, info) for THIS rank's channels [info['j0'], info['j1']); use
    gather_channels for the whole layer."""
    world = _world()
    rank = dist.get_rank() if world > 1 else 0
    sol.hessian_reset()
    for c in token_shard(spec.n_chunks, rank, world):
        sol.hessian_accumulate(chunk(c))
    if world > 1:
        H_raw, ntok = sol.hessian_export()
        total = allreduce_hessian(H_raw, ntok)
        sol.hessian_import(H_raw, total)
    sol.factor(rho=spec.rho())
    j0, j1 = channel_shard(spec.d_out, rank, world)
    Wj = W[j0:j1].contiguous()
    codes, scale, zero, rep = sol.quantize_layer(Wj, spec.bits, spec.group_size, spec.symmetric, resid=resid,
                                                 report=not local_search)
    info = dict(j0=j0, j1=j1, rep=rep, rep_ls=None)
    if local_search:
        info["rep_ls"], info["status"] = sol.local_search(Wj, spec.bits, spec.group_size, codes, scale, zero)
    if resid is not None:
        info["resid"] = combine_residuals(resid)
    return codes, scale, zero, info


def layer_error(info) -> float:
    """Tr(E^T H E) of the whole layer: the shards' errors add (one term per output channel)."""
    rep = info["rep_ls"] if info.get("rep_ls") is not None else info["rep"]
    local = rep.err_after if info.get("rep_ls") is not None else rep.err_before
    return sum_over_ranks(local)


def balance(costs: Sequence[float]) -> float:
    """max / mean of per-rank costs (1.0 = perfectly balanced)."""
    m = sum(costs) / len(costs)
    return max(costs) / m if m > 0 else math.nan
