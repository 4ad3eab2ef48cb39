"""Exchange step of Algorithm 1 (ExchangeGradients) for one process per GPU: worker w = rank w.

The paper exchanges the sparse messages with allGather when the workers kept different
coordinates and with allReduce when they kept the same ones (Methodology, third parameter).
Here the collectives are torch.distributed (NCCL over NVLink on GPUs); the received
messages land in this GPU's own memory, already in the W x k row layout the aggregate kernels
read, and the aggregate is enqueued on the caller's stream right behind the collective: torch
orders the two with a stream event, the host never waits in between.

    vals, idx  : this rank's message, k entries (from sc_compress / sc_compress_batch with W = 1)
    exchange_messages(...) -> (vals_all [W, k], idx rows) ready for sc_aggregate / sc_aggregate_shared

Modes for shared coordinates:
  "allgather"  every rank receives all W value rows and sums them in worker order with
               sc_aggregate_shared: bit-identical to the single-GPU result;
  "allreduce"  the paper's choice, k values per rank on the wire instead of W k: the sum is formed
               by the collective in an order the library does not control, so the result agrees
               with the ordered sum only to rounding (about 1e-7 relative).
"""
from __future__ import annotations

from typing import Optional, Tuple

import torch
import torch.distributed as dist


def exchange_messages(vals: torch.Tensor, idx: torch.Tensor, shared_coordinates: bool, mode: str = "allgather",
                      group: Optional[dist.ProcessGroup] = None) -> Tuple[torch.Tensor, torch.Tensor, int]:
    """Returns (values, coordinates, rows): `values` has `rows` rows of k entries in rank order
    (rows == world size, or 1 after an allreduce, where the row already holds the AVERAGE);
    `coordinates` has one row when the coordinates are shared, else one per rank."""
    if not dist.is_initialized():
        raise RuntimeError("torch.distributed is not initialised")
    world = dist.get_world_size(group)
    k = vals.numel()
    vals = vals.contiguous().view(k)
    idx = idx.contiguous().view(k)
    if shared_coordinates and mode == "allreduce":
        avg = vals.clone()
        if dist.get_backend(group) == "nccl":
            dist.all_reduce(avg, op=dist.ReduceOp.AVG, group=group)
        else:                                              # gloo has no AVG
            dist.all_reduce(avg, op=dist.ReduceOp.SUM, group=group)
            avg /= world
        return avg.view(1, k), idx.view(1, k), 1
    if mode not in ("allgather", "allreduce"):
        raise ValueError("mode must be 'allgather' or 'allreduce'")
    vals_all = torch.empty(world, k, dtype=vals.dtype, device=vals.device)
    dist.all_gather_into_tensor(vals_all.view(-1), vals, group=group)
    if shared_coordinates:
        return vals_all, idx.view(1, k), world
    idx_all = torch.empty(world, k, dtype=idx.dtype, device=idx.device)
    dist.all_gather_into_tensor(idx_all.view(-1), idx, group=group)
    return vals_all, idx_all, world


def exchange_and_aggregate(ctx, vals: torch.Tensor, idx: torch.Tensor, n: int, out: torch.Tensor,
                           shared_coordinates: bool, mode: str = "allgather",
                           group: Optional[dist.ProcessGroup] = None) -> None:
    """Algorithm 1, exchange + aggregate lines on one rank: out[n] <- average of all ranks' messages."""
    k = vals.numel()
    v, i, rows = exchange_messages(vals, idx, shared_coordinates, mode, group)
    if shared_coordinates:
        ctx.sc_aggregate_shared(rows, v, i.view(-1), k, n, out)
    else:
        ctx.sc_aggregate(rows, v, i, k, n, out)


def exchange_and_apply(ctx, vals: torch.Tensor, idx: torch.Tensor, n: int, x: torch.Tensor,
                       shared_coordinates: bool, mode: str = "allgather",
                       group: Optional[dist.ProcessGroup] = None) -> None:
    """Algorithm 1, exchange + aggregate + model-update lines on one rank: x[n] <- x - average of all ranks'
    messages, touching only the coordinates some rank sent (no dense vector is formed)."""
    k = vals.numel()
    v, i, rows = exchange_messages(vals, idx, shared_coordinates, mode, group)
    ctx.sc_aggregate_apply(rows, v, i.view(-1), k, n, x, shared=shared_coordinates)
