"""Host-side helpers for running the solver on several GPUs of one node.

The method treats every layer independently (Sec. 3.2), so the multi-GPU scheme is a plain
partition of the layers: each rank prunes its own contiguous slice with the single-GPU path and
no data-path collective is needed.  ``torch.distributed`` is only used to agree on timings and,
if wanted, to gather the small per-layer results (removal orders, losses) on one rank.

The one stage with a real exchange is an optional token-sharded calibration pass: H = 2 X X^T is
a sum over tokens, so ranks that hold different calibration tokens accumulate partial Hessians
with the single-GPU kernel and add them with one all-reduce per layer family (``token_shard``,
``allreduce_hessian``).
"""
from __future__ import annotations

from typing import Any, List, Tuple


def partition_layers(n_layers: int, world_size: int, rank: int) -> Tuple[int, int]:
    """[begin, end) of the layers owned by ``rank``: contiguous, sizes differ by at most one."""
    if world_size < 1 or not 0 <= rank < world_size or n_layers < 0:
        raise ValueError("need 0 <= rank < world_size and n_layers >= 0")
    return n_layers * rank // world_size, n_layers * (rank + 1) // world_size


def max_over_ranks(value: float, group=None) -> float:
    """Maximum of a host float over all ranks (1-rank runs return the value itself)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return float(value)
    dev = "cuda" if dist.get_backend(group) == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t[0])


def gather_layer_results(local: List[Any], n_layers: int, group=None) -> List[Any]:
    """All ranks' per-layer results (picklable objects, one per owned layer) in layer order.

    Every rank passes the list for the slice ``partition_layers`` gave it and receives the full
    list of ``n_layers`` entries.
    """
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        if len(local) != n_layers:
            raise ValueError("single-rank run must hold every layer")
        return list(local)
    world = dist.get_world_size(group)
    parts: List[Any] = [None] * world
    dist.all_gather_object(parts, list(local), group=group)
    out: List[Any] = []
    for r, part in enumerate(parts):
        b, e = partition_layers(n_layers, world, r)
        if len(part) != e - b:
            raise ValueError(f"rank {r} returned {len(part)} results for {e - b} layers")
        out.extend(part)
    return out


def token_shard(n_tokens: int, world_size: int, rank: int, multiple: int = 1) -> Tuple[int, int]:
    """[begin, end) of the calibration tokens that ``rank`` accumulates: contiguous, every boundary
    but the last a multiple of ``multiple`` (e.g. the sequence length, so that no sequence is
    cut), sizes as even as that allows."""
    if world_size < 1 or not 0 <= rank < world_size or n_tokens < 0 or multiple < 1:
        raise ValueError("need 0 <= rank < world_size, n_tokens >= 0, multiple >= 1")
    units = (n_tokens + multiple - 1) // multiple
    b = min(n_tokens, units * rank // world_size * multiple)
    e = min(n_tokens, units * (rank + 1) // world_size * multiple)
    return b, e


def allreduce_hessian(H, group=None):
    """Sum the ranks' partial Hessians in place (H = sum over ranks of 2 X_r X_r^T) and return H.

    H is a torch tensor [L, d, d] on the device of the process group's backend (CUDA for nccl,
    CPU for gloo).  fp32 sums of a handful of partial results; the order of the additions is
    the collective's, so ranks agree bit for bit with each other but not necessarily with a
    one-rank pass over all tokens."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return H
    dist.all_reduce(H, op=dist.ReduceOp.SUM, group=group)
    return H
