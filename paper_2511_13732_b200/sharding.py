"""Batch sharding across ranks (one process per GPU).

Sequences are verified independently of one another, so the batch dimension
shards with no exchange on the data path: every rank runs the same kernels on
its own sequences and the outputs are disjoint slices.  The only collective is
the max-over-ranks of the measured time (and, if a caller wants one place to
hold all outputs, a gather of a few integers per sequence).
"""
from __future__ import annotations

from typing import List, Optional


def rank_sequences(B: int, rank: int, world: int, weak: bool = True) -> List[int]:
    """Global sequence indices handled by `rank`.

    weak=True : every rank gets B sequences of its own (rank*B .. rank*B+B-1); total work grows with `world`.
    weak=False: the B sequences are split into `world` contiguous, near-equal shards (first ones one longer).
    """
    if not (0 <= rank < world) or B < 0:
        raise ValueError("need 0 <= rank < world and B >= 0")
    if weak:
        return list(range(rank * B, rank * B + B))
    base, extra = divmod(B, world)
    start = rank * base + min(rank, extra)
    return list(range(start, start + base + (1 if rank < extra else 0)))


def max_over_ranks(value: float, dist=None) -> float:
    """Maximum of a per-rank number over the process group (identity without one)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch

    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def gather_outputs(local, dist=None) -> Optional[list]:
    """Gather per-rank integer outputs (a tensor [B_local, ...]) on every rank, in rank order."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return [local]
    import torch

    sizes = [torch.zeros(1, dtype=torch.int64, device=local.device) for _ in range(dist.get_world_size())]
    dist.all_gather(sizes, torch.tensor([local.shape[0]], dtype=torch.int64, device=local.device))
    nmax = int(max(s.item() for s in sizes))
    pad = torch.full((nmax,) + tuple(local.shape[1:]), -1, dtype=local.dtype, device=local.device)
    pad[: local.shape[0]] = local
    bufs = [torch.empty_like(pad) for _ in sizes]
    dist.all_gather(bufs, pad)
    return [b[: int(s.item())] for b, s in zip(bufs, sizes)]
