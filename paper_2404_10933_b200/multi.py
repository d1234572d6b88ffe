"""Host-side plumbing for running independent configuration shards on several GPUs.

The method has no exchange step: every configuration (and every search and selection)
is independent, so ranks never trade event data.  What exists is (1) splitting one grid
into contiguous, cost-balanced shards, (2) concatenating per-rank result slices, and
(3) reducing scalar timings over ranks.  All of it goes through ``torch.distributed``
(NCCL on GPUs, gloo on CPU for tests).
"""
from __future__ import annotations

import os

import numpy as np

from . import grids


def env_rank_world() -> tuple[int, int, int]:
    """(rank, world_size, local_rank) from the torchrun environment."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def shard_of(n_items: int, weights, rank: int, world: int) -> tuple[int, int]:
    """Contiguous [lo, hi) of this rank, balanced by per-item cost (e.g. event counts)."""
    if weights is None:
        weights = np.ones(n_items)
    b = grids.shard_bounds(np.asarray(weights), world)
    return int(b[rank]), int(b[rank + 1])


def reduce_scalar(x: float, op: str, device="cpu") -> float:
    """max / sum of a host scalar over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op={"max": dist.ReduceOp.MAX, "sum": dist.ReduceOp.SUM}[op])
    return float(t.item())


def gather_slices(local, total_len: int, lo: int, device="cpu"):
    """Every rank contributes ``local`` = result[lo : lo + len(local)]; returns the full
    result tensor on every rank.  Slices may differ in length."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return local
    world = dist.get_world_size()
    meta = torch.tensor([lo, local.shape[0]], dtype=torch.int64, device=device)
    metas = [torch.empty_like(meta) for _ in range(world)]
    dist.all_gather(metas, meta)
    longest = max(int(m[1]) for m in metas)
    padded = torch.zeros((longest,) + tuple(local.shape[1:]), dtype=local.dtype, device=device)
    padded[:local.shape[0]] = local
    parts = [torch.empty_like(padded) for _ in range(world)]
    dist.all_gather(parts, padded)
    out = torch.zeros((total_len,) + tuple(local.shape[1:]), dtype=local.dtype, device=device)
    for m, p in zip(metas, parts):
        out[int(m[0]):int(m[0]) + int(m[1])] = p[:int(m[1])]
    return out
