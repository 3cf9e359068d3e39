"""Batch sharding for runs on several GPUs.

Pixels are coded independently (1 x 1 x C blocks, Section 3.1) and the model and codebook are
read-only, so the batch dimension shards with no exchange on the encode / decode path: every
rank codes its own maps into its own stream.  The only collective is the bookkeeping below --
a max over ranks of the device time and a sum of the bytes processed -- which runs on whatever
backend the process group has (NCCL on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

import torch


def shard_range(total: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous, balanced split of `total` maps: returns (first, count) for `rank`."""
    if world < 1 or not (0 <= rank < world):
        raise ValueError("bad rank / world size")
    base, extra = divmod(total, world)
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)


def aggregate(local_bytes: float, local_ms: float, device: str | torch.device = "cpu") -> tuple[float, float]:
    """Whole-job (bytes, milliseconds): bytes summed over ranks, time as the max over ranks.
    Without an initialised process group the local values are returned."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(local_bytes), float(local_ms)
    t = torch.tensor([float(local_ms)], dtype=torch.float64, device=device)
    b = torch.tensor([float(local_bytes)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(b, op=dist.ReduceOp.SUM)
    return float(b.item()), float(t.item())
