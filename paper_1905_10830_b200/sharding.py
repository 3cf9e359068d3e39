"""Batch sharding for runs on several GPUs.

Pixels are coded independently (1 x 1 x C blocks, Section 3.1) and the model and codebook are
read-only, so the batch dimension shards with no exchange on the encode / decode path: every
rank codes its own maps into its own stream.  The collectives are the bookkeeping below -- a
max over ranks of the device time and a sum of the bytes processed -- and, for a fit whose
calibration maps are spread over the ranks, one sum of the running fit state (count, sum of
pixel vectors, sum of outer products: Section 3.1, the covariance can be updated online).
They run on whatever backend the process group has (NCCL on GPUs, gloo in the CPU tests)."""
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


def merge_fit_state(count: int, vec_sum, outer_sum, device: str | torch.device = "cpu"):
    """Sum of the running fit state over all ranks: every rank passes the (count, sum[C],
    outer[C][C]) it exported from its own calibration maps and gets back the state of all maps,
    ready to be imported and finished on any rank.  One all-reduce of C*C + C + 1 doubles.
    Without an initialised process group the local state is returned."""
    import torch.distributed as dist
    s1 = torch.as_tensor(vec_sum, dtype=torch.float64).reshape(-1)
    s2 = torch.as_tensor(outer_sum, dtype=torch.float64)
    c = s1.numel()
    if s2.shape != (c, c):
        raise ValueError("outer-product sum must be C x C")
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return int(count), s1.numpy().copy(), s2.numpy().copy()
    # the count travels as a double: exact up to 2^53 samples
    flat = torch.cat([torch.tensor([float(count)], dtype=torch.float64), s1, s2.reshape(-1)]).to(device)
    dist.all_reduce(flat, op=dist.ReduceOp.SUM)
    flat = flat.cpu()
    return int(round(flat[0].item())), flat[1:1 + c].numpy().copy(), flat[1 + c:].reshape(c, c).numpy().copy()
