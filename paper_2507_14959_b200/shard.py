"""Multi-GPU plumbing of the forward path: frames are independent units, so a job over N GPUs is a
contiguous split of the frame list with the weights replicated and no collective inside the
forward.  The only exchanges are a barrier, the max-over-ranks of device timings, and (optionally)
gathering the per-frame score rows for a single consumer.

Works with any torch.distributed backend (nccl on GPUs, gloo on CPU).
"""
from __future__ import annotations


def shard_range(n_units: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous [begin, end) of `n_units` frames (or streams) owned by `rank`; the first
    n_units % world ranks get one extra unit."""
    if world <= 0 or not 0 <= rank < world or n_units < 0:
        raise ValueError("bad rank/world/n_units")
    base, extra = divmod(n_units, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum over all ranks of a list of floats (identity without a process group)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def gather_rows(local_rows, n_total: int):
    """All ranks' [n_local, K] score rows, concatenated in rank order -> [n_total, K] on every rank.
    Shards may differ in length by one row (see shard_range)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return local_rows
    world = dist.get_world_size()
    width = local_rows.shape[1]
    longest = -(-n_total // world)
    padded = torch.zeros((longest, width), dtype=local_rows.dtype, device=local_rows.device)
    padded[: local_rows.shape[0]] = local_rows
    parts = [torch.empty_like(padded) for _ in range(world)]
    dist.all_gather(parts, padded)
    out = []
    for r, p in enumerate(parts):
        b, e = shard_range(n_total, r, world)
        out.append(p[: e - b])
    return torch.cat(out, dim=0)
