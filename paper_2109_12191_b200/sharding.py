"""Host-side helpers for running the step on several GPUs, one process per GPU.

Examples are independent up to the clipped sum (paper section 2: model replication plus gradient
accumulation), so ranks split the examples (or the chunks) of a step, each accumulates its own clipped
sum, ONE all-reduce adds the accumulators, and every rank then adds the same counter-based noise and
divides by the global batch: no broadcast, and the noise is added once to the global sum, never per rank.
"""
from __future__ import annotations


def shard_range(n_items: int, rank: int, world: int):
    """Contiguous, balanced share of range(n_items) for `rank` (the first n_items % world ranks get one more)."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(n_items, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def allreduce_accumulator(acc, dist=None):
    """Sum the fp32 accumulator over all ranks in place (no-op for a single process)."""
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(acc, op=dist.ReduceOp.SUM)
    return acc


def global_batch(local_examples: int, dist=None) -> int:
    """|B| of the step: the examples all ranks processed together.  Shares may be uneven (shard_range), so every
    rank contributes its own count instead of multiplying one rank's count by the number of ranks."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return int(local_examples)
    import torch
    backend = dist.get_backend()
    t = torch.tensor([int(local_examples)], dtype=torch.int64, device="cuda" if backend == "nccl" else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return int(t.item())
