"""Data-parallel replicas: the only multi-GPU form this path has.

The independent unit of the draft / verify path is the sequence: a batch shards across GPUs with no
exchange at all (every replica holds the whole MTP head). This module holds the little host logic that
sharding needs -- which sequences a rank takes, and the max-over-ranks reduction of a device time --
so that it can be tested with `gloo` on CPU. It contains none of the method's arithmetic.
"""
from __future__ import annotations


def shard_sequences(n_sequences: int, world_size: int, rank: int) -> range:
    """Contiguous block of sequence indices of `rank`: sizes differ by at most one, every sequence
    belongs to exactly one rank."""
    if not 0 <= rank < world_size:
        raise ValueError("rank outside the world")
    base, extra = divmod(n_sequences, world_size)
    lo = rank * base + min(rank, extra)
    return range(lo, lo + base + (1 if rank < extra else 0))


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """Largest `value` over all ranks (a job is as slow as its slowest replica). `dist` is
    torch.distributed (initialised) or None for a single process."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: int, world_size: int, steps: int, max_ms: float) -> float:
    """Whole-job units per second when every rank processes `units_per_rank` per step (weak scaling)
    and the timed region took `max_ms` on the slowest rank."""
    return world_size * units_per_rank * steps / (max_ms * 1e-3)
