"""Replica bookkeeping for runs on several GPUs.

One batch-1 sequence does not shard (Section 4.1 of the paper runs on a single GPU; every step
depends on the previous one), so N GPUs run N independent replicas: no data-path collective,
only a barrier around the timed region and a max over the ranks' device times.
"""
from __future__ import annotations


def barrier(dist, world: int) -> None:
    if world > 1:
        dist.barrier()


def max_over_ranks(dist, world: int, ms: float, device="cpu") -> float:
    """Largest of the ranks' timings (every rank gets it)."""
    if world <= 1:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, max_ms: float) -> float:
    """Units per second of the whole job: all ranks' units over the slowest rank's time."""
    return world * units_per_rank / (max_ms * 1e-3)
