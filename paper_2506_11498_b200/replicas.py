"""Multi-GPU plumbing of the benchmark: one process per GPU, each an independent replica.

The path shards over (batch, KV-head group) units that never exchange data, so N GPUs run N
independent sequences (weak scaling) and the only communication is the timing reduction: the
step time of the job is the slowest rank's.  No data-path collective exists.
"""
from __future__ import annotations

import os


def env_rank_world():
    """(rank, world_size, local_rank) as torchrun exports them; (0, 1, 0) when run directly."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def rank_workload(w, rank: int):
    """The sequence rank `rank` processes: same shape, its own seed (rank 0 keeps the base seed)."""
    return w.with_(seed=w.seed + 1000 * rank)


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """Largest `value` of any rank (all ranks get it); identity without a process group."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_rate(units_per_rank: float, world: int, seconds: float) -> float:
    """Whole-job throughput: every rank processed `units_per_rank` in `seconds` (the max over ranks)."""
    return world * units_per_rank / seconds
