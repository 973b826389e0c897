"""Multi-GPU host logic: one process per GPU, units sharded by sequence, no data-path collective.

Every (sequence, KV head) unit of the SubGen cache is independent in update, prefill and query, so ranks
never exchange cache data. Each rank serves its own batch of sequences (weak scaling); the only
communication is the barrier around the timed region and a MAX reduction of the measured time.
"""
from __future__ import annotations

from typing import Optional

import torch


def rank_workload(w, rank: int):
    """The batch of sequences rank `rank` serves: same shape, its own seeded data."""
    return w.scaled(data_seed=w.data_seed + 7919 * int(rank))


def max_over_ranks(value: float, dist=None, device: Optional[str] = None) -> float:
    """MAX of a host scalar over all ranks (identity without a process group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_steps_per_s(world: int, steps_per_rank: int, slowest_ms: float) -> float:
    """Whole-job throughput: every rank advanced its batch by steps_per_rank steps within slowest_ms."""
    return world * steps_per_rank / (slowest_ms * 1e-3)
