"""Host-side logic of the multi-GPU run: the path has no exchange step, so ranks only shard.

Every (layer, batch, head) unit of the decoding step is independent, hence one process per GPU
decodes its own image batches (weak scaling) and nothing crosses the link inside the path.  What
the ranks share is bookkeeping: which inputs a rank generates, the barrier around the timed
region, the max-over-ranks of the device time and the whole-job throughput.  These helpers hold
that bookkeeping so that it can be exercised with the gloo backend on CPU.
"""
from __future__ import annotations

from typing import Optional

import torch

from .configs import WorkloadConfig
from .synthetic import SyntheticQKV


def rank_generator(cfg: WorkloadConfig, rank: int, device="cpu") -> SyntheticQKV:
    """Inputs of one rank: the workload's recipe with a rank-specific seed (different images)."""
    return SyntheticQKV(cfg, device=device, seed_offset=rank)


def max_over_ranks(local_ms: float, dist=None, device="cpu") -> float:
    """The step time of the job is the slowest rank's device time."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(local_ms)
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(world: int, tokens_per_rank: int, ms_per_step: float) -> float:
    """Whole-job tokens/s: every rank processes tokens_per_rank per step (weak scaling)."""
    return world * tokens_per_rank / (ms_per_step * 1e-3)


def barrier(dist=None) -> None:
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()
