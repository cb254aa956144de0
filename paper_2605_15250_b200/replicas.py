"""Multi-GPU runs of the decode path are independent replicas: the path partitions over sequences with
no exchange step, so every rank owns its own batch and there is no data-path collective.  This module
holds the only cross-rank logic there is: which batch a rank draws, and how a timing is reduced."""
from __future__ import annotations

import torch
import torch.distributed as dist


def replica_seed(base_seed: int, rank: int) -> int:
    """Seed of the synthetic batch of `rank`: distinct batches, same shapes."""
    return base_seed + 0x100 * rank


def max_over_ranks(ms: float, device: torch.device | str = "cpu") -> float:
    """Slowest rank's time (the job finishes when the last replica does).  No-op without a process group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tokens_per_s(world: int, batch: int, s_q: int, ms_per_step: float) -> float:
    """Whole-job throughput: every rank decodes batch * s_q tokens per step (weak scaling)."""
    return world * batch * s_q / (ms_per_step * 1e-3)
