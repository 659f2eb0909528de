"""Host-side bookkeeping for running N independent replicas of the decode workload (one process per GPU).

The path has no exchange step between units, so multi-GPU runs are plain replicas; the only communication is
the reduction of the per-rank step time (maximum over ranks) that the whole-job throughput is computed from.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def max_over_ranks(value: float, device: str = "cpu") -> float:
    """Maximum of a per-rank scalar; identity when no process group is initialised."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(batch_per_replica: int, world_size: int, ms_per_step: float) -> float:
    """Every replica decodes `batch_per_replica` tokens per step; the job's rate uses the slowest rank's step time."""
    return world_size * batch_per_replica / (ms_per_step * 1e-3)


def replica_salt(rank: int, layer: int) -> int:
    """Distinct synthetic data per (rank, layer replica)."""
    return 100 * rank + layer
