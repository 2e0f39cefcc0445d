"""Multi-GPU runs of S2-Attn are independent replicas: the operator has no exchange step (every
(batch, KV head) unit is self-contained), so ranks never communicate on the data path.  The only
collective is the reduction of the measured time: whole-job throughput = work of all ranks divided
by the slowest rank's time.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def slowest_rank_ms(local_ms: float, device=None) -> float:
    """Maximum of `local_ms` over all ranks (the value itself without a process group)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(local_ms)
    t = torch.tensor([float(local_ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, local_ms: float, device=None) -> float:
    """Units per second of the whole job: every rank processed `units_per_rank` units."""
    world = dist.get_world_size() if (dist.is_available() and dist.is_initialized()) else 1
    return world * units_per_rank / (slowest_rank_ms(local_ms, device) * 1e-3)
