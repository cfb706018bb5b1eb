"""Multi-GPU runs are independent replicas: every rank serves its own request batches with its own
library context and no data-path collective (the path has no exchange step).  The only cross-rank
traffic is the measurement protocol below: a barrier around the timed region and a max over ranks of
the device time, so that the reported throughput is that of the slowest rank."""
from __future__ import annotations

import torch
import torch.distributed as dist


def world() -> int:
    return dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1


def barrier() -> None:
    if world() > 1:
        dist.barrier()


def max_over_ranks(value: float, device: torch.device | str = "cpu") -> float:
    """The largest `value` any rank holds (device milliseconds of the timed region)."""
    if world() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, ms_per_rank: float, device: torch.device | str = "cpu") -> float:
    """Aggregate rate of the job: all ranks' units divided by the slowest rank's time (units per second)."""
    return units_per_rank * world() / (max_over_ranks(ms_per_rank, device) * 1e-3)
