"""Multi-GPU runs are independent replicas: every rank serves its own request batches with its own
library context and no data-path collective (the path has no exchange step).  The only cross-rank
traffic is the measurement protocol below: a barrier around the timed region and a max over ranks of
the device time, so that the reported throughput is that of the slowest rank."""
from __future__ import annotations

import socket

import torch
import torch.distributed as dist


def free_port() -> int:
    """A TCP port of the loopback interface that is free right now (rendezvous of ranks started on this machine)."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


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


def _rank_entry(rank: int, n: int, port: int, fn, args) -> None:
    import os
    os.environ.update({"RANK": str(rank), "LOCAL_RANK": str(rank), "WORLD_SIZE": str(n),
                       "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port)})
    fn(rank, *args)


def launch(n: int, fn, *args) -> None:
    """Starts `n` ranks on this machine, one process each, with the rendezvous environment a torchrun launch would
    give them (RANK, LOCAL_RANK, WORLD_SIZE, MASTER_ADDR = 127.0.0.1, MASTER_PORT), and runs fn(rank, *args) in each.
    `fn` must be importable (a module-level function).  Returns when every rank has exited; raises if one failed."""
    import torch.multiprocessing as mp
    mp.spawn(_rank_entry, args=(n, free_port(), fn, args), nprocs=n, join=True)


def init_from_env(backend: str, device: torch.device | None = None) -> None:
    """Joins the process group described by the environment (no-op for a single rank)."""
    import os
    if int(os.environ.get("WORLD_SIZE", "1")) > 1 and not dist.is_initialized():
        if device is not None:
            dist.init_process_group(backend, device_id=device)
        else:
            dist.init_process_group(backend)
