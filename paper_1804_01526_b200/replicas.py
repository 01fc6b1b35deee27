"""Replica plumbing for ``bench.py --gpus N``: the path has no exchange step, so N GPUs run N
independent replicas of the workload. The only communication is the barrier around the timed
region and the max-over-ranks of the measured time (``torch.distributed``: NCCL on GPUs, gloo in
the CPU tests)."""
from __future__ import annotations

import os
from dataclasses import dataclass
from typing import Optional


@dataclass
class Replica:
    world: int
    rank: int
    local_rank: int
    backend: Optional[str]

    @property
    def is_root(self) -> bool:
        return self.rank == 0


def init(backend: Optional[str] = None, device=None) -> Replica:
    """Reads RANK / LOCAL_RANK / WORLD_SIZE (set by torch.distributed.run); a single process needs
    no process group."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world == 1:
        return Replica(1, 0, local, None)
    import torch.distributed as dist
    if backend is None:
        import torch
        backend = "nccl" if torch.cuda.is_available() else "gloo"
    kw = {}
    if backend == "nccl" and device is not None:
        kw["device_id"] = device
    dist.init_process_group(backend, **kw)
    return Replica(world, rank, local, backend)


def barrier(rep: Replica) -> None:
    if rep.world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(rep: Replica, value: float, device="cpu") -> float:
    """The slowest rank's time is the job's time."""
    if rep.world == 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(rep: Replica, units_per_rank: float, seconds_max: float) -> float:
    """Whole-job throughput of independent replicas: all ranks' units over the slowest rank's time."""
    return rep.world * units_per_rank / seconds_max


def shutdown(rep: Replica) -> None:
    if rep.world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
