"""Host-side plumbing for N independent replicas (one process per GPU).

Selection on one sequence does not shard (every row tile needs every earlier row, the
cascade needs all inherited rows), and sequences are independent, so N GPUs run N replicas
of the path with no data-path collective.  The only communication is the barrier around the
timed region and the MAX over ranks of the measured time; `torch.distributed` carries both
(backend nccl on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import os
from dataclasses import dataclass

import torch
import torch.distributed as dist


@dataclass
class Replica:
    rank: int
    world: int
    local_rank: int

    @property
    def seed(self) -> int:
        """Every replica draws its own synthetic sequences."""
        return self.rank


def from_env() -> Replica:
    return Replica(int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
                   int(os.environ.get("LOCAL_RANK", "0")))


def init_process_group(rep: Replica, backend: str, device=None) -> None:
    if rep.world > 1 and not dist.is_initialized():
        kw = {"device_id": device} if (backend == "nccl" and device is not None) else {}
        dist.init_process_group(backend, rank=rep.rank, world_size=rep.world, **kw)


def barrier(rep: Replica) -> None:
    if rep.world > 1:
        dist.barrier()


def max_over_ranks(rep: Replica, value: float, device="cpu") -> float:
    """The slowest replica defines the job's time."""
    if rep.world == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(rep: Replica, units_per_replica: float, seconds: float) -> float:
    """Units processed by all replicas divided by the (max-over-ranks) time."""
    return rep.world * units_per_replica / seconds


def is_reporter(rep: Replica) -> bool:
    return rep.rank == 0
