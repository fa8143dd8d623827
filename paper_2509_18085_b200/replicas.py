"""Host-side plumbing of a multi-GPU run: one process per GPU, every rank an
independent replica of the verification step (the path has no exchange step at
the benchmark shape, so there is no data-path collective).  Only the timing is
reduced over ranks: a step is as slow as its slowest replica.
"""
from __future__ import annotations

import os
from dataclasses import dataclass

import torch
import torch.distributed as dist


@dataclass
class Ranks:
    world: int
    rank: int
    local: int

    @property
    def distributed(self) -> bool:
        return self.world > 1


def from_env() -> Ranks:
    return Ranks(int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
                 int(os.environ.get("LOCAL_RANK", "0")))


def init(r: Ranks, backend: str, device=None) -> None:
    """Join the process group (rendezvous from MASTER_ADDR/MASTER_PORT)."""
    if r.distributed and not dist.is_initialized():
        kw = {"device_id": device} if (device is not None and backend == "nccl") else {}
        dist.init_process_group(backend, rank=r.rank, world_size=r.world, **kw)


def barrier(r: Ranks) -> None:
    if r.distributed:
        dist.barrier()


def max_over_ranks(r: Ranks, values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if r.distributed:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def case_offset(r: Ranks, sets_per_rank: int) -> int:
    """Replicas draw distinct synthetic cases: rank r uses cases
    [r * sets_per_rank, (r + 1) * sets_per_rank)."""
    return r.rank * sets_per_rank


def whole_job_rate(r: Ranks, steps_per_rank: int, slowest_ms: float) -> float:
    """Steps per second of the whole job: every rank ran ``steps_per_rank``
    steps in at most ``slowest_ms``."""
    return r.world * steps_per_rank / (slowest_ms * 1e-3)


def finish(r: Ranks) -> None:
    if r.distributed and dist.is_initialized():
        dist.destroy_process_group()
