"""Multi-GPU plumbing of the benchmark: the decode path shards over independent replicas (one process per GPU,
each with its own batch), so the only things ranks exchange are a barrier and the maximum of their device times.
No collective touches the data path.  Works with any torch.distributed backend: NCCL on GPUs, gloo in the CPU tests."""
from __future__ import annotations

import os
from dataclasses import dataclass
from typing import Sequence

import torch
import torch.distributed as dist


@dataclass
class Replica:
    rank: int
    world: int
    local_rank: int

    @property
    def is_root(self) -> bool:
        return self.rank == 0


def replica_from_env() -> Replica:
    """Rank layout as torchrun exports it (a plain run is a world of one)."""
    return Replica(int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("LOCAL_RANK", "0")))


def init(rep: Replica, backend: str, device=None):
    if rep.world > 1 and not dist.is_initialized():
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=device)
        else:
            dist.init_process_group(backend)


def barrier(rep: Replica):
    if rep.world > 1:
        dist.barrier()


def max_over_ranks(rep: Replica, values: Sequence[float], device="cpu") -> list:
    """Element-wise maximum of each rank's timings: a multi-GPU number is as slow as its slowest rank."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if rep.world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def whole_job_rate(rep: Replica, units_per_rank: float, seconds: float) -> float:
    """Aggregate throughput of `world` replicas that each processed `units_per_rank` in `seconds` (max over ranks)."""
    return rep.world * units_per_rank / seconds


def finish(rep: Replica):
    if rep.world > 1 and dist.is_initialized():
        dist.barrier()
        dist.destroy_process_group()
