"""Host-side logic for running the step on several GPUs as independent replicas.

The draft-and-verify step has no exchange between engines, so N GPUs run N
copies of it, one process per GPU, each on its own seeded batch.  The only
communication is bookkeeping for the measurement: a barrier around the timed
region, the maximum of the ranks' device times, and the sum of the tokens they
processed.  Nothing here touches the data path.
"""
from __future__ import annotations

import dataclasses
import os
from typing import Optional, Tuple

import torch


@dataclasses.dataclass
class Replica:
    rank: int
    local_rank: int
    world: int
    device: torch.device  # where the bookkeeping tensors live (cpu under gloo)
    active: bool  # a process group is up

    @property
    def is_root(self) -> bool:
        return self.rank == 0


def init(backend: str = "nccl", device: Optional[torch.device] = None) -> Replica:
    """Reads RANK / LOCAL_RANK / WORLD_SIZE (set by torch.distributed.run) and
    brings up a process group when there is more than one rank."""
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if device is None:
        device = torch.device("cuda", local) if backend == "nccl" else torch.device("cpu")
    active = world > 1
    if active:
        import torch.distributed as dist
        kw = {"device_id": device} if backend == "nccl" else {}
        dist.init_process_group(backend, rank=rank, world_size=world, **kw)
    return Replica(rank, local, world, device, active)


def workload_for_rank(w, rank: int):
    """Every replica draws its own batch: same shapes, different seed."""
    if rank == 0:
        return w
    return dataclasses.replace(w, seed_salt=w.seed_salt + 100 * rank)


def barrier(r: Replica) -> None:
    if r.active:
        import torch.distributed as dist
        dist.barrier()


def aggregate(r: Replica, tokens_local: int, ms_local: float) -> Tuple[int, float]:
    """(tokens of all ranks, slowest rank's time) - the job's throughput is their ratio."""
    if not r.active:
        return int(tokens_local), float(ms_local)
    import torch.distributed as dist
    t = torch.tensor([float(ms_local)], dtype=torch.float64, device=r.device)
    n = torch.tensor([int(tokens_local)], dtype=torch.int64, device=r.device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return int(n.item()), float(t.item())


def shutdown(r: Replica) -> None:
    if r.active:
        import torch.distributed as dist
        dist.destroy_process_group()
