"""Replica bookkeeping for multi-GPU runs.

The regional step shards by request and needs no exchange between GPUs, so N GPUs run N
independent replicas (one process per GPU).  The only collective work is the bracketing barrier
and the max-over-ranks of the measured time; both live here so that they can be exercised with
the gloo backend on CPU.
"""
from __future__ import annotations

import os
from dataclasses import dataclass


@dataclass
class Replica:
    rank: int
    world: int
    local_rank: int

    @property
    def is_lead(self) -> bool:
        return self.rank == 0


def from_env() -> Replica:
    return Replica(int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
                   int(os.environ.get("LOCAL_RANK", "0")))


def init(rep: Replica, backend: str, device=None) -> None:
    """Joins the process group when there is more than one replica (rendezvous from the MASTER_* env)."""
    if rep.world <= 1:
        return
    import torch.distributed as dist
    if dist.is_initialized():
        return
    if backend == "nccl":
        dist.init_process_group(backend, device_id=device)
    else:
        dist.init_process_group(backend, rank=rep.rank, world_size=rep.world)


def barrier(rep: Replica) -> None:
    if rep.world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(rep: Replica, value: float, device="cpu") -> float:
    """The job's time is the slowest replica's time."""
    if rep.world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(rep: Replica, value: float, device="cpu") -> float:
    if rep.world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def replica_seed(rep: Replica, seed: int) -> int:
    """Every replica owns its own batch of requests (weak scaling)."""
    return seed + 17 * rep.rank


def place_requests(rep: Replica, costs, load=None):
    """Which replica serves which incoming request: each request is one monotask without a home and goes, in
    arrival order, to the replica the least-maximum-load rule picks (Sec. 4.3; for such a task that is the least
    loaded replica).  Every rank evaluates the same rule on the same numbers, so no exchange is needed.
    Returns (replica of every request [n] int32, loads after placement [world] float64)."""
    import numpy as np
    from .binding import fd_sched_pack
    load = np.zeros(rep.world, np.float64) if load is None else np.array(load, np.float64)
    costs = np.asarray(costs, np.float64)
    where = fd_sched_pack(load, costs, np.full(costs.size, -1, np.int32))
    return where, load


def job_throughput(units_all_ranks: float, slowest_ms: float) -> float:
    """Whole-job rate: units processed by all replicas divided by the slowest replica's time."""
    return units_all_ranks / (slowest_ms * 1e-3)


def shutdown(rep: Replica) -> None:
    if rep.world > 1:
        import torch.distributed as dist
        if dist.is_initialized():
            dist.destroy_process_group()
