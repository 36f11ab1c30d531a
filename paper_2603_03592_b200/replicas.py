"""Host-side plumbing for running independent replicas of the check on several GPUs.

The verifier check has no cross-GPU data path: stage boundaries, and the two kinds of a
boundary, are independent, so N GPUs run N replicas of the workload and exchange nothing but
the timing (a barrier around the timed region and a max over ranks).  ``torch.distributed``
is used for exactly that; with one process it is never initialised.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def init_from_env(backend: str = "nccl"):
    """(rank, world_size, local_rank) from the torchrun environment; joins the process group
    when world_size > 1."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        if backend == "nccl":
            torch.cuda.set_device(local_rank)
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world, local_rank


def _reduce_device():
    if dist.get_backend() == "nccl":
        return torch.device("cuda", torch.cuda.current_device())
    return torch.device("cpu")


def barrier() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float) -> float:
    """The slowest rank's figure (a time): what a multi-GPU number must be quoted on."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=_reduce_device())
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float) -> float:
    """Units processed by all replicas together."""
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=_reduce_device())
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def boundaries_of_rank(n_boundaries: int, rank: int, world: int) -> list[int]:
    """Which stage boundaries a rank verifies when a sweep of independent boundaries is spread
    over GPUs: round-robin, every boundary on exactly one rank."""
    return [b for b in range(n_boundaries) if b % world == rank]


def aggregate_throughput(units_this_rank: float, elapsed_ms_this_rank: float) -> float:
    """Whole-job throughput in units per second: all ranks' units over the slowest rank's time."""
    units = sum_over_ranks(units_this_rank)
    ms = max_over_ranks(elapsed_ms_this_rank)
    return units / (ms * 1e-3)


def shutdown() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.barrier()
        dist.destroy_process_group()
