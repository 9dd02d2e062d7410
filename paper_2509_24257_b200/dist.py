"""Multi-process plumbing for running independent verifier replicas, one process per GPU.

The verifier path has no exchange step: sequences are independent and every rank holds a full copy of
the model, so ranks share nothing but the timing protocol (barrier, max over ranks) and the final
aggregation of how many tokens were verified.  NCCL on GPUs, gloo on CPUs.
"""
from __future__ import annotations

import dataclasses
import os
from typing import Tuple

import torch
import torch.distributed as dist


def env_ranks() -> Tuple[int, int, int]:
    return int(os.environ.get("RANK", 0)), int(os.environ.get("WORLD_SIZE", 1)), int(os.environ.get("LOCAL_RANK", 0))


def init(backend: str | None = None) -> Tuple[int, int, int]:
    """Joins the process group described by RANK / WORLD_SIZE / MASTER_ADDR / MASTER_PORT (no-op for one rank)."""
    rank, world, local = env_ranks()
    if world > 1 and not dist.is_initialized():
        if backend is None:
            backend = "nccl" if torch.cuda.is_available() else "gloo"
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        kwargs = {}
        if backend == "nccl":
            torch.cuda.set_device(local)
            kwargs["device_id"] = torch.device("cuda", local)
        dist.init_process_group(backend=backend, rank=rank, world_size=world, **kwargs)
    return rank, world, local


def _device() -> torch.device:
    if dist.is_initialized() and dist.get_backend() == "nccl":
        return torch.device("cuda", torch.cuda.current_device())
    return torch.device("cpu")


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float) -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=_device())
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float) -> float:
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=_device())
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def replica_workload(wl, rank: int):
    """The workload of one replica: same model and shapes, its own token streams / check set / tampering."""
    if rank == 0:
        return wl
    return dataclasses.replace(wl, name=f"{wl.name}-r{rank}", token_seed_offset=1000 * rank)


def aggregate_throughput(units_this_rank: float, seconds_this_rank: float) -> float:
    """Whole-job units per second: all ranks' units over the slowest rank's time."""
    total = sum_over_ranks(units_this_rank)
    slowest = max_over_ranks(seconds_this_rank)
    return total / slowest if slowest > 0 else 0.0


def shutdown() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
