"""Multi-GPU launch plumbing: independent replicas, one process per GPU.

The grouped decode step does not shard (one GPU holds all weights and its own sequences'
cache; there is no exchange step), so N GPUs run N independent copies of the library over
disjoint batches.  The only communication is benchmark bookkeeping: a barrier on both sides
of the timed region and a max over ranks of the device time.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_rank() -> tuple[int, int, int]:
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str | None = None) -> tuple[int, int, int]:
    rank, local_rank, world = env_rank()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29517")
        if backend is None:
            backend = "nccl" if torch.cuda.is_available() else "gloo"
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def barrier():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device: str = "cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device: str = "cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def all_agree(flag: bool, device: str = "cpu") -> bool:
    """True when `flag` holds on every rank (a rank-uniform decision, e.g. when to leave a timing loop)."""
    if not (dist.is_available() and dist.is_initialized()):
        return bool(flag)
    t = torch.tensor([1.0 if flag else 0.0], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MIN)
    return bool(t.item() > 0.5)


def aggregate_throughput(units_this_rank: float, ms_this_rank: float, device: str = "cpu") -> tuple[float, float]:
    """Whole-job throughput: units processed by all ranks / the slowest rank's time.
    Returns (units per second, max ms)."""
    ms = max_over_ranks(ms_this_rank, device)
    units = sum_over_ranks(units_this_rank, device)
    return units / (ms * 1e-3), ms


def shutdown():
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
