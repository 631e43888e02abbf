"""Multi-GPU plumbing for the benchmark: the path does not shard (one GEMM, one GPU), so
N GPUs run N independent replicas.  The only cross-rank steps are a barrier around the
timed region and the max-over-ranks / sum-over-ranks bookkeeping below; there is no
data-path collective.  Works on any torch.distributed backend (nccl on GPUs, gloo on CPU).
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_world() -> tuple[int, int, int]:
    """(rank, local_rank, world_size) from the launcher's environment; (0, 0, 1) if absent."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str, device: torch.device | None = None):
    """Join the process group when launched with more than one rank."""
    rank, _, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        kwargs = {}
        if backend == "nccl" and device is not None:
            kwargs["device_id"] = device
        dist.init_process_group(backend=backend, rank=rank, world_size=world, **kwargs)
    return rank, world


def barrier():
    if dist.is_initialized():
        dist.barrier()


def aggregate(elapsed_ms: float, units: float, device: torch.device | str = "cpu") -> tuple[float, float]:
    """(max over ranks of elapsed_ms, sum over ranks of units).

    Whole-job throughput is then units_total / max_ms: every rank's work counts, and the
    slowest rank sets the time."""
    if not dist.is_initialized():
        return float(elapsed_ms), float(units)
    t = torch.tensor([float(elapsed_ms)], dtype=torch.float64, device=device)
    u = torch.tensor([float(units)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def any_rank(flag: bool, device: torch.device | str = "cpu") -> bool:
    """True on every rank if `flag` is true on any rank.  Decisions that change how many barriers a
    rank goes through (measuring a workload again) must be taken alike by all ranks."""
    if not dist.is_initialized():
        return bool(flag)
    t = torch.tensor([1 if flag else 0], dtype=torch.int32, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return bool(t.item())


def shutdown():
    if dist.is_initialized():
        dist.destroy_process_group()
