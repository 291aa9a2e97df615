"""Host-side plumbing of the multi-rank benchmark: one process per GPU, independent replicas.

The path has no exchange step on one node ("replicas only"): every rank compresses and decodes
its own seeded gradients.  What the ranks share is the timing protocol: barrier, then the maximum
over ranks of the device time, and the sum of the units processed.  Backend `nccl` on GPUs,
`gloo` in the CPU tests.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_rank():
    """(rank, world size, local rank) from the torchrun environment (defaults: single process)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def rank_seed(rank: int, base: int = 0) -> int:
    """Distinct, reproducible seed block per rank (workers of rank r use seed + w)."""
    return base + 1000 * rank


def init(backend: str, device=None) -> None:
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29511")
    if backend == "nccl":
        dist.init_process_group("nccl", device_id=device)
    else:
        dist.init_process_group(backend)


def barrier(world: int, cuda: bool) -> None:
    if world > 1:
        dist.barrier()
    if cuda:
        torch.cuda.synchronize()


def max_over_ranks(value: float, world: int, device="cpu") -> float:
    if world <= 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, world: int, device="cpu") -> float:
    if world <= 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def job_throughput(units_local: float, ms_local: float, world: int, device="cpu") -> tuple[float, float]:
    """Whole-job rate: units of all ranks / the slowest rank's time.  -> (units per second, ms)."""
    ms = max_over_ranks(ms_local, world, device)
    units = sum_over_ranks(units_local, world, device)
    return units / (ms * 1e-3), ms
