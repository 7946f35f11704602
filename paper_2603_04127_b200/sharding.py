"""Data-parallel plumbing of the benchmark and of multi-process runs: the path shards over independent (batch, head)
units, so ranks take disjoint batches and exchange nothing on the data path; only the gradient of the per-head geometry
M, which sums over the batch, is all-reduced (as any data-parallel parameter gradient). Works with the NCCL backend
(one rank per GPU) and with gloo on CPU tensors."""
from __future__ import annotations

import os
from dataclasses import replace

import torch
import torch.distributed as dist

from . import inputs


def env_rank_world():
    """(rank, world size, local rank) from the launcher's environment; (0, 1, 0) when not launched by one."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("LOCAL_RANK", "0")))


def rank_workload(wl: inputs.Workload, rank: int) -> inputs.Workload:
    """The batch rank `rank` processes under weak scaling: the same shapes and distributions, its own random streams
    (the workload id, which seeds every tensor, is shifted by the rank). M and W are parameters, not data: the shift
    changes their draws too, so callers that need replicated parameters take them from rank 0's workload."""
    return replace(wl, wid=wl.wid + 100 * rank)


def all_reduce_dm(dM: torch.Tensor) -> torch.Tensor:
    """Sum the gradient of M over the ranks, in place (no-op for a single process)."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(dM, op=dist.ReduceOp.SUM)
    return dM


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's time: a multi-rank step is as slow as its slowest rank."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: float, world: int, seconds_slowest: float) -> float:
    """Whole-job throughput: the units all ranks processed divided by the slowest rank's time."""
    return world * units_per_rank / seconds_slowest
