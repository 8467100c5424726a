"""Host-side logic of the multi-GPU benchmark path (no arithmetic of the method).

(batch, window, head) pairs are independent, so N GPUs run N independent batches: every rank draws
its own seeded batch, nothing crosses ranks on the data path, and the only exchange is the timing
reduction below (maximum over ranks, as the slowest rank sets the job's duration).  Works with any
``torch.distributed`` backend: NCCL on GPUs, gloo in the CPU tests.
"""
from __future__ import annotations

import dataclasses

import torch
import torch.distributed as dist


def rank_workload(wl, rank: int):
    """The workload of `rank`: same shape, a seed of its own (rank 0 keeps the configuration's seed)."""
    return dataclasses.replace(wl, seed=wl.seed + 1000 * rank)


def max_over_ranks(values, device="cpu") -> list[float]:
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def job_throughput(units_per_rank: float, ms_per_step_max: float, world: int) -> float:
    """Whole-job units per second: every rank processed `units_per_rank` per step, the step took the slowest rank's time."""
    return units_per_rank * world / (ms_per_step_max * 1e-3)
