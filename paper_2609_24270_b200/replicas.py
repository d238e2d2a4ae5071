"""Whole-job numbers for independent replicas.

The path does not shard: the SM map and the chunk map are measurements of one chip, so every GPU
runs its own discovery, its own plans and its own GEMMs, and nothing is exchanged on the data path.
The only communication is this: after the timed region every rank contributes its time per step,
the job's time is the slowest rank's, and the job's throughput is the work of all ranks over that
time.  Works with any torch.distributed backend (nccl on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def slowest_rank_ms(ms_per_step: float, device: torch.device | str = "cpu") -> float:
    """Max over ranks of the per-step time (identity when no process group is up)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms_per_step)
    t = torch.tensor([float(ms_per_step)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(ms_per_step: float, work_per_step_per_rank: float, device: torch.device | str = "cpu"):
    """(whole-job work per second, job ms per step): every rank does `work_per_step_per_rank` per
    step (weak scaling), the job advances at the pace of the slowest rank."""
    world = dist.get_world_size() if (dist.is_available() and dist.is_initialized()) else 1
    ms = slowest_rank_ms(ms_per_step, device)
    return world * work_per_step_per_rank / (ms * 1e-3), ms
