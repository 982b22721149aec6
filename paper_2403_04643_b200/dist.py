"""Multi-GPU bookkeeping for the benchmark.

Every (layer, batch, head) of the path is an independent problem, so ranks never exchange
data on the path: each rank works on its own batch (weak scaling).  The only communication
is the barrier around the timed region and the reduction of the timings: the job's time is
the slowest rank's, the job's work is the sum over ranks.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of a rank's own synthetic batch (distinct data per rank, same distribution)."""
    return int(base_seed) + 7777 * int(rank)


def barrier(device=None):
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()
    if device is not None and torch.device(device).type == "cuda":
        torch.cuda.synchronize(device)


def aggregate(ms_local: float, units_local: float, device="cpu"):
    """(max over ranks of the time, sum over ranks of the work units)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms_local), float(units_local)
    t = torch.tensor([float(ms_local)], dtype=torch.float64, device=device)
    u = torch.tensor([float(units_local)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def throughput(ms_job: float, units_job: float) -> float:
    """Whole-job units per second."""
    return units_job / (ms_job * 1e-3)
