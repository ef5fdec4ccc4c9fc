"""Host-side logic of the multi-GPU benchmark: how a job is split over ranks and how the ranks'
timings become one number.  The path has no exchange step (rows, windows and requests are
independent), so ranks only meet at a barrier and at the max-reduction of the measured time."""
from __future__ import annotations

from typing import Optional

import torch


def rank_workload(workload, rank: int):
    """Every rank draws its own batch of the same shape (weak scaling): same recipe, another seed."""
    return workload.scaled(seed=workload.seed + 101 * rank)


def shard_rows(rows: int, window: int, rank: int, world: int):
    """[begin, end) of the rows rank `rank` owns when one batch is split (strong scaling).
    Whole windows only: a draft window never straddles two ranks."""
    nw = rows // window
    per, extra = divmod(nw, world)
    w0 = rank * per + min(rank, extra)
    w1 = w0 + per + (1 if rank < extra else 0)
    return w0 * window, w1 * window


def max_over_ranks(x: float, world: int, device: Optional[torch.device] = None) -> float:
    """The slowest rank's time: what the job as a whole took."""
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(x: float, world: int, device: Optional[torch.device] = None) -> float:
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def job_throughput(rows_this_rank: int, steps: int, ms_this_rank: float, world: int,
                   device: Optional[torch.device] = None) -> float:
    """Whole-job tokens/s: the rows all ranks processed over the slowest rank's time."""
    total_rows = sum_over_ranks(float(rows_this_rank), world, device)
    ms = max_over_ranks(ms_this_rank, world, device)
    return total_rows * steps / (ms * 1e-3)
