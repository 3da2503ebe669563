"""Aggregation of per-rank timings when the benchmark runs N independent replicas.

The hot path has no exchange step (rows, output features and experts are independent), so several GPUs
run replicas of the same workload: no data-path collective.  Only the timing is reduced: the job's time is
the slowest rank's, the job's throughput is all ranks' work divided by that time.
"""
from __future__ import annotations


def job_time_and_throughput(seconds_this_rank: float, units_this_rank: float, dist=None, device=None):
    """Returns (max time over ranks, total units over ranks / that time).  `dist` is torch.distributed (already
    initialised) or None for a single process."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return seconds_this_rank, units_this_rank / seconds_this_rank
    import torch

    t = torch.tensor([seconds_this_rank], dtype=torch.float64, device=device)
    u = torch.tensor([units_this_rank], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item()) / float(t.item())
