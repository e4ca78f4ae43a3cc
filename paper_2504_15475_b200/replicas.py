"""Multi-GPU bookkeeping of the benchmark: independent replicas, no data-path collective.

Every (sequence, position) unit of the race is independent and the accepted-prefix scan needs
one sequence's winners only, so N GPUs run N independent copies of the call on their own
batches.  The only exchange is the timing: a barrier on both sides of the timed region and the
maximum of the ranks' device times.  The helpers take the process group's backend as it comes
(NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import torch


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """The largest `value` any rank holds (all ranks get it); `dist` None means one rank."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank_step: int, steps: int, ms_total_this_rank: float, dist=None,
                   device="cpu"):
    """(units per second over all ranks, ms per step) from this rank's device time for `steps` steps.

    Weak scaling: every rank processes `units_per_rank_step` units per step; the job's time is the
    slowest rank's."""
    world = 1 if dist is None or not dist.is_initialized() else dist.get_world_size()
    ms_total = max_over_ranks(ms_total_this_rank, dist, device)
    ms_step = ms_total / steps
    return world * units_per_rank_step / (ms_step * 1e-3), ms_step


def replica_call_index(rank: int, step_set: int) -> int:
    """Seed offset of a rank's input set: replicas race different synthetic batches."""
    return rank * 100 + step_set
