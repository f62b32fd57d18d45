"""Host-side aggregation for N independent replicas of the round (one process per GPU).

Requests are independent, so the path has no exchange step: every rank runs the same workload on its own GPU
and only the measurement is combined - the job's time is the slowest rank's device time, its work the sum of
the ranks' requests x rounds.  Works with any torch.distributed backend (NCCL on GPUs, gloo in the CPU tests).
"""
from typing import Optional, Tuple

import torch


def whole_job(local_ms: float, local_units: int, dist=None, device: Optional[torch.device] = None) -> Tuple[float, int, float]:
    """Returns (max over ranks of local_ms, sum over ranks of local_units, units per second of the whole job).
    dist: the initialised torch.distributed module, or None for a single process."""
    ms, units = float(local_ms), int(local_units)
    if dist is not None:
        t = torch.tensor([ms], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        u = torch.tensor([units], dtype=torch.int64, device=device)
        dist.all_reduce(u, op=dist.ReduceOp.SUM)
        ms, units = float(t.item()), int(u.item())
    if ms <= 0.0:
        raise ValueError("the timed region has no duration")
    return ms, units, units / (ms / 1000.0)
