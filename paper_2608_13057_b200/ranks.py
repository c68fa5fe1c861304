"""Multi-rank bookkeeping of the benchmark.  The expert block does not shard across GPUs without the
all-to-alls this build leaves out, so N GPUs run N independent ranks ("replicas only"): no data-path
collective.  The only cross-rank traffic is the reduction of the timing itself: the makespan is the
MAX over ranks (the paper's microbenchmark takes an all-reduce MAX of per-rank times, Section 5.1) and
the work done is the SUM of the ranks' units."""
from __future__ import annotations

from typing import Optional, Tuple

import torch
import torch.distributed as dist


def reduce_step(ms_per_step: float, units: float, device: Optional[str] = None) -> Tuple[float, float]:
    """(max over ranks of the step time, sum over ranks of the units one step processes)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms_per_step), float(units)
    dev = torch.device(device) if device else torch.device("cpu")
    t = torch.tensor([ms_per_step], dtype=torch.float64, device=dev)
    u = torch.tensor([units], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())
