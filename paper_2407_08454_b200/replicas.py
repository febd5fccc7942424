"""Host-side bookkeeping for running the compression path as independent replicas, one process per GPU.

Units (layer, batch entry, KV head) never exchange data, so several GPUs simply compress different layers.
These helpers hold everything a multi-process run needs beyond the single-GPU library: which layers a rank
takes, the job-wide step time (the slowest rank's), and the aggregate throughput.  They use torch.distributed
only through the process group they are given (NCCL on GPUs, gloo in the CPU tests); no tensor of the
compression path itself ever crosses ranks.
"""
from __future__ import annotations

from typing import List, Optional

import torch


def layers_for_rank(rank: int, world: int, per_rank: int) -> List[int]:
    """Layer indices rank `rank` of `world` compresses: a contiguous, disjoint block of `per_rank` layers."""
    if not (0 <= rank < world) or per_rank < 1:
        raise ValueError("rank must lie in [0, world) and per_rank must be positive")
    return list(range(rank * per_rank, (rank + 1) * per_rank))


def slowest_rank_ms(ms: float, dist=None, device: Optional[torch.device] = None) -> float:
    """The job's time for a timed region is the maximum over ranks of each rank's device-measured time."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(world: int, steps: int, units_per_step: int, ms: float) -> float:
    """Whole-job units per second when every one of `world` ranks ran `steps` steps in `ms` milliseconds."""
    if ms <= 0:
        raise ValueError("elapsed time must be positive")
    return world * steps * units_per_step / (ms * 1e-3)
