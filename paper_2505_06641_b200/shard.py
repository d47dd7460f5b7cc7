"""Sharding of the batched workload over ranks and the reduction of per-rank timings (host logic only).

Independent scheduling instances are the unit of sharding: rank r of a world of N takes instances
[r * n, (r + 1) * n) of the global numbering, n instances per rank (weak scaling).  No data crosses ranks on
the data path; the only collectives are the two small reductions below, used to report whole-job figures.
"""
from __future__ import annotations

from typing import Sequence, Tuple

import torch
import torch.distributed as dist


def instance_shard(rank: int, world: int, instances_per_rank: int) -> Tuple[int, int]:
    """(first global instance, number of instances) of ``rank``."""
    if not (0 <= rank < world) or instances_per_rank < 0:
        raise ValueError("bad rank / world / instances_per_rank")
    return rank * instances_per_rank, instances_per_rank


def reduce_step_stats(ms: float, counts: Sequence[int], device) -> Tuple[float, list]:
    """Slowest rank's time (MAX) and job-wide totals of ``counts`` (SUM); identity when not distributed."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms), [int(c) for c in counts]
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    c = torch.tensor(list(counts), dtype=torch.int64, device=device)
    dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return float(t.item()), [int(x) for x in c.tolist()]
