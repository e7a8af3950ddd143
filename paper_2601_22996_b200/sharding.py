"""Multi-GPU sharding of the path: instances are independent, so each rank takes its own block of
instances and nothing is exchanged on the data path.  Only the timing (max over ranks) and the unit
counts (sum over ranks) are reduced for reporting.  Works with any torch.distributed backend."""
from __future__ import annotations

import torch


def shard_first_instance(rank: int, instances_per_rank: int) -> int:
    """Weak scaling: rank r generates / owns instances [r*I, (r+1)*I) of the seeded stream."""
    return rank * instances_per_rank


def reduce_report(times, counts, device, world: int):
    """(max over ranks of each time, sum over ranks of each count) as python floats."""
    t = torch.tensor(list(times), dtype=torch.float64, device=device)
    c = torch.tensor(list(counts), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return [float(x) for x in t.tolist()], [float(x) for x in c.tolist()]
