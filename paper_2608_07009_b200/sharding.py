"""Host-side plumbing for more than one GPU.

The path shards by request and has no exchange step: caches are managed independently per request and layer
(paper Sec. 3.2), so each rank owns a handle, its requests and their pinned histories, and no collective
touches the data path.  What ranks do share is the measurement: the slowest rank's device time and the sum of
the selections all ranks resolved.
"""
from __future__ import annotations

from typing import List, Tuple


def requests_of_rank(num_requests: int, world_size: int, rank: int) -> List[int]:
    """Request r of a fixed set is served by rank r mod world_size."""
    if not (0 <= rank < world_size):
        raise ValueError("rank out of range")
    return list(range(rank, num_requests, world_size))


def aggregate(elapsed_s: float, units: float, device=None) -> Tuple[float, float]:
    """(max over ranks of elapsed_s, sum over ranks of units); identity without a process group."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(elapsed_s), float(units)
    t = torch.tensor([elapsed_s], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    c = torch.tensor([units], dtype=torch.float64, device=device)
    dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return float(t.item()), float(c.item())
