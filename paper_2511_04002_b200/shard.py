"""Host-side plumbing for running the codec on several GPUs, one process per GPU.

Token rows are independent through every step of the method except the placement scan, and that
scan is local to a blob, so the path shards by contiguous token ranges with each rank producing its
own blob: there is no exchange step and no collective on the data path.  The only communication is
the bookkeeping below (a barrier, and the reduction of the timing and byte counters).
"""
from __future__ import annotations

from typing import Tuple

import torch
import torch.distributed as dist


def token_range(tokens: int, rank: int, world: int) -> Tuple[int, int]:
    """Rows [start, stop) of rank `rank`: contiguous, disjoint, covering, sizes differing by at most one."""
    if world < 1 or not 0 <= rank < world or tokens < 0:
        raise ValueError("bad partition request: tokens=%d rank=%d world=%d" % (tokens, rank, world))
    base, extra = divmod(tokens, world)
    start = rank * base + min(rank, extra)
    return start, start + base + (1 if rank < extra else 0)


def reduce_job(elapsed_ms: float, bytes_done: float, launches: int, device) -> Tuple[float, float, int]:
    """Whole-job figures from per-rank ones: the slowest rank's time, the sums of bytes and launches."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(elapsed_ms), float(bytes_done), int(launches)
    t = torch.tensor([float(elapsed_ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    s = torch.tensor([float(bytes_done), float(launches)], dtype=torch.float64, device=device)
    dist.all_reduce(s, op=dist.ReduceOp.SUM)
    return float(t.item()), float(s[0].item()), int(s[1].item())
