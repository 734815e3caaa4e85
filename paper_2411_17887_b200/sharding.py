"""Host-side helpers for running the scan on several GPUs of one node.

The scan shards across GPUs only as independent problems (whole arrays, or blocks of rows of a
batched scan): every rank runs the single-GPU library on its own share and there is no exchange
step in the data path.  These helpers hold the bookkeeping that such a run needs - which rows a
rank owns, and how per-rank timings combine into a whole-job figure - so that it can be tested
with the ``gloo`` backend on CPU.
"""
from __future__ import annotations

from typing import Tuple

import torch
import torch.distributed as dist


def shard_rows(rows: int, world: int, rank: int) -> Tuple[int, int]:
    """Half-open range [lo, hi) of the rows owned by `rank`: contiguous, disjoint, covering, and
    differing in size by at most one row."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    base, extra = divmod(rows, world)
    lo = rank * base + min(rank, extra)
    hi = lo + base + (1 if rank < extra else 0)
    return lo, hi


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's time: the figure a whole-job throughput has to be computed from."""
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])


def whole_job_rate(units_per_rank: int, world: int, seconds_local: float, device="cpu") -> float:
    """Units processed by all ranks divided by the slowest rank's time."""
    return units_per_rank * world / max_over_ranks(seconds_local, device)
