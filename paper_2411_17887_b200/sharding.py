"""Running the scan on several GPUs of one node: one process per GPU, ``torch.distributed`` for the plumbing.

Two ways to use more than one device:

* independent problems (whole arrays, or blocks of rows of a batched scan): every rank runs the single-GPU
  library on its own share and nothing is exchanged; ``shard_rows`` says which rows a rank owns, and
  ``max_over_ranks`` / ``whole_job_rate`` turn per-rank timings into a whole-job figure (``bench.py`` uses them);
* ONE array split into contiguous shards, one per rank (``ShardedScan``): the paper's Section 2.2 with one
  segment per device - every rank takes the total of its shard (step 2), the totals are exchanged (8 bytes per
  rank, an all-gather into local memory), every rank sums the totals of the shards before its own (step 3) and
  scans its shard starting from that carry (step 4 folded into the scan: the carry seeds the first tile).  The
  exchange is the only collective; no kernel reads another device's memory.

All arithmetic happens in the library's CUDA kernels (``tcu_reduce_total``, ``tcu_carry_exclusive_prefix``,
``tcu_scan_ex``); this module only moves pointers and calls the collective.
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


def shard_elements(n: int, world: int, rank: int, align: int = 128) -> Tuple[int, int]:
    """Half-open range [lo, hi) of the elements of one array owned by `rank`: contiguous, disjoint, covering;
    every boundary except the end of the array is a multiple of `align` elements (so that a shard that is a
    view into a larger buffer still starts on a 16-byte boundary in both the input and the output)."""
    blocks = (n + align - 1) // align
    lo_b, hi_b = shard_rows(blocks, world, rank)
    return min(lo_b * align, n), min(hi_b * align, n)


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's time: the figure a whole-job throughput has to be computed from."""
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])


def whole_job_rate(units_per_rank: int, world: int, seconds_local: float, device="cpu") -> float:
    """Units processed by all ranks divided by the slowest rank's time."""
    return units_per_rank * world / max_over_ranks(seconds_local, device)


class ShardedScan:
    """Inclusive or exclusive scan of one array whose shards live on the ranks of a process group.

    ``ops`` is the module that provides ``tcu_reduce_total``, ``tcu_carry_exclusive_prefix``, ``tcu_scan_ex``,
    ``tcu_scan_workspace_bytes``, ``tcu_scan_workspace_init`` and ``check`` - the ctypes binding of the CUDA
    library unless a test passes a stand-in.  ``gather`` exchanges the totals; by default it is
    ``torch.distributed.all_gather_into_tensor`` on the given group (NCCL on GPUs), and with a single process
    it is a copy.
    """

    def __init__(self, max_local_elements: int, dtype: str, s: int = 16, group=None, device="cuda", ops=None,
                 rank: int = None, world: int = None):
        if ops is None:
            from . import binding as ops          # raises if the CUDA library is missing: there is no fallback
        self.ops = ops
        self.dt = ops.DTYPES[dtype]
        self.s = s
        self.group = group
        initialised = dist.is_available() and dist.is_initialized()
        self.rank = rank if rank is not None else (dist.get_rank(group) if initialised else 0)
        self.world = world if world is not None else (dist.get_world_size(group) if initialised else 1)
        self.ws_bytes = ops.tcu_scan_workspace_bytes(1, max_local_elements + 128 * 128, self.dt, s)
        self._ws = torch.zeros(self.ws_bytes + 256, dtype=torch.uint8, device=device)
        self.ws_ptr = self._ws.data_ptr() + (-self._ws.data_ptr()) % 256
        self.max_local = max_local_elements
        # 8-byte carries: this rank's total, everybody's totals, and the carry in front of this shard
        self.total = torch.zeros(1, dtype=torch.int64, device=device)
        self.totals = torch.zeros(self.world, dtype=torch.int64, device=device)
        self.carry = torch.zeros(1, dtype=torch.int64, device=device)

    def _stream(self):
        return torch.cuda.current_stream().cuda_stream if self.total.is_cuda else 0

    def gather(self, totals: torch.Tensor, total: torch.Tensor) -> None:
        if self.world == 1:
            totals.copy_(total)
        else:
            dist.all_gather_into_tensor(totals, total, group=self.group)

    def scan(self, x_local: torch.Tensor, out_local: torch.Tensor, exclusive: bool = False) -> None:
        """Scan this rank's shard in place of the whole array: out_local[i] = (sum of all earlier shards) +
        (scan of x_local up to i).  Every rank of the group must call this, with shards in rank order."""
        ops, n, stream = self.ops, x_local.numel(), self._stream()
        if n > self.max_local:
            raise ValueError("shard larger than this object was sized for")
        ops.check(ops.tcu_reduce_total(x_local, n, self.dt, self.total, self.ws_ptr, self.ws_bytes, stream))
        self.gather(self.totals, self.total)
        ops.check(ops.tcu_carry_exclusive_prefix(self.totals, self.world, self.rank, self.dt, self.carry, stream))
        ops.check(ops.tcu_scan_ex(x_local, out_local, 1, n, self.dt, self.s, self.ws_ptr, self.ws_bytes, stream,
                                  exclusive=int(exclusive), d_carry_in=self.carry))
