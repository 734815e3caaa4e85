"""The multi-GPU run is N independent single-GPU scans; its host-side bookkeeping (row ownership,
max-over-ranks timing) is exercised here with two gloo ranks on CPU."""
import os
import socket

import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2411_17887_b200 import sharding


def test_shard_rows_cover_exactly():
    for rows in (0, 1, 7, 4096, 4097):
        for world in (1, 2, 3, 8):
            got = []
            for r in range(world):
                lo, hi = sharding.shard_rows(rows, world, r)
                assert 0 <= lo <= hi <= rows and hi - lo in (rows // world, rows // world + 1)
                got += list(range(lo, hi))
            assert got == list(range(rows))


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        lo, hi = sharding.shard_rows(101, world, rank)
        seconds = 0.5 + 0.25 * rank                    # rank 1 is the slow one
        slowest = sharding.max_over_ranks(seconds)
        rate = sharding.whole_job_rate(1000, world, seconds)
        out.put((rank, lo, hi, slowest, rate))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_gloo():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    (r0, lo0, hi0, s0, rate0), (r1, lo1, hi1, s1, rate1) = res
    assert (lo0, hi0, lo1, hi1) == (0, 51, 51, 101)
    assert s0 == s1 == 0.75                           # both ranks agree on the slowest time
    assert rate0 == rate1 == 2000 / 0.75
