"""Host-side logic of the multi-GPU runs, exercised with two gloo ranks on CPU: which rows / elements a rank
owns, how per-rank timings combine, and the exchange step of the sharded scan (every rank's total reaches
every rank, in rank order, and each rank seeds its scan with the sum of the totals before it).  The three
device calls are replaced here by a stand-in that computes with the CPU oracle - the CUDA kernels themselves
are checked on a GPU in test_gpu_sharded.py."""
import os
import socket

import numpy as np
import torch
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


def test_shard_elements_cover_exactly_on_aligned_boundaries():
    for n in (0, 1, 127, 128, 129, 1000, 1 << 20, (1 << 20) + 77):
        for world in (1, 2, 3, 8):
            edges = [sharding.shard_elements(n, world, r) for r in range(world)]
            assert edges[0][0] == 0 and edges[-1][1] == n
            for (lo, hi), (lo2, _) in zip(edges, edges[1:]):
                assert hi == lo2 and lo <= hi
            assert all(lo % 128 == 0 or lo == n for lo, _ in edges)


class OracleOps:
    """Stand-in for the CUDA binding on CPU tensors (tests only): same call names, int8 input, 8-byte carries
    as zero-extended uint32."""
    DTYPES = {"i8": 0}
    TCU_OK = 0

    @staticmethod
    def check(rc):
        assert rc == 0

    @staticmethod
    def tcu_scan_workspace_bytes(rows, cols, dt, s):
        return 1024

    @staticmethod
    def tcu_reduce_total(x, n, dt, total, ws, ws_bytes, stream):
        from oracle import scan_oracle as so
        y = so.scan_i8(x.numpy()[:n])
        total[0] = (int(y[-1]) if n else 0) & 0xFFFFFFFF
        return 0

    @staticmethod
    def tcu_carry_exclusive_prefix(totals, count, index, dt, carry, stream):
        carry[0] = int(sum(int(v) for v in totals[:index].tolist())) & 0xFFFFFFFF
        return 0

    @staticmethod
    def tcu_scan_ex(x, out, rows, cols, dt, s, ws, ws_bytes, stream, exclusive=0, d_carry_in=None):
        from oracle import scan_oracle as so
        y = so.scan_i8(x.numpy()[:cols], bool(exclusive), init=int(d_carry_in[0]))
        out[:cols] = torch.from_numpy(so.wrap_int32(y))
        return 0


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        lo, hi = sharding.shard_rows(101, world, rank)
        seconds = 0.5 + 0.25 * rank                    # rank 1 is the slow one
        slowest = sharding.max_over_ranks(seconds)
        rate = sharding.whole_job_rate(1000, world, seconds)
        # one array of 1000 + 77 elements split over the ranks
        from paper_2411_17887_b200 import inputs
        n = 1077
        x = inputs.int8_uniform(n, -127, 127, 5)
        elo, ehi = sharding.shard_elements(n, world, rank)
        job = sharding.ShardedScan(ehi - elo, "i8", device="cpu", ops=OracleOps)
        y_local = torch.zeros(ehi - elo, dtype=torch.int32)
        job.scan(torch.from_numpy(x[elo:ehi].copy()), y_local)
        out.put((rank, lo, hi, slowest, rate, elo, ehi, y_local.numpy().tolist(), job.totals.tolist()))
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
    (r0, lo0, hi0, s0, rate0, elo0, ehi0, y0, t0), (r1, lo1, hi1, s1, rate1, elo1, ehi1, y1, t1) = res
    assert (lo0, hi0, lo1, hi1) == (0, 51, 51, 101)
    assert s0 == s1 == 0.75                           # both ranks agree on the slowest time
    assert rate0 == rate1 == 2000 / 0.75
    # the sharded scan: both ranks saw both totals in rank order, and the pieces join into the scan of the whole
    from paper_2411_17887_b200 import inputs
    x = inputs.int8_uniform(1077, -127, 127, 5).astype(np.int64)
    assert (elo0, ehi0, elo1, ehi1) == (0, 640, 640, 1077)
    assert t0 == t1 == [int(x[:640].sum()) & 0xFFFFFFFF, int(x[640:].sum()) & 0xFFFFFFFF]
    assert y0 + y1 == np.cumsum(x).tolist()
