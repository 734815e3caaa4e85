"""One array split into shards (the multi-GPU form of the scan, Section 2.2 with one segment per device),
checked on a single GPU: the shards are scanned one after the other by the same three library calls a rank
would make - total of the shard, exclusive prefix of the totals, scan seeded with that carry - with the
all-gather replaced by writing every shard's total into one device array.  No kernel of one shard waits for
another, so running them in turn on one device is the same computation."""
import numpy as np
import pytest
import torch

from oracle import scan_oracle as so
from paper_2411_17887_b200 import binding as B
from paper_2411_17887_b200 import inputs, sharding

pytestmark = pytest.mark.gpu
TILE = 128 * 128


def gen(dtype, n, seed):
    if dtype == "i8":
        return inputs.int8_uniform(n, -127, 127, seed)
    if dtype == "f16":
        return inputs.f16_uniform(n, 0.0, 1.0, seed)       # all positive: the tolerance is purely relative
    return inputs.bf16_normal(n, seed)


@pytest.mark.parametrize("dtype", ["i8", "f16", "bf16"])
@pytest.mark.parametrize("world,exclusive", [(2, False), (3, True), (8, False)])
def test_shards_scanned_in_turn_join_into_the_whole_scan(dtype, world, exclusive):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from tests.gpu_util import to_device
    n = 37 * TILE + 128 * 5 + 77
    x = gen(dtype, n, 900 + world)
    d_in = to_device(x, dtype)
    d_out = torch.zeros(n, dtype=torch.int32 if dtype == "i8" else torch.float32, device="cuda")
    dt = B.DTYPES[dtype]
    bounds = [sharding.shard_elements(n, world, r) for r in range(world)]
    ranks = [sharding.ShardedScan(hi - lo, dtype, s=16, rank=r, world=world) for r, (lo, hi) in enumerate(bounds)]
    totals = torch.zeros(world, dtype=torch.int64, device="cuda")
    # step 2 on every "rank": the shard totals (what the all-gather would distribute)
    for r, (lo, hi) in enumerate(bounds):
        B.check(B.tcu_reduce_total(d_in[lo:hi], hi - lo, dt, ranks[r].total, ranks[r].ws_ptr, ranks[r].ws_bytes, 0))
        totals[r:r + 1].copy_(ranks[r].total)
    # steps 3-4 on every "rank"
    for r, (lo, hi) in enumerate(bounds):
        job = ranks[r]
        job.gather = lambda dst, src: dst.copy_(totals)      # the exchange, already done above
        job.scan(d_in[lo:hi], d_out[lo:hi], exclusive)
        B.check(B.tcu_scan_device_status(job.ws_ptr, 0))
    got = d_out.cpu().numpy()
    ref = so.scan(x, dtype, exclusive)
    if dtype == "i8":
        assert np.array_equal(got, ref["y32"])
        want_totals = [int(x[lo:hi].astype(np.int64).sum()) & 0xFFFFFFFF for lo, hi in bounds]
        assert totals.cpu().tolist() == want_totals
    else:
        assert (np.abs(got.astype(np.float64) - ref["y"]) <= so.float_tolerance(ref["a"])).all()


@pytest.mark.parametrize("dtype", ["i8", "f16"])
def test_reduce_total_and_carry_chain(dtype):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from tests.gpu_util import to_device
    dt = B.DTYPES[dtype]
    ws_bytes = B.tcu_scan_workspace_bytes(1, 1 << 22, dt, 16)
    ws = torch.zeros(ws_bytes + 256, dtype=torch.uint8, device="cuda")
    ptr = ws.data_ptr() + (-ws.data_ptr()) % 256
    total = torch.zeros(1, dtype=torch.int64, device="cuda")
    for n in (0, 1, 15, 16, 17, 128, TILE - 3, 5 * TILE + 9, 200 * TILE + 1):
        x = gen(dtype, n, n % 89)
        d_in = to_device(x, dtype) if n else torch.zeros(16, dtype=torch.int8, device="cuda")
        total.fill_(-1)
        B.check(B.tcu_reduce_total(d_in, n, dt, total, ptr, ws_bytes, 0))
        if dtype == "i8":
            assert int(total.item()) == int(x.astype(np.int64).sum()) & 0xFFFFFFFF
        else:
            got = float(total.view(torch.float64).item())
            exact = float(so.widen(x, dtype).sum())
            assert abs(got - exact) <= 1e-5 * float(np.abs(so.widen(x, dtype)).sum()) + 1e-6
    # a scan continued across two calls through d_carry_out / d_carry_in equals the scan of the whole
    n = 21 * TILE + 300
    cut = 9 * TILE + 128 * 3          # where the first call stops
    x = gen(dtype, n, 4)
    d_in = to_device(x, dtype)
    d_out = torch.zeros(n, dtype=torch.int32 if dtype == "i8" else torch.float32, device="cuda")
    carry = torch.zeros(1, dtype=torch.int64, device="cuda")
    B.check(B.tcu_scan_ex(d_in[:cut], d_out[:cut], 1, cut, dt, 64, ptr, ws_bytes, 0, d_carry_out=carry))
    B.check(B.tcu_scan_ex(d_in[cut:], d_out[cut:], 1, n - cut, dt, 64, ptr, ws_bytes, 0, d_carry_in=carry, d_carry_out=carry))
    B.check(B.tcu_scan_device_status(ptr, 0))
    got = d_out.cpu().numpy()
    ref = so.scan(x, dtype)
    if dtype == "i8":
        assert np.array_equal(got, ref["y32"])
        assert int(carry.item()) == int(ref["y"][-1]) & 0xFFFFFFFF            # the second call's total, tail included
    else:
        assert (np.abs(got.astype(np.float64) - ref["y"]) <= so.float_tolerance(ref["a"])).all()
        assert abs(float(carry.view(torch.float64).item()) - ref["y"][-1]) <= so.float_tolerance(ref["a"])[-1]
