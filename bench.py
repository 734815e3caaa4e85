#!/usr/bin/env python
"""Benchmark of the tensor-core-unit scan library on B200.

    python bench.py --gpus N --steps K --warmup W            # this library (CUDA, through the C ABI)
    python bench.py --impl reference --steps K --warmup W    # the CPU oracle on the host cores
    python bench.py --fixed-cost                             # where the microseconds of a small launch go
    python bench.py --wait-counters | --tile-trace           # debug build: waits per role; the life of a tile
    python bench.py --profile ...                            # the bare loop that is wrapped in ncu

A step is one scan of the headline workload: n = 2^28 int8 values uniform in [-127, 127],
int32 output, s = 16 (256 MiB read, 1 GiB written).  With N > 1 every rank scans its own
array of that size (independent problems, no exchange in the data path): weak scaling.
Prints one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "elements/sec and achieved HBM GB/s (% of peak) for n=2^28 scan on 1 B200"
N_ELEMS = 1 << 28
S_TILE = 16
BYTES_PER_ELEM = 5          # int8 read + int32 written
FALLBACK_HBM_GBS = 6650.0
# From the ncu capture of the main kernel on 2^26 elements (profiles/tcu_scan_kernel_int8_s16_n2p26_ncu_full.md):
# DRAM bytes read / input bytes, and bytes the SMs wrote to L2 / output bytes.  DRAM *write* bytes of a capture are
# not used: tens of MB of the output are still dirty in L2 when the kernel ends, a constant that does not grow with n.
NCU_READ_RATIO = 1.002
NCU_WRITE_RATIO = 1.004


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def cpu_model() -> str:
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(gpu_index)], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        sm, smmax, reasons = [], [], set()
        for line in self.tmp.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                smmax.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.unlink(self.tmp.name)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(smmax), samples=len(sm), reasons=sorted(reasons))
        return out


def oracle_leg(x: np.ndarray, reps: int):
    """Time the CPU oracle as it stands (sequential int64 loop, one thread) on the whole input."""
    from oracle import scan_oracle as so
    best, y = None, None
    for _ in range(reps):
        t0 = time.perf_counter()
        y = so.scan_i8(x)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    return x.size / best, y


def oracle_all_cores(x: np.ndarray, threads: int):
    """A second, separately labelled CPU figure: the same C loop of the oracle on every host core.  The array is
    cut into one chunk per thread; pass 1 scans every chunk from zero to learn its total, pass 2 scans it again
    starting from the sum of the chunks before it (the classical chunked two-pass scan; ctypes releases the GIL
    inside the C loop, so Python threads do run side by side)."""
    from oracle import scan_oracle as so
    bounds = np.linspace(0, x.size, threads + 1).astype(np.int64)
    totals = [0] * threads

    def pass1(k):
        totals[k] = int(so.scan_i8(x[bounds[k]:bounds[k + 1]])[-1]) if bounds[k + 1] > bounds[k] else 0

    def pass2(k, carry):
        so.scan_i8(x[bounds[k]:bounds[k + 1]], init=carry)

    def run(fn, args):
        ts = [threading.Thread(target=fn, args=a) for a in args]
        for t in ts:
            t.start()
        for t in ts:
            t.join()

    t0 = time.perf_counter()
    run(pass1, [(k,) for k in range(threads)])
    carries = np.concatenate(([0], np.cumsum(totals)[:-1]))
    run(pass2, [(k, int(carries[k])) for k in range(threads)])
    return x.size / (time.perf_counter() - t0)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2411_17887_b200 import inputs
    x = inputs.make(inputs.CONFIGS["C3"])
    from oracle import scan_oracle as so
    for _ in range(args.warmup):
        so.scan_i8(x[: 1 << 24])
    t0 = time.perf_counter()
    for _ in range(args.steps):
        so.scan_i8(x)
    dt = time.perf_counter() - t0
    value = x.size * args.steps / dt
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "elements/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "i64", "data": "synthetic",
        "config": {"workload": "C3: inclusive scan, n=2^28 int8 uniform[-127,127] -> int32, s=16, one array per GPU"},
        "cpu_baseline": {"value": value, "unit": "elements/s", "cores": 1, "kind": "oracle",
                         "sample": f"whole 2^28-element input per step, {args.steps} steps",
                         "host_cores": os.cpu_count(), "cpu_model": cpu_model()},
        "e2e": {"value": value, "unit": "elements/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


class Timer:
    """CUDA-event timing of back-to-back launches on torch's current stream (the stream every call is given)."""

    def __init__(self, torch):
        self.torch = torch

    def loop(self, call, reps):
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            call()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    def each(self, call, reps):
        """Every launch between its own pair of events: median and best in microseconds."""
        torch = self.torch
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
        ev[0].record()
        for i in range(reps):
            call()
            ev[i + 1].record()
        torch.cuda.synchronize()
        us = [1e3 * ev[i].elapsed_time(ev[i + 1]) for i in range(reps)]
        return statistics.median(us), min(us)


def time_extra(B, torch, x, rows, cols, dt, s, ws_ptr, ws_bytes, reps=10, **options):
    """One of the other workloads: microseconds per scan, GB/s of algorithmic traffic, and the call's statistics."""
    out = torch.empty(rows * cols, dtype=torch.int32 if dt == 0 else torch.float32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    plain = not (set(options) - {"exclusive"})      # the three basic entry points cost the host least

    def call():
        if not plain:
            B.check(B.tcu_scan_ex(x, out, rows, cols, dt, s, ws_ptr, ws_bytes, stream, **options))
        elif rows > 1:
            B.check(B.tcu_scan_batched(x, out, rows, cols, dt, s, options.get("exclusive", 0), ws_ptr, ws_bytes, stream))
        elif options.get("exclusive", 0):
            B.check(B.tcu_scan_exclusive(x, out, cols, dt, s, ws_ptr, ws_bytes, stream))
        else:
            B.check(B.tcu_scan_inclusive(x, out, cols, dt, s, ws_ptr, ws_bytes, stream))
    for _ in range(3):
        call()
    torch.cuda.synchronize()
    ms = Timer(torch).loop(call, reps)
    stats = B.tcu_scan_last_stats()
    nbytes = rows * cols * ((1 if dt == 0 else 2) + 4)
    del out
    return {"us": round(1e3 * ms, 2), "GBps": round(nbytes / (ms * 1e-3) / 1e9, 1)}, stats


def fixed_cost(args):
    """Takes the time of a small launch apart with the kernel's own time stamps (%globaltimer at fixed points,
    written only when the caller passes a stamp buffer) and with host clocks around the call."""
    import torch
    from paper_2411_17887_b200 import binding as B
    torch.cuda.set_device(0)
    stream = torch.cuda.current_stream().cuda_stream
    ws_bytes = B.tcu_scan_workspace_bytes(1, 1 << 26, 0, 16)
    ws = torch.empty(ws_bytes + 256, dtype=torch.uint8, device="cuda")
    ws_ptr = ws.data_ptr() + (-ws.data_ptr()) % 256
    B.check(B.tcu_scan_workspace_init(ws_ptr, ws_bytes, stream))
    g = torch.Generator(device="cuda").manual_seed(1)
    xi = torch.randint(-127, 128, (1 << 26,), device="cuda", dtype=torch.int8, generator=g)
    xf = (torch.rand(1 << 26, device="cuda", generator=g) * 2 - 1).half()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    stamps = torch.zeros(sms * B.TCU_SCAN_STAMPS_PER_CTA, dtype=torch.int64, device="cuda")
    report = []
    for name, x, n, dt in [("C1 n=2^16 int8", xi, 1 << 16, 0), ("C2 n=2^24 fp16", xf, 1 << 24, 1), ("C5 n=2^26 fp16", xf, 1 << 26, 1)]:
        out = torch.empty(n, dtype=torch.int32 if dt == 0 else torch.float32, device="cuda")

        def plain():
            B.check(B.tcu_scan_inclusive(x, out, n, dt, 16, ws_ptr, ws_bytes, stream))

        def stamped():
            B.check(B.tcu_scan_ex(x, out, 1, n, dt, 16, ws_ptr, ws_bytes, stream, d_stamps=stamps))
        for _ in range(5):
            plain()
        torch.cuda.synchronize()
        t = Timer(torch)
        back_to_back_us = 1e3 * t.loop(plain, 200)
        med_us, best_us = t.each(plain, 200)
        # host cost of one call (argument checks, tensor-map encoding, launch), the GPU kept busy so nothing blocks
        t0 = time.perf_counter()
        for _ in range(200):
            plain()
        host_us = 1e6 * (time.perf_counter() - t0) / 200
        torch.cuda.synchronize()
        # device-side stamps: isolated launches (stream idle before each), and a launch right behind another one
        rows = {}
        for mode in ("isolated", "behind_another"):
            acc = []
            for _ in range(20):
                stamps.zero_()
                torch.cuda.synchronize()
                if mode == "behind_another":
                    plain()
                stamped()
                torch.cuda.synchronize()
                st = stamps.cpu().numpy().reshape(sms, B.TCU_SCAN_STAMPS_PER_CTA)
                grid = min(sms, (n + 16383) // 16384)
                st = st[:grid]
                t_first = st[:, 0].min()
                acc.append([float((st[:, k][st[:, k] > 0] - t_first).max()) / 1e3 if (st[:, k] > 0).any() else None
                            for k in range(len(B.STAMP_NAMES))])
            rows[mode] = {nm: round(statistics.median([a[k] for a in acc if a[k] is not None]), 2)
                          for k, nm in enumerate(B.STAMP_NAMES) if any(a[k] is not None for a in acc)}
        nbytes = n * ((1 if dt == 0 else 2) + 4)
        report.append({"workload": name + ", s=16", "back_to_back_us": round(back_to_back_us, 2),
                       "per_launch_us_median": round(med_us, 2), "per_launch_us_best": round(best_us, 2),
                       "host_us_per_call": round(host_us, 2), "roofline_us_at_measured_peak": round(nbytes / measured_peak()[0] / 1e3, 2),
                       "stamps_us_after_first_cta_entry_max_over_ctas": rows})
        del out
    print(json.dumps({"fixed_cost": report}))


def wait_counters(args):
    """Where each role of the kernel waits, at the headline size: loads the debug build of the library
    (``python -m paper_2411_17887_b200.build --profile``, compiled with -DTCU_PROFILE), runs one scan per workload
    with a counter buffer attached and prints, per role, the mean over the CTAs of the time spent in each wait.
    Counters perturb the kernel (it runs about a quarter slower); read the proportions, not the totals."""
    import ctypes
    import torch
    from paper_2411_17887_b200 import build as lib_build
    lib = ctypes.CDLL(lib_build.build_profile())
    vp, sz, ci = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
    lib.tcu_scan_workspace_bytes.argtypes = [sz, sz, ci, ci]
    lib.tcu_scan_workspace_bytes.restype = sz
    lib.tcu_scan_workspace_init.argtypes = [vp, sz, vp]
    lib.tcu_scan_inclusive.argtypes = [vp, vp, sz, ci, ci, vp, sz, vp]
    lib.tcu_scan_batched.argtypes = [vp, vp, sz, sz, ci, ci, ci, vp, sz, vp]
    lib.tcu_scan_debug_set_profile_buffer.argtypes = [vp]
    torch.cuda.set_device(0)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    ghz = torch.cuda.get_device_properties(0).clock_rate / 1e6 if hasattr(torch.cuda.get_device_properties(0), "clock_rate") else 1.965
    n = 1 << 28
    ws_bytes = lib.tcu_scan_workspace_bytes(4096, 65536, 0, 16)
    ws = torch.zeros(ws_bytes + 256, dtype=torch.uint8, device="cuda")
    ws_ptr = ws.data_ptr() + (-ws.data_ptr()) % 256
    prof = torch.zeros(sms * 64, dtype=torch.int64, device="cuda")
    assert lib.tcu_scan_debug_set_profile_buffer(prof.data_ptr()) == 0
    g = torch.Generator(device="cuda").manual_seed(1)
    xi = torch.randint(-127, 128, (n,), device="cuda", dtype=torch.int8, generator=g)
    xf = (torch.rand(n, device="cuda", generator=g) * 2 - 1).half()
    out = torch.empty(n, dtype=torch.int32, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    names = {0: "producer: wait for a free input stage", 1: "producer: ticket", 2: "producer: issue loads",
             4: "scan MMA: wait for the tile", 5: "scan MMA: wait for a free accumulator", 6: "scan MMA: issue",
             8: "total MMA: wait for the tile", 9: "total MMA: wait for a free small accumulator", 10: "total MMA: issue",
             12: "look-back warp: wait for the tile's total", 13: "look-back warp: walk",
             28: "totals warps: wait", 29: "totals warps: work",
             32: "store group 0: wait for the carry", 33: "store group 0: wait for the accumulator",
             34: "store group 0: TMEM load", 35: "store group 0: add + stage", 36: "store group 0: read back + store"}
    counts = {3: "tiles per CTA", 14: "look-back rounds of one warp", 15: "tiles of one look-back warp"}
    report = []
    for label, fn in [("C3 int8 n=2^28", lambda: lib.tcu_scan_inclusive(xi.data_ptr(), out.data_ptr(), n, 0, 16, ws_ptr, ws_bytes, st)),
                      ("fp16 n=2^28", lambda: lib.tcu_scan_inclusive(xf.data_ptr(), out.data_ptr(), n, 1, 16, ws_ptr, ws_bytes, st)),
                      ("C4-shaped 4096x65536 fp16", lambda: lib.tcu_scan_batched(xf.data_ptr(), out.data_ptr(), 4096, 65536, 1, 16, 0, ws_ptr, ws_bytes, st))]:
        for _ in range(2):
            assert fn() == 0
        torch.cuda.synchronize()
        prof.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        assert fn() == 0
        e1.record()
        torch.cuda.synchronize()
        p = prof.cpu().numpy().reshape(sms, 64)
        entry = {"workload": label, "us_with_counters": round(1e3 * e0.elapsed_time(e1), 1),
                 "mean_us_per_cta": {nm: round(float(p[:, k].mean()) / (ghz * 1e3), 1) for k, nm in names.items()},
                 "mean_count_per_cta": {nm: round(float(p[:, k].mean()), 1) for k, nm in counts.items()}}
        report.append(entry)
    print(json.dumps({"wait_counters": report, "sm_ghz_assumed": ghz}))


def tile_trace(args):
    """The life of a tile and the rate at which tiles are completed over a launch: loads the debug build of the
    library (-DTCU_PROFILE), attaches a buffer of eight time stamps per tile (claimed, row-total product issued, totals
    warps woken, total published, walk started, carry known, store started, stored; ``%globaltimer``), runs one scan
    per workload and prints (a) the median time from the claim to each point for tiles of the first waves and of the
    steady state, (b) the algorithmic GB/s at which tiles are stored between given fractions of the launch.  The
    stamps slow the kernel by a few per cent; the point is where the time goes, and whether the middle of a launch runs
    at the rate of a plain copy of the same traffic."""
    import ctypes
    import numpy as np
    import torch
    from paper_2411_17887_b200 import build as lib_build
    lib = ctypes.CDLL(lib_build.build_profile())
    vp, sz, ci = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
    lib.tcu_scan_workspace_bytes.argtypes = [sz, sz, ci, ci]
    lib.tcu_scan_workspace_bytes.restype = sz
    lib.tcu_scan_workspace_init.argtypes = [vp, sz, vp]
    lib.tcu_scan_inclusive.argtypes = [vp, vp, sz, ci, ci, vp, sz, vp]
    lib.tcu_scan_debug_set_trace_buffer.argtypes = [vp]
    torch.cuda.set_device(0)
    st = torch.cuda.current_stream().cuda_stream
    g = torch.Generator(device="cuda").manual_seed(1)
    points = ["claimed", "row_total_product_issued", "totals_warps_woken", "total_published", "walk_started", "carry_known",
              "store_started", "stored"]
    report = []
    for label, logn, dt in [("C3 int8 n=2^28", 28, 0), ("fp16 n=2^28", 28, 1), ("C5 fp16 n=2^26", 26, 1)]:
        n = 1 << logn
        tiles = n // (128 * 128)
        ws_bytes = lib.tcu_scan_workspace_bytes(1, n, dt, 16)
        ws = torch.zeros(ws_bytes + 256, dtype=torch.uint8, device="cuda")
        ws_ptr = ws.data_ptr() + (-ws.data_ptr()) % 256
        x = (torch.randint(-127, 128, (n,), device="cuda", dtype=torch.int8, generator=g) if dt == 0
             else (torch.rand(n, device="cuda", generator=g) * 2 - 1).half())
        out = torch.empty(n, dtype=torch.int32, device="cuda")
        trace = torch.zeros(tiles * 8, dtype=torch.int64, device="cuda")
        lib.tcu_scan_debug_set_trace_buffer(None)
        for _ in range(3):
            assert lib.tcu_scan_inclusive(x.data_ptr(), out.data_ptr(), n, dt, 16, ws_ptr, ws_bytes, st) == 0
        torch.cuda.synchronize()
        assert lib.tcu_scan_debug_set_trace_buffer(trace.data_ptr()) == 0
        assert lib.tcu_scan_inclusive(x.data_ptr(), out.data_ptr(), n, dt, 16, ws_ptr, ws_bytes, st) == 0
        torch.cuda.synchronize()
        lib.tcu_scan_debug_set_trace_buffer(None)
        T = trace.cpu().numpy().reshape(tiles, 8).astype(np.int64)
        t0 = int(T[:, 0].min())
        entry = {"workload": label, "tiles": tiles, "us_since_claim_median": {}, "stored_rate_GBps": {}}
        for lo, hi in [(0, 32), (32, 148), (148, 740), (740, 1480), (tiles // 2, tiles // 2 + 1000), (tiles - 1000, tiles - 300)]:
            med = np.median((T[lo:hi] - T[lo:hi, :1]) / 1e3, axis=0)
            entry["us_since_claim_median"][f"tiles {lo}-{hi}"] = {nm: round(float(v), 2) for nm, v in zip(points, med)}
        stored = np.sort((T[:, 7] - t0) / 1e3)
        claimed = np.sort((T[:, 0] - t0) / 1e3)
        bpe = 5 if dt == 0 else 6
        entry["us_after_first_claim"] = {"first_stored": round(float(stored[0]), 1), "last_claimed": round(float(claimed[-1]), 1),
                                         "99pct_stored": round(float(stored[-tiles // 100]), 1), "last_stored": round(float(stored[-1]), 1)}
        for a, b in [(0.0, 0.05), (0.05, 0.95), (0.1, 0.5), (0.5, 0.9), (0.95, 1.0)]:
            ia, ib = int(a * tiles), min(int(b * tiles), tiles - 1)
            entry["stored_rate_GBps"][f"{a:.2f}-{b:.2f}"] = round((ib - ia) * 128 * 128 * bpe / (stored[ib] - stored[ia]) / 1e3)
        entry["whole_launch_GBps"] = round(n * bpe / float(stored[-1]) / 1e3)
        report.append(entry)
        del x, out, trace, ws
    print(json.dumps({"tile_trace": report}))


def run_sharded(args):
    """One array of 2^n_log2 int8 elements split into contiguous shards, one per rank (strong scaling): every step
    each rank takes the total of its shard, the totals are all-gathered (8 bytes per rank), each rank sums the totals
    before its own and scans its shard from that carry (paper Section 2.2 steps 2-4 with one segment per device).
    With one rank the exchange is a copy.  Prints one JSON line on rank 0."""
    import torch
    import torch.distributed as dist
    from paper_2411_17887_b200 import binding as B
    from paper_2411_17887_b200 import inputs, sharding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    n = 1 << args.n_log2
    lo, hi = sharding.shard_elements(n, world, rank)
    x_local = torch.from_numpy(inputs.int8_uniform((hi - lo,), -127, 127, 3 + 1000 * rank)).cuda()
    out_local = torch.empty(hi - lo, dtype=torch.int32, device="cuda")
    job = sharding.ShardedScan(hi - lo, "i8", s=S_TILE)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
    for _ in range(max(args.warmup, 3)):
        job.scan(x_local, out_local)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        job.scan(x_local, out_local)
    e1.record()
    barrier()
    ms_total = sharding.max_over_ranks(e0.elapsed_time(e1), "cuda")
    B.check(B.tcu_scan_device_status(job.ws_ptr, torch.cuda.current_stream().cuda_stream))
    if rank == 0:
        ms_step = ms_total / args.steps
        print(json.dumps({"metric": METRIC, "value": n * args.steps / (ms_total * 1e-3), "unit": "elements/s", "n_gpus": world,
                          "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
                          "scaling": "strong", "vs_baseline": None, "dtype": "i32", "data": "synthetic",
                          "config": {"workload": f"one array of 2^{args.n_log2} int8 sharded over {world} GPU(s): shard total, "
                                                 "all-gather of the totals, scan from the carry; 6 B/elt per rank (input read twice)"},
                          "gpu_launches": 4 * args.steps}))
    if world > 1:
        dist.destroy_process_group()


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2411_17887_b200 import binding as B      # raises if the CUDA library is missing
    from paper_2411_17887_b200 import inputs, sharding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    cfg = inputs.CONFIGS["C3"]
    x_host = inputs.int8_uniform((1 << args.n_log2,), -127, 127, cfg.index + 1000 * rank)   # each rank its own array
    n = x_host.size
    d_in = torch.from_numpy(x_host).cuda()
    d_out = torch.empty(n, dtype=torch.int32, device="cuda")
    ws_bytes = max(B.tcu_scan_workspace_bytes(4096, 65536, 0, S_TILE), B.tcu_scan_workspace_bytes(1, 1 << 28, 0, S_TILE),
                   B.tcu_scan_segmented_workspace_bytes(1 << 28, 0, S_TILE))
    if args.profile:
        args.no_extras = True
    ws = torch.empty(ws_bytes + 256, dtype=torch.uint8, device="cuda")
    ws_ptr = ws.data_ptr() + (-ws.data_ptr()) % 256
    stream = torch.cuda.current_stream().cuda_stream
    B.check(B.tcu_scan_workspace_init(ws_ptr, ws_bytes, stream))

    def step():
        B.check(B.tcu_scan_inclusive(d_in, d_out, n, B.TCU_I8_I32, S_TILE, ws_ptr, ws_bytes, stream))

    if args.profile:
        # the loop that is wrapped in ncu: optionally another input type, tile size or variant of the upper levels
        if args.profile_dtype == "f16":
            d_in = torch.from_numpy(inputs.f16_uniform((n,), -1.0, 1.0, cfg.index)).cuda()
            d_out = torch.empty(n, dtype=torch.float32, device="cuda")
        prof_dt = B.DTYPES[args.profile_dtype]

        def step():  # noqa: F811
            B.check(B.tcu_scan_ex(d_in, d_out, 1, n, prof_dt, args.profile_s, ws_ptr, ws_bytes, stream,
                                  upper_level_path=args.upper_level_path, down_sweep_path=args.down_sweep_path))

    # ---- device-resident timing
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    sampler = ClockSampler(local) if rank == 0 else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    ms_total = e0.elapsed_time(e1)
    B.check(B.tcu_scan_device_status(ws_ptr, stream))

    if args.profile:
        if rank == 0:
            ms_step = ms_total / args.steps
            bpe = 5 if args.profile_dtype == "i8" else 6
            print(json.dumps({"profile_run": True, "n": n, "dtype": args.profile_dtype, "s": args.profile_s,
                              "upper_level_path": args.upper_level_path, "down_sweep_path": args.down_sweep_path,
                              "ms_per_step": ms_step, "hbm_gb_per_s": bpe * n / (ms_step * 1e-3) / 1e9}))
        if sampler:
            sampler.stop()
        if world > 1:
            dist.destroy_process_group()
        return

    # every launch between its own events as well (outside the timed region above): median and best
    launch_med_us, launch_best_us = Timer(torch).each(step, min(args.steps, 50))

    # ---- end to end through the host-buffer entry point (pinned host memory, copies timed)
    h_in = torch.from_numpy(x_host).pin_memory()
    h_out = torch.empty(n, dtype=torch.int32).pin_memory()
    e2e_steps = max(1, min(args.steps, 5))

    def e2e_step():
        B.check(B.tcu_scan_host(h_in, h_out, n, B.TCU_I8_I32, S_TILE, 0, d_in, d_out, ws_ptr, ws_bytes, stream))
        torch.cuda.current_stream().synchronize()
    e2e_step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    barrier()
    e2e_s = time.perf_counter() - t0
    clocks = sampler.stop() if sampler else None

    # the slowest rank's times are the job's times
    ms_total = sharding.max_over_ranks(ms_total, "cuda")
    e2e_s = sharding.max_over_ranks(e2e_s, "cuda")

    if rank == 0:
        ms_step = ms_total / args.steps
        value = world * n * args.steps / (ms_total * 1e-3)
        peak, peak_kind = measured_peak()
        achieved = BYTES_PER_ELEM * n / (ms_step * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": "elements/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "i32", "data": "synthetic",
            "config": {"workload": f"C3: inclusive scan, n=2^{args.n_log2} int8 uniform[-127,127] -> int32, s=16, one array per GPU",
                       "n": n, "s": S_TILE, "l2": "working set 1.25 GiB per step, about 10x the L2, no flush needed",
                       "hbm_gb_per_s": achieved, "pct_of_8TBps": 100 * achieved / 8000.0,
                       "pct_of_measured_copy": 100 * achieved / peak,
                       "launch_us_median": launch_med_us, "launch_us_best": launch_best_us},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": n * (NCU_READ_RATIO * 1 + NCU_WRITE_RATIO * 4), "peak_kind": f"of {peak_kind}",
                         "traffic_method": "algorithmic bytes x the ratios of an ncu capture at n=2^26 (DRAM read / input "
                                           f"= {NCU_READ_RATIO}, SM-to-L2 write / output = {NCU_WRITE_RATIO}); DRAM write bytes of a "
                                           "capture are not scaled: part of the output is still in L2 when the kernel ends",
                         "kernel": "tcu_scan_kernel<int8,s=16,inclusive>", "algorithmic_bytes_per_launch": BYTES_PER_ELEM * n},
            "e2e": {"value": world * n * e2e_steps / e2e_s, "unit": "elements/s", "h2d_bytes_per_step": n,
                    "d2h_bytes_per_step": 4 * n, "steps": e2e_steps, "ms_per_step": 1e3 * e2e_s / e2e_steps},
            "gpu_launches": args.steps,
            "clocks": clocks,
        }
        if world == 1:
            # oracle on the host cores, and a full comparison of the GPU result against it
            step()
            torch.cuda.synchronize()
            got = d_out.cpu().numpy()
            from oracle import scan_oracle as so
            rate, y = oracle_leg(x_host, 5)
            line["parity"] = "bit-exact on all outputs" if np.array_equal(got, so.wrap_int32(y)) else "MISMATCH"
            del got, y
            cores = os.cpu_count() or 1
            line["cpu_baseline"] = {"value": rate, "unit": "elements/s", "cores": 1, "kind": "oracle",
                                    "sample": f"whole 2^{args.n_log2}-element input, best of 5 sequential passes",
                                    "host_cores": cores, "cpu_model": cpu_model(),
                                    "all_cores": {"value": oracle_all_cores(x_host, cores), "unit": "elements/s", "threads": cores,
                                                  "method": "the oracle's C loop on one chunk per thread, two passes "
                                                            "(chunk totals, then every chunk rescanned from its carry)"}}
            if not args.no_extras:
                g = torch.Generator(device="cuda").manual_seed(inputs.BASE_SEED)
                xf = (torch.rand(1 << 28, device="cuda", generator=g) * 2 - 1).half()

                def frac(r, nbytes=None):
                    r["frac_of_peak"] = round(r["GBps"] / peak, 3)
                    return r
                # the second bandwidth target: fp16 -> fp32 at the headline size (kept in `config` so that it is
                # part of the parsed line, not of the long tail)
                r, _ = time_extra(B, torch, xf, 1, 1 << 28, 1, 16, ws_ptr, ws_bytes)
                line["config"]["fp16_n2p28_s16"] = dict(frac(r), pct_of_8TBps=round(100 * r["GBps"] / 8000.0, 1),
                                                        elements_per_s=(1 << 28) / (r["us"] * 1e-6))
                extra = {}
                extra["C2_n2p24_f16_incl"] = frac(time_extra(B, torch, xf, 1, 1 << 24, 1, 16, ws_ptr, ws_bytes, reps=50)[0])
                extra["C2_n2p24_f16_excl"] = frac(time_extra(B, torch, xf, 1, 1 << 24, 1, 16, ws_ptr, ws_bytes, reps=50, exclusive=1)[0])
                for s in (16, 64, 128):
                    r, st = time_extra(B, torch, xf.abs(), 1, 1 << 26, 1, s, ws_ptr, ws_bytes, reps=20)
                    extra[f"C5_n2p26_f16_s{s}"] = dict(frac(r), levels_used=st["levels_used"], depth_bound=st["depth_bound"],
                                                       sxs_products=st["sxs_products"], mma=st["mma_instructions"])
                xb = torch.randn(1 << 28, device="cuda", generator=g).bfloat16()
                extra["C4_4096x65536_bf16"] = frac(time_extra(B, torch, xb, 4096, 65536, 2, 16, ws_ptr, ws_bytes)[0])
                del xb
                extra["C1_n2p16_i8"] = time_extra(B, torch, d_in, 1, 1 << 16, 0, 16, ws_ptr, ws_bytes, reps=200)[0]
                # the same 64 Ki-element scan replayed from a CUDA graph of 20 launches: the host's 3-6 us per call
                # (ctypes, tensor-map encoding, launch) are out of the loop
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph):
                    cap = torch.cuda.current_stream().cuda_stream
                    for _ in range(20):
                        B.check(B.tcu_scan_inclusive(d_in, d_out, 1 << 16, 0, 16, ws_ptr, ws_bytes, cap))
                for _ in range(3):
                    graph.replay()
                torch.cuda.synchronize()
                ms_g = Timer(torch).loop(graph.replay, 25) / 20
                extra["C1_n2p16_i8_cuda_graph"] = {"us": round(1e3 * ms_g, 2), "GBps": round(5 * (1 << 16) / (ms_g * 1e-3) / 1e9, 1)}
                B.check(B.tcu_scan_device_status(ws_ptr, stream))
                del graph
                # plain widening copies with the scans' read / write mixes (1 : 4 and 2 : 4), no dependence between
                # elements: what the memory system gives that mix when nothing has to be carried along
                d_out_f = d_out.view(torch.float32)
                for key, src, dst, dtc, bpe in (("widening_copy_i8_i32_n2p28", d_in, d_out, 0, 5),
                                                ("widening_copy_f16_f32_n2p28", xf, d_out_f, 1, 6)):
                    def widen():
                        B.check(B.tcu_widen_copy(src, dst, n, dtc, stream))
                    for _ in range(3):
                        widen()
                    torch.cuda.synchronize()
                    ms_w = Timer(torch).loop(widen, 20)
                    extra[key] = frac({"us": round(1e3 * ms_w, 2), "GBps": round(bpe * n / (ms_w * 1e-3) / 1e9, 1)})
                line["config"]["scan_time_over_widening_copy_time"] = {
                    "i8": round(1e3 * ms_step / extra["widening_copy_i8_i32_n2p28"]["us"], 4),
                    "f16": round(line["config"]["fp16_n2p28_s16"]["us"] / extra["widening_copy_f16_f32_n2p28"]["us"], 4)}
                ms_t = Timer(torch).loop(lambda: d_out.copy_(d_in), 10)      # the framework's own converting copy, same mix
                extra["torch_copy_i8_to_i32_n2p28"] = frac({"us": round(1e3 * ms_t, 2), "GBps": round(5 * n / (ms_t * 1e-3) / 1e9, 1)})
                # the same scans in the two-sweep structure (reduce, scan the totals, scan with every carry known)
                extra["C3_two_sweep"] = frac(time_extra(B, torch, d_in, 1, n, 0, 16, ws_ptr, ws_bytes, variant=1)[0])
                extra["f16_n2p28_two_sweep"] = frac(time_extra(B, torch, xf, 1, 1 << 28, 1, 16, ws_ptr, ws_bytes, variant=1)[0])
                # ... with the scan of the tile totals sent through the tensor-core scan again (narrow terms, one inner scan each)
                extra["C3_two_sweep_totals_by_scan"] = frac(time_extra(B, torch, d_in, 1, n, 0, 16, ws_ptr, ws_bytes, variant=1,
                                                                       upper_level_path=1)[0])
                extra["f16_n2p28_two_sweep_totals_by_scan"] = frac(time_extra(B, torch, xf, 1, 1 << 28, 1, 16, ws_ptr, ws_bytes,
                                                                              variant=1, upper_level_path=1)[0])
                # upper level (scan over the 128 row totals) as a tcgen05 product on exact narrow terms
                # (path 2: the chunk level inside a row as a product as well)
                for path in (1, 2):
                    extra[f"C3_upper_level_path{path}"] = frac(time_extra(B, torch, d_in, 1, n, 0, 16, ws_ptr, ws_bytes, upper_level_path=path)[0])
                    extra[f"f16_n2p28_upper_level_path{path}"] = frac(time_extra(B, torch, xf, 1, 1 << 28, 1, 16, ws_ptr, ws_bytes, upper_level_path=path)[0])
                # fp16, s = 128: carries added by a tensor-core product (the paper's B_s step) instead of vector adds
                for path in (0, 1):
                    extra[f"f16_n2p28_s128_down_sweep_path{path}"] = frac(
                        time_extra(B, torch, xf, 1, 1 << 28, 1, 128, ws_ptr, ws_bytes, down_sweep_path=path)[0])
                # the same for s = 16: one carry per chunk, from the chunk-level product (upper_level_path = 2)
                extra["f16_n2p28_s16_upper_level_path2_down_sweep_path1"] = frac(
                    time_extra(B, torch, xf, 1, 1 << 28, 1, 16, ws_ptr, ws_bytes, upper_level_path=2, down_sweep_path=1)[0])
                del xf
                # segmented scan of the headline array: random cut points, mean segment length 2^10, 2^14, 2^18
                for logm in (10, 14, 18):
                    cuts = torch.randint(0, n, (n >> logm,), device="cuda", generator=g, dtype=torch.int64)
                    off = torch.cat([torch.zeros(1, dtype=torch.int64, device="cuda"), cuts.sort().values,
                                     torch.full((1,), n, dtype=torch.int64, device="cuda")])
                    seg_out = torch.empty(n, dtype=torch.int32, device="cuda")

                    def seg_call():
                        B.check(B.tcu_scan_segmented(d_in, seg_out, n, off, off.numel() - 1, 0, 16, 0, ws_ptr, ws_bytes, stream))
                    for _ in range(2):
                        seg_call()
                    torch.cuda.synchronize()
                    ms_seg = Timer(torch).loop(seg_call, 10)
                    extra[f"segmented_n2p28_i8_mean2p{logm}"] = frac({"us": round(1e3 * ms_seg, 1),
                                                                      "GBps": round(5 * n / (ms_seg * 1e-3) / 1e9, 1)})
                    del seg_out, off, cuts
                # application: radix sort of 2^24 keys by 32 one-bit splits, each an exclusive scan of int8 flags
                ns = 1 << 24
                keys = torch.randint(0, 1 << 31, (ns,), device="cuda", dtype=torch.int32, generator=g)
                sorted_out = torch.empty_like(keys)
                tmp_bytes = B.tcu_sort_tmp_bytes(ns)
                tmp = torch.empty(tmp_bytes + 256, dtype=torch.uint8, device="cuda")
                tmp_ptr = tmp.data_ptr() + (-tmp.data_ptr()) % 256

                def sort_call():
                    B.check(B.tcu_sort_u32(keys, sorted_out, ns, tmp_ptr, tmp_bytes, ws_ptr, ws_bytes, stream))
                for _ in range(2):
                    sort_call()
                torch.cuda.synchronize()
                ms_sort = Timer(torch).loop(sort_call, 3)
                extra["radix_sort_2p24_u32"] = {"us": round(1e3 * ms_sort, 1), "keys_per_s": ns / (ms_sort * 1e-3),
                                                "sorted": bool((sorted_out[1:] >= sorted_out[:-1]).all())}
                line["extra"] = extra
            if args.sweep_ctas:
                sms = torch.cuda.get_device_properties(local).multi_processor_count
                sweep = []
                for pcount in [1, 2, 4, 8, 16, 32, 64, 128, sms]:
                    def pstep():
                        B.check(B.tcu_scan_ex(d_in, d_out, 1, n, B.TCU_I8_I32, S_TILE, ws_ptr, ws_bytes, stream, max_ctas=pcount))
                    pstep()
                    torch.cuda.synchronize()
                    sweep.append({"p": pcount, "ms": Timer(torch).loop(pstep, 2 if pcount < 8 else 5)})
                t1 = sweep[0]["ms"]
                for e in sweep:
                    e["speedup_vs_p1"] = t1 / e["ms"]
                    e["efficiency"] = t1 / e["ms"] / e["p"]
                line["p_tcu_sweep"] = sweep
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the timings of the other configurations")
    ap.add_argument("--profile-dtype", default="i8", choices=["i8", "f16"], help="input type of the --profile loop")
    ap.add_argument("--profile-s", type=int, default=16, help="tile size s of the --profile loop")
    ap.add_argument("--upper-level-path", type=int, default=0, choices=[0, 1, 2],
                    help="--profile loop: 1 scans the row totals with a tensor-core product on exact narrow terms, "
                         "2 the chunk totals of every row as well")
    ap.add_argument("--down-sweep-path", type=int, default=0, choices=[0, 1],
                    help="--profile loop: 1 adds the row carries with a tensor-core product (fp16 input, s = 128)")
    ap.add_argument("--sweep-ctas", action="store_true",
                    help="also time the headline scan on p = 1, 2, 4, ... persistent CTAs (one per SM) and report time vs p")
    ap.add_argument("--n-log2", type=int, default=28, help="log2 of the array length (28 = the headline workload)")
    ap.add_argument("--profile", action="store_true",
                    help="device-resident loop only (no end-to-end leg, no oracle): the command to wrap in ncu")
    ap.add_argument("--sharded", action="store_true",
                    help="one array split over the ranks (strong scaling) instead of one array per rank")
    ap.add_argument("--wait-counters", action="store_true",
                    help="debug build of the library: where each role of the kernel waits, at the headline size")
    ap.add_argument("--tile-trace", action="store_true",
                    help="debug build: eight time stamps per tile; the life of a tile and the completion rate over a launch")
    ap.add_argument("--fixed-cost", action="store_true",
                    help="break the time of small launches (C1, C2, C5) into phases with the kernel's time stamps")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.fixed_cost:
        fixed_cost(args)
    elif args.wait_counters:
        wait_counters(args)
    elif args.tile_trace:
        tile_trace(args)
    elif args.sharded:
        run_sharded(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
