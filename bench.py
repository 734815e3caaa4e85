#!/usr/bin/env python
"""Benchmark of the tensor-core-unit scan library on B200.

    python bench.py --gpus N --steps K --warmup W            # this library (CUDA, through the C ABI)
    python bench.py --impl reference --steps K --warmup W    # the CPU oracle on the host cores

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
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "elements/sec and achieved HBM GB/s (% of peak) for n=2^28 scan on 1 B200"
N_ELEMS = 1 << 28
S_TILE = 16
BYTES_PER_ELEM = 5          # int8 read + int32 written
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the main kernel on 2^26 elements, from the
# ncu capture summarised in profiles/ (traffic grows in proportion to n: one read and one write per element)
NCU_TRAFFIC_BYTES_PER_2P26 = 278.2e6   # profiles/tcu_scan_kernel_int8_s16_n2p26_ncu_full.md; scaled by n / 2^26 below


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


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
        "config": {"workload": "C3: inclusive scan, n=2^28 int8 uniform[-127,127] -> int32, s=16"},
        "cpu_baseline": {"value": value, "unit": "elements/s", "cores": 1, "kind": "oracle",
                         "sample": f"whole 2^28-element input per step, {args.steps} steps"},
        "e2e": {"value": value, "unit": "elements/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def time_extra(B, torch, name, x, rows, cols, dt, s, exclusive, ws_ptr, ws_bytes, reps=10, two_sweep=False):
    out = torch.empty(rows * cols, dtype=torch.int32 if dt == 0 else torch.float32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream

    def call():
        if two_sweep:
            B.check(B.tcu_scan_inclusive_twosweep(x, out, cols, dt, s, ws_ptr, ws_bytes, stream))
        elif rows == 1:
            fn = B.tcu_scan_exclusive if exclusive else B.tcu_scan_inclusive
            B.check(fn(x, out, cols, dt, s, ws_ptr, ws_bytes, stream))
        else:
            B.check(B.tcu_scan_batched(x, out, rows, cols, dt, s, int(exclusive), ws_ptr, ws_bytes, stream))
    for _ in range(3):
        call()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        call()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    nbytes = rows * cols * ((1 if dt == 0 else 2) + 4)
    del out
    st = B.tcu_scan_last_stats()
    return {"workload": name, "ms": ms, "elements_per_s": rows * cols / (ms * 1e-3), "GB_per_s": nbytes / (ms * 1e-3) / 1e9,
            "levels_used": st["levels_used"], "depth_bound_2floor_log_s_n": st["depth_bound"],
            "sxs_products": st["sxs_products"], "n_over_s2": rows * cols // (s * s), "mma_instructions": st["mma_instructions"]}


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2411_17887_b200 import binding as B      # raises if the CUDA library is missing
    from paper_2411_17887_b200 import inputs

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
    ws_bytes = B.tcu_scan_workspace_bytes(4096, 1 << 28, 0, S_TILE)
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
        B.check(B.tcu_scan_set_upper_level_path(args.upper_level_path))
        B.check(B.tcu_scan_set_down_sweep_path(args.down_sweep_path))
        if args.profile_dtype == "f16":
            d_in = torch.from_numpy(inputs.f16_uniform((n,), -1.0, 1.0, cfg.index)).cuda()
            d_out = torch.empty(n, dtype=torch.float32, device="cuda")
        prof_dt = B.DTYPES[args.profile_dtype]

        def step():  # noqa: F811
            B.check(B.tcu_scan_inclusive(d_in, d_out, n, prof_dt, args.profile_s, ws_ptr, ws_bytes, stream))

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

    times = torch.tensor([ms_total, e2e_s], dtype=torch.float64, device="cuda")
    if world > 1:
        dist.all_reduce(times, op=dist.ReduceOp.MAX)
    ms_total, e2e_s = float(times[0]), float(times[1])

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
                       "pct_of_measured_copy": 100 * achieved / peak},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": NCU_TRAFFIC_BYTES_PER_2P26 * n / (1 << 26), "peak_kind": f"of {peak_kind}",
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
            line["cpu_baseline"] = {"value": rate, "unit": "elements/s", "cores": 1, "kind": "oracle",
                                    "sample": f"whole 2^{args.n_log2}-element input, best of 5 sequential passes",
                                    "host_cores": os.cpu_count()}
            line["parity"] = "bit-exact on all outputs" if np.array_equal(got, so.wrap_int32(y)) else "MISMATCH"
            del got, y
            if not args.no_extras:
                extras = []
                g = torch.Generator(device="cuda").manual_seed(inputs.BASE_SEED)
                xf = (torch.rand(1 << 28, device="cuda", generator=g) * 2 - 1).half()
                extras.append(time_extra(B, torch, "n=2^28 fp16 uniform[-1,1) -> fp32, s=16", xf, 1, 1 << 28, 1, 16, False, ws_ptr, ws_bytes))
                extras.append(time_extra(B, torch, "C2: n=2^24 fp16, s=16, inclusive", xf, 1, 1 << 24, 1, 16, False, ws_ptr, ws_bytes))
                extras.append(time_extra(B, torch, "C2: n=2^24 fp16, s=16, exclusive", xf, 1, 1 << 24, 1, 16, True, ws_ptr, ws_bytes))
                for s in (16, 64, 128):
                    extras.append(time_extra(B, torch, f"C5: n=2^26 fp16, s={s}", xf.abs(), 1, 1 << 26, 1, s, False, ws_ptr, ws_bytes))
                xb = torch.randn(1 << 28, device="cuda", generator=g).bfloat16()
                extras.append(time_extra(B, torch, "C4: 4096 x 65536 bf16 normal -> fp32, s=16, row-wise", xb, 4096, 65536, 2, 16, False, ws_ptr, ws_bytes))
                extras.append(time_extra(B, torch, "C1: n=2^16 int8, s=16", d_in, 1, 1 << 16, 0, 16, False, ws_ptr, ws_bytes))
                extras.append(time_extra(B, torch, "C3 in the two-sweep structure (reduce, scan totals, scan): n=2^28 int8, s=16",
                                         d_in, 1, n, 0, 16, False, ws_ptr, ws_bytes, two_sweep=True))
                extras.append(time_extra(B, torch, "fp16 n=2^28 in the two-sweep structure, s=16",
                                         xf, 1, 1 << 28, 1, 16, False, ws_ptr, ws_bytes, two_sweep=True))
                # the same scan with the row-total level on tensor cores (8-bit limbs) instead of warp shuffles
                B.check(B.tcu_scan_set_upper_level_path(1))
                extras.append(time_extra(B, torch, "C3 with the scan over row totals as a tcgen05 product on 8-bit limbs (upper_level_path = 1)",
                                         d_in, 1, n, 0, 16, False, ws_ptr, ws_bytes))
                B.check(B.tcu_scan_set_upper_level_path(0))
                # fp16, s = 128: carries added by a tensor-core product (the paper's B_s step) instead of vector adds
                for path in (0, 1):
                    B.check(B.tcu_scan_set_down_sweep_path(path))
                    extras.append(time_extra(B, torch, f"fp16 n=2^28, s=128, down_sweep_path = {path}", xf, 1, 1 << 28, 1, 128,
                                             False, ws_ptr, ws_bytes))
                B.check(B.tcu_scan_set_down_sweep_path(0))
                # application: radix sort of 2^24 keys by 32 one-bit splits, each an exclusive scan of int8 flags
                ns = 1 << 24
                keys = torch.randint(0, 1 << 31, (ns,), device="cuda", dtype=torch.int32, generator=g)
                sorted_out = torch.empty_like(keys)
                tmp_bytes = B.tcu_sort_tmp_bytes(ns)
                tmp = torch.empty(tmp_bytes + 256, dtype=torch.uint8, device="cuda")
                tmp_ptr = tmp.data_ptr() + (-tmp.data_ptr()) % 256
                for _ in range(2):
                    B.check(B.tcu_sort_u32(keys, sorted_out, ns, tmp_ptr, tmp_bytes, ws_ptr, ws_bytes, stream))
                torch.cuda.synchronize()
                s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                s0.record()
                for _ in range(3):
                    B.check(B.tcu_sort_u32(keys, sorted_out, ns, tmp_ptr, tmp_bytes, ws_ptr, ws_bytes, stream))
                s1.record()
                torch.cuda.synchronize()
                ms_sort = s0.elapsed_time(s1) / 3
                ok = bool((sorted_out[1:] >= sorted_out[:-1]).all())
                extras.append({"workload": "radix sort of 2^24 uint32 keys by 32 one-bit splits (32 exclusive scans)",
                               "ms": ms_sort, "keys_per_s": ns / (ms_sort * 1e-3), "sorted": ok})
                line["extra"] = extras
            if args.sweep_ctas:
                sms = torch.cuda.get_device_properties(local).multi_processor_count
                sweep = []
                ps = [1, 2, 4, 8, 16, 32, 64, 128, sms]
                for pcount in ps:
                    B.check(B.tcu_scan_set_max_ctas(pcount))
                    reps = 2 if pcount < 8 else 5
                    step()
                    torch.cuda.synchronize()
                    a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a0.record()
                    for _ in range(reps):
                        step()
                    a1.record()
                    torch.cuda.synchronize()
                    sweep.append({"p": pcount, "ms": a0.elapsed_time(a1) / reps})
                B.check(B.tcu_scan_set_max_ctas(0))
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
    ap.add_argument("--upper-level-path", type=int, default=0, choices=[0, 1],
                    help="1: scan the row totals with a tensor-core product on 8-bit limbs (int8 input)")
    ap.add_argument("--down-sweep-path", type=int, default=0, choices=[0, 1],
                    help="1: add the row carries with a tensor-core product (fp16 input, s = 128)")
    ap.add_argument("--sweep-ctas", action="store_true",
                    help="also time the headline scan on p = 1, 2, 4, ... persistent CTAs (one per SM) and report time vs p")
    ap.add_argument("--n-log2", type=int, default=28, help="log2 of the array length (28 = the headline workload)")
    ap.add_argument("--profile", action="store_true",
                    help="device-resident loop only (no end-to-end leg, no oracle): the command to wrap in ncu")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
