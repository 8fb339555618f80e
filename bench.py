#!/usr/bin/env python
"""Benchmark of the fault-injected GEMM hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Workload at one GPU: config 2 (BF16 4096^3, A,B ~ N(0,1)/64, operand single-bit faults,
BoundCheck detection + correction). One step = one fault-injected GEMM through the library
(site table decode, operand flip in the staged tile, tcgen05 main loop, fused check, flags),
each step taking the next trial of the config's table as its site. L2 is flushed between steps.

Reported on one JSON line: GEMM TFLOP/s with inputs resident in HBM (`value`), the same through
pinned host buffers with the copies inside the timed region (`e2e`), the same kernel with injection
and detection disabled, the campaign's trials/s, the roofline fraction of the GEMM kernel, and the
CPU oracle timed on a bounded sample of the same workload (`cpu_baseline`).

With N > 1 (torchrun, one rank per GPU) every rank runs the same workload on its own share of the
trial table; there is no data-path collective (weak scaling); the time is the max over ranks.

`--impl reference` times the CPU oracle instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

WORKLOAD = "c2"      # the configuration the headline metric is quoted on; --config times another one
METRIC = "fault-injected GEMM TFLOP/s"
DTYPE_NAMES = {0: "fp16", 1: "bf16", 2: "tf32"}
WORKLOAD_TEXT = {
    "c1": "c1: FP16 GEMM M=N=K=256, A,B ~ N(0,1)/16; per step one single-bit output-element fault from the seeded "
          "64-trial table; BoundCheck detection",
    "c2": "c2: BF16 GEMM M=N=K=4096, A,B ~ N(0,1)/64, FP32 accumulate and output; per step one single-bit operand "
          "fault (A or B, bit 0-15) from the seeded 1024-trial table; BoundCheck detection+correction",
    "c3a": "c3a: FP16 GEMM M=16384 N=4096 K=1024, A ~ N(0,1), B ~ N(0,0.02); per step one single-bit output-element "
           "fault from the seeded 4096-trial table; BoundCheck detection",
    "c3b": "c3b: FP16 GEMM M=16384 N=1024 K=4096, A ~ GELU(N(0,1)), B ~ N(0,0.02); per step one single-bit "
           "output-element fault from the seeded 4096-trial table; BoundCheck detection",
    "c4": "c4: TF32 GEMM M=N=K=8192, A,B ~ U(-1,1); per step one accumulator fault (two adjacent bits after a "
          "uniformly chosen k-step boundary) from the seeded 2048-trial table; BoundCheck detection",
    "c5": "c5: FP16 GEMM M=802816 N=64 K=576 (im2col of a 3x3 conv), A ~ ReLU(N(0,1)), B ~ N(0,sqrt(2/576)); per step "
          "one single-bit fault from the seeded 100000-trial table (operand / accumulator / output mix); BoundCheck "
          "detection+correction",
}
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the GEMM kernel, from the ncu capture summarised
# under profiles/ (the capture names the kernel source it was taken on); None for a config without a capture of the
# present kernel
KERNEL_TRAFFIC_BYTES = {"c2": 151.2e6, "c3a": 266.6e6}
FALLBACK_PEAKS = {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0}


def env_int(name, default):
    try:
        return int(os.environ.get(name, default))
    except ValueError:
        return default


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            with open(path) as f:
                d = json.load(f)
            return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """nvidia-smi sampling of SM clock and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) != 7:
                continue
            try:
                sm.append(float(parts[0])); smax.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        # the samples under load are the ones drawing the most power
        cut = 0.6 * max(power)
        loaded = [c for c, p in zip(sm, power) if p >= cut] or sm
        return {"sm_mhz": statistics.median(loaded), "sm_max_mhz": max(smax), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power)}


def oracle_sample_run(w, rows, n_sites=1):
    """Fault-injected oracle GEMM on the first `rows` rows of A (a row panel of the workload)."""
    import oracle as orc
    A = np.ascontiguousarray(w.A[:rows])
    sites = w.sites[:n_sites].copy()
    sites["row"] = sites["row"] % rows
    t0 = time.perf_counter()
    orc.gemm(w.dtype, A, w.Bt, sites, w.detect_mode)
    return time.perf_counter() - t0


def cpu_baseline(w, limit_s=12.0):
    import oracle as orc
    orc.build()
    t_small, t_probe = oracle_sample_run(w, 32), oracle_sample_run(w, 160)
    per_row = max((t_probe - t_small) / 128.0, 1e-6)          # the fixed part (widening Bt) is not per-row work
    rows = int(min(w.M, max(160, (limit_s - t_small) / per_row)))
    rows = max(32, (rows // 32) * 32)
    t = oracle_sample_run(w, rows)
    flops = 2.0 * rows * w.N * w.K
    return {"value": flops / t / 1e12, "unit": "TFLOP/s", "cores": orc.num_threads(), "kind": "oracle",
            "sample": f"rows 0..{rows - 1} of A ({rows}x{w.N}x{w.K} of the {w.M}x{w.N}x{w.K} GEMM), one site of the "
                      f"trial table, the config's check, {t:.2f} s"}


def quick_config(name, mpg, synth, torch, dev, flush, peaks, steps=40, out16=False):
    """One config in brief, for the `all_configs` key: us per injected GEMM (L2 flushed, per-step events), its rate and
    roofline fraction, the time ratio against the same kernel without injection and check (alternating launches), and
    the campaign's trials/s. out16: the GEMM writes an FP16 result (mpgemmfi_gemm_out16) instead of FP32."""
    w = synth.make_workload(name)
    M, N, K, dtype, mode = w.M, w.N, w.K, w.dtype, w.detect_mode
    view = np.int32 if dtype == synth.DTYPE_TF32 else np.int16
    A = torch.from_numpy(w.A.view(view)).to(dev)
    Bt = torch.from_numpy(w.Bt.view(view)).to(dev)
    host_sites = torch.from_numpy(w.sites.view(np.int32).reshape(-1, 8).copy()).pin_memory()
    sites = host_sites.to(dev)
    C = torch.empty((M, N), dtype=torch.float16 if out16 else torch.float32, device=dev)
    flags = torch.empty(mpg.mpgemmfi_flags_bytes(M, N, 1) // 4, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream(dev)
    sh = stream.cuda_stream
    n = len(w.sites)

    def step(i, kind):
        # kind: "host" = the step's site handed over in host memory (it travels in the launch parameters),
        # "device" = the same site read from the table in device memory, "off" = no injection, no check
        table = host_sites if kind == "host" else sites
        sp, nf, md, fl = (table.data_ptr() + 32 * (i % n), 1, mode, flags.data_ptr()) if kind != "off" else (None, 0, 0, None)
        if out16:
            rc = mpg.mpgemmfi_gemm_out16(dtype, M, N, K, A.data_ptr(), Bt.data_ptr(), None, mpg.OUT_FP16, C.data_ptr(), sp, nf,
                                         md, fl, sh)
        else:
            rc = mpg.mpgemmfi_gemm(dtype, M, N, K, A.data_ptr(), Bt.data_ptr(), C.data_ptr(), sp, nf, md, fl, sh)
        if rc != 0:
            raise mpg.MpgemmfiError(rc, "mpgemmfi_gemm")

    kinds = ("host", "device", "off")
    for i in range(3):
        for kind in kinds:
            flush.zero_(); step(i, kind)
    torch.cuda.synchronize(dev)
    ev = []
    for i in range(steps):
        for kind in kinds[i % 3:] + kinds[:i % 3]:       # every kind follows every other kind equally often
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream); step(i, kind); e1.record(stream)
            ev.append((kind, e0, e1))
    torch.cuda.synchronize(dev)
    t_on, t_dev, t_off = (statistics.median(e0.elapsed_time(e1) for k, e0, e1 in ev if k == kind) * 1e-3 for kind in kinds)
    if int(flags[0].item()) & mpg.STATUS_WAIT_LIMIT:
        raise SystemExit(f"device wait limit hit on {name}")
    flops = 2.0 * M * N * K
    out = {"us_per_gemm": t_on * 1e6, "us_per_gemm_device_table": t_dev * 1e6, "tflops": flops / t_on / 1e12,
           "injected_over_plain_time": t_on / t_off,
           "dtype": DTYPE_NAMES[dtype], "output": "fp16" if out16 else "fp32", "steps": steps}
    es = A.element_size()
    min_bytes = (M * K + N * K) * es + M * N * C.element_size() + M * ((N + 31) // 32) * 4
    if name == "c1":
        out.update({"bound": "latency", "frac": None})          # one wave of four tiles: launch and pipeline fill
    elif name == "c5":
        gbs = min_bytes / t_on / 1e9
        out.update({"bound": "hbm", "achieved_gbs": gbs, "frac": gbs / peaks["hbm_gbs"]})
    else:
        peak = peaks["bf16_tflops"] * (0.5 if dtype == synth.DTYPE_TF32 else 1.0)
        out.update({"bound": "tensor", "frac": out["tflops"] / peak})
    if not out16:
        rec = torch.empty((n, 12), dtype=torch.int32, device=dev)
        Cc = C
        ws = torch.empty(mpg.mpgemmfi_campaign_workspace_bytes(dtype, M, N, K, n), dtype=torch.uint8, device=dev)
        ts = []
        for i in range(5):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            rc = mpg.mpgemmfi_campaign(dtype, M, N, K, A.data_ptr(), Bt.data_ptr(), Cc.data_ptr(), sites.data_ptr(), n, mode,
                                       rec.data_ptr(), ws.data_ptr(), ws.numel(), sh)
            e1.record(stream)
            if rc != 0:
                raise mpg.MpgemmfiError(rc, "mpgemmfi_campaign")
            ts.append((e0, e1))
        torch.cuda.synchronize(dev)
        t_c = statistics.median(e0.elapsed_time(e1) for e0, e1 in ts[2:]) * 1e-3
        out.update({"campaign_trials": n, "campaign_ms": t_c * 1e3, "campaign_trials_per_s": n / t_c})
    return out


def run_reference(args):
    """The CPU oracle as the reference arm: each step is a bounded row-panel sample of the workload."""
    import oracle as orc
    import synth
    rank = env_int("RANK", 0)
    if rank != 0:
        return
    orc.build()
    w = synth.make_workload(WORKLOAD)
    t_probe = oracle_sample_run(w, 32)
    total_steps = max(1, args.steps + args.warmup)
    rows = int(min(w.M, max(32, 32 * (60.0 / total_steps) / max(t_probe, 1e-3))))
    rows = max(32, (rows // 32) * 32)
    for _ in range(args.warmup):
        oracle_sample_run(w, rows)
    t = 0.0
    for _ in range(args.steps):
        t += oracle_sample_run(w, rows)
    flops = 2.0 * rows * w.N * w.K * args.steps
    value = flops / t / 1e12
    sample = f"per step: rows 0..{rows - 1} of A ({rows}x{w.N}x{w.K}) with one operand site, BoundCheck+correction"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD_TEXT[WORKLOAD], "sample": sample},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": orc.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing (profiling runs)")
    ap.add_argument("--config", default=WORKLOAD, help="workload to time (c1, c2, c3a, c3b, c4, c5); default c2")
    ap.add_argument("--no-all-configs", action="store_true", help="skip the brief pass over the other workloads")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "b200" else args.warmup

    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist

    import paper_2311_05782_b200 as mpg
    import synth
    from paper_2311_05782_b200.sharding import campaign_sharded, shard_range, reduce_max, reduce_sum

    world = env_int("WORLD_SIZE", 1)
    rank = env_int("RANK", 0)
    local_rank = env_int("LOCAL_RANK", 0)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    if env_int("MPGEMMFI_BENCH_ONE_DEVICE", 0):
        local_rank = 0      # rehearsal of the N > 1 path where there is one GPU: every rank on device 0, gloo instead of nccl
    torch.cuda.set_device(local_rank)
    if world > 1:
        if env_int("MPGEMMFI_BENCH_ONE_DEVICE", 0):
            dist.init_process_group("gloo")
        else:
            dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    mpg.load_library()

    w = synth.make_workload(args.config)
    M, N, K, dtype, mode = w.M, w.N, w.K, w.dtype, w.detect_mode
    view = np.int32 if dtype == synth.DTYPE_TF32 else np.int16
    lo, hi = shard_range(len(w.sites), rank, world)          # this rank's share of the trial table
    my_sites = w.sites[lo:hi]
    dev = torch.device("cuda", local_rank)
    A = torch.from_numpy(w.A.view(view)).to(dev)
    Bt = torch.from_numpy(w.Bt.view(view)).to(dev)
    sites_dev = torch.from_numpy(my_sites.view(np.int32).reshape(-1, 8)).to(dev)
    C = torch.empty((M, N), dtype=torch.float32, device=dev)
    flags = torch.empty(mpg.mpgemmfi_flags_bytes(M, N, 1) // 4, dtype=torch.int32, device=dev)
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)     # larger than the 126 MB L2
    stream = torch.cuda.current_stream(dev)
    sh = stream.cuda_stream
    n_my = len(my_sites)
    flops = 2.0 * M * N * K

    # the step's one site is handed over in (pinned) host memory: it travels in the launch parameters
    sites_host = torch.from_numpy(my_sites.view(np.int32).reshape(-1, 8).copy()).pin_memory()

    def gemm_step(i, inject=True):
        if inject:
            sp = sites_host.data_ptr() + 32 * (i % n_my)
            rc = mpg.mpgemmfi_gemm(dtype, M, N, K, A.data_ptr(), Bt.data_ptr(), C.data_ptr(), sp, 1, mode,
                                   flags.data_ptr(), sh)
        else:
            rc = mpg.mpgemmfi_gemm(dtype, M, N, K, A.data_ptr(), Bt.data_ptr(), C.data_ptr(), None, 0, 0, None, sh)
        if rc != 0:
            raise mpg.MpgemmfiError(rc, "mpgemmfi_gemm")

    def timed(fn, steps, warmup, sampler=None):
        """Sum of per-step CUDA-event times on the launching stream, L2 flushed before every step."""
        for i in range(warmup):
            flush.zero_()
            fn(i)
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)
        if sampler:
            sampler.start()
        t_region0 = time.perf_counter()
        starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        stops = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        for i in range(steps):
            flush.zero_()
            starts[i].record(stream)
            fn(warmup + i)
            stops[i].record(stream)
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)
        ms = sum(s.elapsed_time(e) for s, e in zip(starts, stops))
        clocks = None
        if sampler:
            # nvidia-smi needs a few hundred ms to deliver samples: when the timed region was shorter, keep the
            # same load running (untimed, identical steps) until the sampler has seen about 0.4 s of it
            t_end = time.perf_counter() + max(0.0, 0.4 - (time.perf_counter() - t_region0))
            i = 0
            while time.perf_counter() < t_end:
                flush.zero_()
                fn(warmup + steps + i)
                i += 1
                if i % 32 == 0:
                    torch.cuda.synchronize(dev)
            torch.cuda.synchronize(dev)
            clocks = sampler.stop()
            clocks["untimed_tail_steps"] = i
        return ms, clocks

    # ---- main arm: injection + detection + correction, inputs resident in HBM
    sampler = ClockSampler(local_rank) if rank == 0 else None
    ms_inj, clocks = timed(lambda i: gemm_step(i, True), args.steps, args.warmup, sampler)
    hdr = flags[:16].cpu().numpy().view(np.uint32)
    if hdr[0] & mpg.STATUS_WAIT_LIMIT:
        raise SystemExit("device wait limit hit during the benchmark")
    ms_inj_max = reduce_max(ms_inj, world, dev)
    total_flops = reduce_sum(flops * args.steps, world, dev)
    value = total_flops / (ms_inj_max * 1e-3) / 1e12

    # ---- what a launch costs by itself under this timing: a kernel that does nothing, same flush, same event pair
    def null_step(i):
        rc = mpg.mpgemmfi_null_launch(sh)
        if rc != 0:
            raise mpg.MpgemmfiError(rc, "mpgemmfi_null_launch")

    ms_null, _ = timed(null_step, 100, 5)
    launch_floor_us = ms_null / 100 * 1e3

    # ---- same kernel, injection and detection disabled: launches with and without injection alternate in one
    # loop (each with its own event pair and L2 flush), so that both see the same clocks and temperatures
    off_steps = max(10, args.steps // 4)
    ms_pair = [0.0, 0.0]
    for i in range(3):
        for inject in (True, False):
            flush.zero_()
            gemm_step(i, inject)
    torch.cuda.synchronize(dev)
    pair_events = []
    for i in range(off_steps):
        for inject in (True, False):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            gemm_step(i, inject)
            e1.record(stream)
            pair_events.append((0 if inject else 1, e0, e1))
    torch.cuda.synchronize(dev)
    for which, e0, e1 in pair_events:
        ms_pair[which] += e0.elapsed_time(e1)
    tflops_off = flops * off_steps / (ms_pair[1] * 1e-3) / 1e12
    on_over_off_time = ms_pair[0] / ms_pair[1]

    # ---- campaign: one clean GEMM + this rank's trials per launch
    rec = torch.empty((n_my, 12), dtype=torch.int32, device=dev)
    ws = torch.empty(mpg.mpgemmfi_campaign_workspace_bytes(dtype, M, N, K, n_my), dtype=torch.uint8, device=dev)

    def campaign_step(i):
        rc = mpg.mpgemmfi_campaign(dtype, M, N, K, A.data_ptr(), Bt.data_ptr(), C.data_ptr(), sites_dev.data_ptr(), n_my,
                                   mode, rec.data_ptr(), ws.data_ptr(), ws.numel(), sh)
        if rc != 0:
            raise mpg.MpgemmfiError(rc, "mpgemmfi_campaign")

    ms_one, _ = timed(campaign_step, 1, 3)
    camp_steps = max(3, min(200, args.steps // 10, int(3000.0 / max(ms_one, 1e-3))))     # about 3 s of launches
    ms_camp, _ = timed(campaign_step, camp_steps, 0)
    ms_camp_max = reduce_max(ms_camp, world, dev)
    trials_total = reduce_sum(float(n_my * camp_steps), world, dev)
    trials_per_s = trials_total / (ms_camp_max * 1e-3)

    # ---- N > 1: the whole table through the library's sharded campaign (every rank its share, then ONE all_gather of
    # the 48-byte records): time of the gather included, on the device, max over ranks
    sharded = None
    if world > 1:
        def local_campaign(dt_, A_, Bt_, share, mode_):
            campaign_step(0)
            return C, rec

        for _ in range(2):
            campaign_sharded(dtype, A, Bt, w.sites, mode, run_local=local_campaign)
        torch.cuda.synchronize(dev)
        dist.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        _, allrec = campaign_sharded(dtype, A, Bt, w.sites, mode, run_local=local_campaign)
        e1.record(stream)
        torch.cuda.synchronize(dev)
        ms_sh = reduce_max(e0.elapsed_time(e1), world, dev)
        sharded = {"trials": len(w.sites), "ms": ms_sh, "trials_per_s": len(w.sites) / (ms_sh * 1e-3),
                   "gathered_record_bytes": int(allrec.numel() * 4), "collective": f"one all_gather ({dist.get_backend()})"}

    # ---- end to end: pinned host buffers, copies inside the timed region
    hA = torch.from_numpy(w.A.view(view)).pin_memory()
    hB = torch.from_numpy(w.Bt.view(view)).pin_memory()
    hS = sites_host
    hC = torch.empty((M, N), dtype=torch.float32).pin_memory()
    hF = torch.empty(flags.numel(), dtype=torch.int32).pin_memory()

    def e2e_step(i):
        A.copy_(hA, non_blocking=True)
        Bt.copy_(hB, non_blocking=True)
        rc = mpg.mpgemmfi_gemm(dtype, M, N, K, A.data_ptr(), Bt.data_ptr(), C.data_ptr(), hS.data_ptr() + 32 * (i % n_my), 1, mode,
                               flags.data_ptr(), sh)
        if rc != 0:
            raise mpg.MpgemmfiError(rc, "mpgemmfi_gemm")
        hC.copy_(C, non_blocking=True)
        hF.copy_(flags, non_blocking=True)

    e2e_steps = max(5, min(50, args.steps // 20))
    ms_e2e, _ = timed(e2e_step, e2e_steps, 3)
    ms_e2e_max = reduce_max(ms_e2e, world, dev)
    e2e_serial = reduce_sum(flops * e2e_steps, world, dev) / (ms_e2e_max * 1e-3) / 1e12

    # The same steps as a user with more than one GEMM to run would queue them: two streams, two sets of device and
    # pinned result buffers, step i on stream i % 2, so that the upload of one step's operands overlaps the download of
    # the previous step's result (the link is full duplex). Every step still copies all of its inputs up and all of its
    # results down; timed from an event before the first step to an event after the last copy of both streams.
    streams2 = [torch.cuda.Stream(dev), torch.cuda.Stream(dev)]
    dbuf = [(A, Bt, C, flags, hC, hF)]
    dbuf.append((torch.empty_like(A), torch.empty_like(Bt), torch.empty_like(C), torch.empty_like(flags),
                 torch.empty((M, N), dtype=torch.float32).pin_memory(), torch.empty(flags.numel(), dtype=torch.int32).pin_memory()))
    flush2 = [flush, torch.empty_like(flush)]

    def e2e_pipelined(n_steps, first):
        for i in range(n_steps):
            k = i % 2
            dA, dB, dC, dF, oC, oF = dbuf[k]
            with torch.cuda.stream(streams2[k]):
                flush2[k].zero_()
                dA.copy_(hA, non_blocking=True)
                dB.copy_(hB, non_blocking=True)
                rc = mpg.mpgemmfi_gemm(dtype, M, N, K, dA.data_ptr(), dB.data_ptr(), dC.data_ptr(),
                                       hS.data_ptr() + 32 * ((first + i) % n_my), 1, mode,
                                       dF.data_ptr(), streams2[k].cuda_stream)
                if rc != 0:
                    raise mpg.MpgemmfiError(rc, "mpgemmfi_gemm")
                oC.copy_(dC, non_blocking=True)
                oF.copy_(dF, non_blocking=True)

    torch.cuda.synchronize(dev)
    e2e_pipelined(4, 0)
    torch.cuda.synchronize(dev)
    if world > 1:
        dist.barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for st2 in streams2:
        st2.wait_event(ev0)
    e2e_pipelined(e2e_steps, 4)
    for st2 in streams2:
        tail = torch.cuda.Event()
        tail.record(st2)
        stream.wait_event(tail)
    ev1.record(stream)
    torch.cuda.synchronize(dev)
    ms_e2e_pipe = reduce_max(ev0.elapsed_time(ev1), world, dev)
    e2e_value = reduce_sum(flops * e2e_steps, world, dev) / (ms_e2e_pipe * 1e-3) / 1e12
    if int(dbuf[1][5][0].item()) & mpg.STATUS_WAIT_LIMIT:
        raise SystemExit("device wait limit hit during the end-to-end steps")
    h2d = hA.numel() * hA.element_size() + hB.numel() * hB.element_size()      # (the 32-byte site rides in the launch)
    d2h = hC.numel() * 4 + hF.numel() * 4

    peaks, peak_src = load_peaks()
    achieved = flops / (ms_inj / args.steps * 1e-3) / 1e12

    min_bytes = (M * K + N * K) * A.element_size() + M * N * 4 + M * ((N + 31) // 32) * 4
    if args.config == "c1":
        # 33.6 MFLOP on four tiles: a single wave, bound by launch and pipeline-fill latency; reported in microseconds
        us = ms_inj / args.steps * 1e3
        roofline = {"bound": "latency", "achieved": us, "peak": None, "unit": "us per GEMM", "frac": None, "traffic": None,
                    "kernel": "gemm_kernel", "flops_per_launch": flops, "min_bytes_per_launch": min_bytes,
                    "note": "one wave of tiles: neither the tensor pipe nor HBM can be kept busy"}
    elif args.config == "c5":
        # narrow N: about 52 flop per byte, below the ridge; the GEMM is bound by HBM
        gbs = min_bytes / (ms_inj / args.steps * 1e-3) / 1e9
        roofline = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": gbs / peaks["hbm_gbs"], "traffic": None, "peak_source": f"{peak_src} (copy bandwidth)",
                    "kernel": "gemm_kernel", "bytes_per_launch": min_bytes}
    else:
        tensor_peak = peaks["bf16_tflops"] * (0.5 if dtype == synth.DTYPE_TF32 else 1.0)
        roofline = {"bound": "tensor", "achieved": achieved, "peak": tensor_peak, "unit": "TFLOP/s",
                    "frac": achieved / tensor_peak, "traffic": KERNEL_TRAFFIC_BYTES.get(args.config),
                    "peak_source": f"{peak_src} (cuBLAS bf16 burst" + (", halved for tf32)" if dtype == synth.DTYPE_TF32 else ")"),
                    "frac_of_sustained": achieved / (peaks["bf16_tflops_sustained"] * (0.5 if dtype == synth.DTYPE_TF32 else 1.0)),
                    "frac_of_nominal": achieved / (1125.0 if dtype == synth.DTYPE_TF32 else 2250.0),
                    "kernel": "gemm_kernel", "flops_per_launch": flops, "min_bytes_per_launch": min_bytes}
        # context only (frac above is the figure): the same with the empty-launch time taken off every step
        net_s = (ms_inj / args.steps - launch_floor_us * 1e-3) * 1e-3
        if net_s > 0:
            roofline["frac_net_of_launch_floor"] = flops / net_s / 1e12 / tensor_peak
        if dtype == synth.DTYPE_TF32 and rank == 0:
            # there is no measured TF32 peak: time the library's TF32 GEMM on the same shape, in this run (context for
            # the halved BF16 figure above; FP32 inputs, FP32 output, L2 flushed before every launch like the steps)
            import torch.backends.cuda
            old = torch.backends.cuda.matmul.allow_tf32
            torch.backends.cuda.matmul.allow_tf32 = True
            try:
                xa = A.view(torch.float32)
                xb = Bt.view(torch.float32).t()
                for _ in range(3):
                    flush.zero_()
                    torch.matmul(xa, xb, out=C)
                torch.cuda.synchronize(dev)
                evs = []
                for _ in range(10):
                    flush.zero_()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                    torch.matmul(xa, xb, out=C)
                    e1.record(stream)
                    evs.append((e0, e1))
                torch.cuda.synchronize(dev)
                lib_ms = statistics.median(e0.elapsed_time(e1) for e0, e1 in evs)
                roofline["library_tf32_tflops"] = flops / (lib_ms * 1e-3) / 1e12
                roofline["frac_of_library_tf32"] = achieved / roofline["library_tf32_tflops"]
            finally:
                torch.backends.cuda.matmul.allow_tf32 = old

    all_configs = None
    if world == 1 and not args.no_all_configs:
        # the other workloads in brief (same timing rules, fewer steps), so that one run shows all of them
        del hA, hB, hC, hF, dbuf, flush2
        all_configs = {}
        for name, o16 in (("c1", False), ("c2", False), ("c3a", False), ("c3a", True), ("c3b", False), ("c4", False), ("c5", False)):
            key = name + ("_fp16_output" if o16 else "")
            all_configs[key] = quick_config(name, mpg, synth, torch, dev, flush, peaks, steps=12 if name == "c4" else 40, out16=o16)
            torch.cuda.empty_cache()

    if rank == 0:
        baseline = None
        if world == 1 and not args.no_cpu_baseline:
            baseline = cpu_baseline(w)
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_inj_max / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": DTYPE_NAMES[dtype], "data": "synthetic",
            "config": {"workload": WORKLOAD_TEXT[args.config],
                       "l2": "flushed (256 MB memset) before every timed step",
                       "timing": "sum of per-step CUDA-event intervals on the launching stream",
                       "clocks_sampling": "nvidia-smi every 20 ms over the timed steps, continued over identical untimed "
                                          "steps until 0.4 s of load have been seen",
                       "site_table": "the step's site is handed over in host memory and travels in the kernel's launch "
                                     "parameters (all_configs.*.us_per_gemm_device_table: the same read from device memory)",
                       "trials_per_rank": n_my},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": "TFLOP/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps, "ms_per_step": ms_e2e_pipe / e2e_steps,
                    "how": "steps alternate between two streams with their own device and pinned buffers, so one step's "
                           "upload overlaps the previous step's download; every step copies all inputs and all results",
                    "one_stream": {"value": e2e_serial, "ms_per_step": ms_e2e_max / e2e_steps}},
            "gpu_launches": args.steps,
            "launch_floor_us": launch_floor_us,
            "roofline": roofline,
            "injection_off": {"tflops": tflops_off, "steps": off_steps,
                              "injected_over_plain_time": on_over_off_time,
                              "how": "launches with and without injection alternate in one loop"},
            "campaign": {"trials_per_s": trials_per_s, "trials_per_launch": n_my, "launches": camp_steps,
                         "ms_per_launch": ms_camp_max / camp_steps, "sharded": sharded},
            "cpu_baseline": baseline,
            "all_configs": all_configs,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
