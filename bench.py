#!/usr/bin/env python
"""Benchmark of the dense-contraction hot path on B200.

A step is one call of the headline workload: C = -(A . B^T), bf16 in / fp32 accumulate / bf16 out,
M = N = K = 4096, N(0,1) operands (seed 1), B stored N x K.  Inputs are resident in HBM; the step
rotates over several buffer sets whose total footprint exceeds L2, so operands are not served from
a warm cache.  One JSON line is printed by rank 0.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl tdx|reference]

With N > 1 (launched by torch.distributed.run) every rank runs an independent replica on its own
GPU -- the path has no exchange step, so there is no data-path collective; the reported value is
the sum over replicas divided by the slowest rank's time.

--impl reference times the CPU oracle (oracle/, fp64 loops) on a bounded row sample of the same
workload on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

M = N = K = 4096
SEED = 1
FLOP_PER_STEP = 2.0 * M * N * K
ALGO_BYTES_PER_STEP = 3 * M * N * 2          # each operand read once, the output written once (bf16)
METRIC = "GEMM/conv2d TFLOP/s at 1 B200 and fraction of dense bf16 (fp32) peak"
WORKLOAD = "gemm_bf16_negated_transB_4096"
BUFFER_SETS = 8                              # 8 x 96 MiB = 805 MB of operands and outputs > 126 MB of L2
FALLBACK_PEAKS = {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu, self.samples, self.proc, self.thread = gpu_index, [], None, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 7:
                self.samples.append(parts)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for p in self.samples:
            try:
                sm.append(float(p[0]))
                mx.append(float(p[1]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), p[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def oracle_sample(rows_target_seconds: float = 12.0):
    """Times the CPU oracle on a row sample of the workload; returns (tflops, cores, description)."""
    import numpy as np

    import oracle
    import seeded_inputs as si

    A, B = si.gemm_bf16_normal(M, N, K, seed=SEED, transB=1)
    oracle.gemm(8, N, K, 0, 1, -1.0, "bf16", A[:8], B)                 # page in, spin up the thread pool
    rows = np.arange(0, M, M // 16, dtype=np.int64)                      # 16 rows
    t0 = time.perf_counter()
    oracle.gemm(M, N, K, 0, 1, -1.0, "bf16", A, B, rows=rows)
    t = time.perf_counter() - t0
    n_rows = int(min(M, max(16, 16 * rows_target_seconds / max(t, 1e-3))))
    n_rows -= n_rows % 8
    rows = np.linspace(0, M - 1, n_rows).astype(np.int64)
    t0 = time.perf_counter()
    oracle.gemm(M, N, K, 0, 1, -1.0, "bf16", A, B, rows=rows)
    t = time.perf_counter() - t0
    tflops = 2.0 * n_rows * N * K / t / 1e12
    return tflops, oracle.num_threads(), f"{n_rows} of {M} output rows (all {N} columns), {t:.1f} s", t, n_rows


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import numpy as np

    import oracle
    import seeded_inputs as si

    A, B = si.gemm_bf16_normal(M, N, K, seed=SEED, transB=1)
    # size the per-step sample from a short probe so that the whole run takes about a minute
    oracle.gemm(M, N, K, 0, 1, -1.0, "bf16", A, B, rows=np.arange(8, dtype=np.int64))
    t0 = time.perf_counter()
    oracle.gemm(M, N, K, 0, 1, -1.0, "bf16", A, B, rows=np.arange(16, dtype=np.int64))
    rows_per_s = 16.0 / max(time.perf_counter() - t0, 1e-4)
    rows_per_step = int(max(1, min(256, rows_per_s * 60.0 / max(1, args.steps + args.warmup))))
    rows = np.linspace(0, M - 1, rows_per_step).astype(np.int64)
    for _ in range(args.warmup):
        oracle.gemm(M, N, K, 0, 1, -1.0, "bf16", A, B, rows=rows)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.gemm(M, N, K, 0, 1, -1.0, "bf16", A, B, rows=rows)
    t = time.perf_counter() - t0
    flops = 2.0 * rows_per_step * N * K * args.steps
    value = flops / t / 1e12
    sample = f"each step = {rows_per_step} of {M} output rows (all columns) of the workload"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "M": M, "N": N, "K": K, "transB": 1, "alpha": -1.0, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def run_tdx(args):
    import numpy as np
    import torch

    import paper_2409_03864_b200 as tdx
    import seeded_inputs as si

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    distributed = world > 1
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the tdx path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if distributed:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    tdx.lib()

    # CPU baseline first (rank 0, single-GPU runs only), before the GPU is busy
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, cores, desc, _, _ = oracle_sample()
        cpu_baseline = {"value": v, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": desc}

    A, B = si.gemm_bf16_normal(M, N, K, seed=SEED, transB=1)
    hA = torch.from_numpy(A.view(np.int16)).pin_memory()
    hB = torch.from_numpy(B.view(np.int16)).pin_memory()
    hC = torch.empty(M * N, dtype=torch.int16).pin_memory()
    sets = []
    for _ in range(BUFFER_SETS):
        sets.append((hA.cuda(non_blocking=True), hB.cuda(non_blocking=True),
                     torch.empty(M * N, dtype=torch.int16, device="cuda")))
    stream = torch.cuda.current_stream()
    st_cfg, cfg = tdx.tdx_default_gemm_config(M, N, K, 0, 1, tdx.TDX_BF16)

    def step(i):
        a, b, c = sets[i % BUFFER_SETS]
        tdx.check(tdx.tdx_gemm(M, N, K, 0, 1, -1.0, tdx.TDX_BF16, a, b, c, stream))

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    if distributed:
        dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    n0 = tdx.tdx_kernel_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(args.steps):
        step(i)
    e1.record(stream)
    torch.cuda.synchronize()
    launches = tdx.tdx_kernel_launch_count() - n0
    ms_total = e0.elapsed_time(e1)

    # per-launch durations of the dominant kernel (CUDA events on the launching stream)
    n_k = min(args.steps, 200)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_k)]
    for i, (a, b) in enumerate(evs):
        a.record(stream)
        step(i)
        b.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    kernel_ms = statistics.mean(a.elapsed_time(b) for a, b in evs)
    tdx.check(tdx.tdx_check_device_status(stream))

    if distributed:
        t = torch.tensor([ms_total], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_total = float(t.item())
        dist.barrier()
    value = world * FLOP_PER_STEP * args.steps / (ms_total * 1e-3) / 1e12

    # end to end through the host-buffer entry point: H2D of A and B, the GEMM, D2H of C, every step
    e2e_steps = max(3, min(args.steps, 20))
    for _ in range(3):
        tdx.check(tdx.tdx_gemm_host(M, N, K, 0, 1, -1.0, tdx.TDX_BF16, hA, hB, hC, stream))
    torch.cuda.synchronize()
    if distributed:
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        tdx.check(tdx.tdx_gemm_host(M, N, K, 0, 1, -1.0, tdx.TDX_BF16, hA, hB, hC, stream))
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    if distributed:
        t = torch.tensor([e2e_s], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_s = float(t.item())
    e2e_value = world * FLOP_PER_STEP * e2e_steps / e2e_s / 1e12

    if rank == 0:
        peaks, peak_kind = measured_peaks()
        peak = float(peaks["bf16_tflops"])
        achieved = FLOP_PER_STEP / (kernel_ms * 1e-3) / 1e12
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "M": M, "N": N, "K": K, "transA": 0, "transB": 1, "alpha": -1.0,
                       "accumulate": "fp32", "out": "bf16", "parallelism": f"replicas x{world}",
                       "l2": f"rotating {BUFFER_SETS} buffer sets ({BUFFER_SETS * ALGO_BYTES_PER_STEP / 1e6:.0f} MB) larger than L2",
                       "tile_config": cfg.as_dict() if st_cfg == 0 else None},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": "TFLOP/s", "h2d_bytes_per_step": 2 * M * K * 2,
                    "d2h_bytes_per_step": M * N * 2, "steps": e2e_steps, "api": "tdx_gemm_host (pinned host buffers)"},
            "gpu_launches": int(launches),
            "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                         "frac": achieved / peak, "traffic": None, "kernel": "umma_contract_kernel<false>",
                         "kernel_ms": kernel_ms, "peak_source": f"{peak_kind} bf16_tflops (burst)",
                         "frac_of_sustained_peak": achieved / float(peaks.get("bf16_tflops_sustained", peak)),
                         "hbm_gbs_algorithmic": ALGO_BYTES_PER_STEP / (kernel_ms * 1e-3) / 1e9},
            "cpu_baseline": cpu_baseline,
        }
        print(json.dumps(line))
    if distributed:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="tdx", choices=["tdx", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_tdx(args)


if __name__ == "__main__":
    sys.exit(main())
