#!/usr/bin/env python
"""Benchmark of the dense-contraction hot path on B200.

A step is one call of the headline workload: C = -(A . B^T), bf16 in / fp32 accumulate / bf16 out,
M = N = K = 4096, N(0,1) operands (seed 1), B stored N x K.  Inputs are resident in HBM; the step
rotates over several buffer sets whose total footprint exceeds L2, so operands are not served from
a warm cache.  One JSON line is printed by rank 0.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl tdx|reference] [--workload c2]

The line's top level is the headline workload timed over exactly K back-to-back steps.  Beside it:
  roofline     the dominant kernel against the measured peak (plus per-launch min / median from CUDA events around
               single launches, and a sustained figure from a loop of at least two seconds with the SM clock sampled)
  parity       the output of the last timed step compared with the CPU oracle on a row sample
  e2e          the same step through the host-buffer entry point (pinned host memory, copies inside the timed region)
  cpu_baseline the CPU oracle timed on a bounded sample of the same workload
  workloads    every other configuration (c1, c3, c4, c5a..c5e, the paper's batch-matmul nest in fp32 and bf16, the
               add_of_zero_pad op), each timed the same way with short loops, each with its own roofline fraction,
               clock record and parity check.  --no-table leaves it out; --workload X makes X the headline.

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

METRIC = "GEMM/conv2d TFLOP/s at 1 B200 and fraction of dense bf16 (fp32) peak"
FALLBACK_PEAKS = {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0}
L2_BYTES = 126e6
TOL = {"f32": 1e-5, "bf16": 2e-2}          # normalised error per output row, as the parity tests use

# DRAM bytes (read + write) per launch of the dominant kernel from an ncu capture of this program, with the file that
# holds the capture and the tile configuration it was taken with.  A run whose tile configuration differs reports
# null: the figure then describes another kernel variant.
TRAFFIC = {
    "c2": dict(bytes=98.8e6, profile="profiles/bench_dram_traffic.md",
               tile_config=dict(tile_m=256, tile_n=256, stages=3, split_k=1, store_mode=2, fit=2)),
    "c4": dict(bytes=56.0e6, profile="profiles/bench_dram_traffic.md",
               tile_config=dict(tile_m=256, tile_n=256, stages=3, split_k=1, store_mode=2, halo=3)),
    "azp": dict(bytes=111.0e6, profile="profiles/bench_dram_traffic.md", tile_config=None),
}

# name: (kind, dims..., seed, bound).  The default (headline) workload is c2.
WORKLOADS = {
    "c1": dict(kind="gemm", dtype="f32", M=256, N=256, K=256, tA=0, tB=0, alpha=1.0, seed=0, bound="alu",
               label="gemm_f32_256"),
    "c2": dict(kind="gemm", dtype="bf16", M=4096, N=4096, K=4096, tA=0, tB=1, alpha=-1.0, seed=1, bound="tensor",
               label="gemm_bf16_negated_transB_4096"),
    "c3": dict(kind="conv", N=4, H=128, W=128, Cin=64, Cout=64, R=3, S=3, pad=1, stride=1, seed=2, bound="tensor",
               label="conv_bf16_4x128x128x64_k3"),
    "c4": dict(kind="conv", N=32, H=56, W=56, Cin=256, Cout=256, R=3, S=3, pad=1, stride=1, seed=3, bound="tensor",
               label="conv_bf16_32x56x56x256_k3"),
    "c5a": dict(kind="gemm", dtype="bf16", M=1024, N=1024, K=1024, tA=0, tB=0, alpha=1.0, seed=4, bound="tensor",
                label="gemm_bf16_1024"),
    "c5b": dict(kind="gemm", dtype="bf16", M=8192, N=8192, K=8192, tA=0, tB=0, alpha=1.0, seed=4, bound="tensor",
                label="gemm_bf16_8192"),
    "c5c": dict(kind="gemm", dtype="bf16", M=128, N=8192, K=8192, tA=0, tB=0, alpha=1.0, seed=4, bound="hbm",
                label="gemm_bf16_128x8192x8192"),
    "c5d": dict(kind="gemm", dtype="bf16", M=8192, N=128, K=8192, tA=0, tB=0, alpha=1.0, seed=4, bound="hbm",
                label="gemm_bf16_8192x128x8192"),
    "c5e": dict(kind="gemm", dtype="bf16", M=4096, N=4096, K=512, tA=0, tB=0, alpha=1.0, seed=4, bound="tensor",
                label="gemm_bf16_4096x4096x512"),
    # the paper's own workload (Case Study 4): C[b,i,j] += A[b,i,k] * B[b,k,j], b < 6, i < 196, j < 256, k < 2305.
    # fp32: six bf16 piece products per multiply-add on the tensor cores for fp32 accuracy, so the fp32 problem is
    # reported against the fp32 ALU peak (what a CUDA-core kernel could reach at best); bf16: against the bf16 peak.
    "cs4": dict(kind="gemm_batched", dtype="f32", batch=6, M=196, N=256, K=2305, tA=0, tB=0, alpha=1.0, beta=1.0, seed=5,
                bound="alu", label="batch_matmul_accumulate_f32_6x196x256x2305"),
    "cs4_bf16": dict(kind="gemm_batched", dtype="bf16", batch=6, M=196, N=256, K=2305, tA=0, tB=0, alpha=1.0, beta=1.0,
                     seed=5, bound="tensor", label="batch_matmul_accumulate_bf16_6x196x256x2305"),
    # Case Study 3's add_of_zero_pad pattern as an op: y += zero_pad(x) in place, the activation shape of c4
    "azp": dict(kind="add_zero_pad", dtype="bf16", N=32, H=56, W=56, C=256, pad=1, seed=6, bound="hbm",
                label="add_of_zero_pad_bf16_32x56x56x256_pad1_in_place"),
}
TABLE_ORDER = ("c1", "c2", "c3", "c4", "c5a", "c5b", "c5c", "c5d", "c5e", "cs4", "cs4_bf16", "azp")


class Workload:
    """Shapes, algorithmic flops/bytes, seeded host inputs and oracle calls of one configuration."""

    def __init__(self, name):
        self.name, self.w = name, WORKLOADS[name]
        w = self.w
        if w["kind"] == "add_zero_pad":
            self.el = 2
            interior = w["N"] * w["H"] * w["W"] * w["C"]
            self.padded = w["N"] * (w["H"] + 2 * w["pad"]) * (w["W"] + 2 * w["pad"]) * w["C"]
            self.flops = float(interior)                       # one add per interior element
            self.in_bytes = 2 * interior * self.el             # x and the interior of y; the ring is never read
            self.out_bytes = interior * self.el
            self.out_elems = self.padded
            self.rows = w["N"]                                 # the oracle sample is taken in whole images
            self.unit = "images"
            self.h2d_bytes = (interior + self.padded) * self.el    # the host-buffer call moves x and the whole y
            self.d2h_bytes = self.padded * self.el
        elif w["kind"] == "gemm_batched":
            self.el = 4 if w["dtype"] == "f32" else 2
            self.flops = 2.0 * w["batch"] * w["M"] * w["N"] * w["K"]
            self.in_bytes = w["batch"] * (w["M"] * w["K"] + w["K"] * w["N"] + w["M"] * w["N"]) * self.el   # A, B and C read
            self.out_bytes = w["batch"] * w["M"] * w["N"] * self.el
            self.out_elems = w["batch"] * w["M"] * w["N"]
            self.rows = w["batch"]            # the oracle sample is taken in whole batches
            self.unit = "batches"
        elif w["kind"] == "gemm":
            self.el = 4 if w["dtype"] == "f32" else 2
            self.flops = 2.0 * w["M"] * w["N"] * w["K"]
            self.in_bytes = (w["M"] * w["K"] + w["K"] * w["N"]) * self.el
            self.out_bytes = w["M"] * w["N"] * self.el
            self.out_elems = w["M"] * w["N"]
            self.rows = w["M"]
        else:
            self.el = 2
            self.P = (w["H"] + 2 * w["pad"] - w["R"]) // w["stride"] + 1
            self.Q = (w["W"] + 2 * w["pad"] - w["S"]) // w["stride"] + 1
            self.rows = w["N"] * self.P * self.Q
            self.flops = 2.0 * self.rows * w["Cout"] * w["R"] * w["S"] * w["Cin"]
            self.in_bytes = (w["N"] * w["H"] * w["W"] * w["Cin"] + w["Cout"] * w["R"] * w["S"] * w["Cin"]) * 2 + w["Cout"] * 4
            self.out_bytes = self.rows * w["Cout"] * 2
            self.out_elems = self.rows * w["Cout"]
        self.unit = getattr(self, "unit", "output rows (all columns)")
        self.algo_bytes = self.in_bytes + self.out_bytes       # each operand read once, the output written once
        self.dtype = w.get("dtype", "bf16")

    def host_inputs(self):
        import seeded_inputs as si
        w = self.w
        if w["kind"] == "add_zero_pad":
            return (si.normal(w["seed"], 0, (w["N"], w["H"], w["W"], w["C"]), "bf16"),
                    si.normal(w["seed"], 1, (w["N"], w["H"] + 2 * w["pad"], w["W"] + 2 * w["pad"], w["C"]), "bf16"))
        if w["kind"] == "gemm_batched":
            gen = si.uniform if w["dtype"] == "f32" else si.normal
            return (gen(w["seed"], 0, (w["batch"], w["M"], w["K"]), w["dtype"]),
                    gen(w["seed"], 1, (w["batch"], w["K"], w["N"]), w["dtype"]),
                    gen(w["seed"], 2, (w["batch"], w["M"], w["N"]), w["dtype"]))
        if w["kind"] == "gemm":
            if w["dtype"] == "f32":
                return si.gemm_f32_uniform(w["M"], w["N"], w["K"], seed=w["seed"])
            return si.gemm_bf16_normal(w["M"], w["N"], w["K"], seed=w["seed"], transA=w["tA"], transB=w["tB"])
        return si.conv_bf16(w["N"], w["H"], w["W"], w["Cin"], w["Cout"], w["R"], w["S"], seed=w["seed"])

    def config_dict(self):
        return {k: v for k, v in self.w.items() if k not in ("kind", "seed", "bound", "label")}

    def oracle_rows(self, host, rows):
        """The oracle's result for the units `rows` (output rows; whole images / batches for the in-place kinds)."""
        import numpy as np

        import oracle
        w = self.w
        if w["kind"] == "add_zero_pad":      # rows = image indices
            p = w["pad"]
            return np.stack([oracle.add_zero_pad(1, w["H"], w["W"], w["C"], p, p, p, p, "bf16", host[0][n], host[1][n])[0]
                             for n in rows])
        if w["kind"] == "gemm_batched":      # rows = batch indices
            return np.stack([oracle.gemm_batched(1, w["M"], w["N"], w["K"], w["tA"], w["tB"], w["alpha"], w["beta"], w["dtype"],
                                                 host[0][b], host[1][b], host[2][b])[0] for b in rows])
        if w["kind"] == "gemm":
            return oracle.gemm(w["M"], w["N"], w["K"], w["tA"], w["tB"], w["alpha"], w["dtype"], host[0], host[1], rows=rows)
        return oracle.conv2d(w["N"], w["H"], w["W"], w["Cin"], w["Cout"], w["R"], w["S"], w["pad"], w["stride"], "bf16",
                             host[0], host[1], host[2], 1, rows=rows)

    def flops_for_rows(self, n_rows):
        return self.flops * n_rows / self.rows

    # ---- parity of a device result against the oracle on a sample of units
    def parity_units(self):
        import numpy as np
        if self.w["kind"] in ("add_zero_pad", "gemm_batched"):
            return np.unique(np.array([0, self.rows - 1], dtype=np.int64))
        # rows 0, 1, 63, 64, 126, 127 of up to eight 128-row blocks spread over the output, the last row included
        nblk = -(-self.rows // 128)
        blocks = np.unique(np.linspace(0, nblk - 1, min(nblk, 8)).astype(np.int64))
        rows = [b * 128 + r for b in blocks for r in (0, 1, 63, 64, 126, 127)] + [self.rows - 1]
        return np.unique(np.array([r for r in rows if r < self.rows], dtype=np.int64))

    def parity(self, host, out_host):
        """max normalised error of `out_host` (the device result, storage type) over the sampled units."""
        import numpy as np

        import oracle
        w, units = self.w, self.parity_units()
        ref = self.oracle_rows(host, units)
        if w["kind"] == "add_zero_pad":
            got = oracle.decode(out_host.reshape(w["N"], -1)[units], "bf16").reshape(len(units), -1)
            ref = ref.reshape(len(units), -1)
            # an elementwise sum: |x| + |y| bounds each output; one row per image, scaled by the image's largest bound
            xp = np.zeros((len(units),) + host[1].shape[1:])
            p = w["pad"]
            xp[:, p:p + w["H"], p:p + w["W"], :] = np.abs(oracle.decode(host[0][units], "bf16"))
            sc = (xp + np.abs(oracle.decode(host[1][units], "bf16"))).reshape(len(units), -1).max(axis=1)
            desc = f"images {units.tolist()} of {self.rows}"
        elif w["kind"] == "gemm_batched":
            got = oracle.decode(out_host.reshape(w["batch"], w["M"], w["N"])[units], w["dtype"]).reshape(-1, w["N"])
            ref = ref.reshape(-1, w["N"])
            sc = np.concatenate([oracle.gemm_batched_row_scales(1, w["M"], w["N"], w["K"], w["tA"], w["tB"], w["alpha"], w["beta"],
                                                                w["dtype"], host[0][b], host[1][b], host[2][b]) for b in units])
            desc = f"batches {units.tolist()} of {self.rows}, all rows"
        elif w["kind"] == "gemm":
            got = oracle.decode(out_host.reshape(w["M"], w["N"])[units], w["dtype"])
            sc = oracle.gemm_row_scales(w["M"], w["N"], w["K"], w["tA"], w["tB"], w["alpha"], w["dtype"], host[0], host[1], rows=units)
            desc = f"{len(units)} of {self.rows} rows, all columns"
        else:
            got = oracle.decode(out_host.reshape(self.rows, w["Cout"])[units], "bf16")
            sc = oracle.conv_row_scales(w["N"], w["H"], w["W"], w["Cin"], w["Cout"], w["R"], w["S"], w["pad"], w["stride"],
                                        "bf16", host[0], host[1], host[2], rows=units)
            desc = f"{len(units)} of {self.rows} output pixels, all channels"
        err = oracle.max_normalised_error(got, ref, sc)
        tol = TOL[self.dtype]
        return {"max_err": err, "tol": tol, "ok": bool(err < tol), "rows": desc}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int, period_ms: int = 100):
        self.gpu, self.samples, self.proc, self.thread, self.period = gpu_index, [], None, None, period_ms
        self.lock = threading.Lock()

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", str(self.period)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 7:
                with self.lock:
                    self.samples.append(parts)

    def mark(self):
        """Index of the next sample: summary(mark) later covers only what was sampled from here on."""
        with self.lock:
            return len(self.samples)

    def summary(self, since=0):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        with self.lock:
            part = list(self.samples[since:])
        sm, mx, reasons = [], [], set()
        for p in part:
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

    def stop(self, since=0):
        if self.proc is None:
            return self.summary()
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        return self.summary(since)


def max_over_ranks(x, device):
    """Slowest rank's figure (the job's time); a no-op without a process group.  Works with NCCL (cuda tensors)
    and gloo (cpu tensors)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_throughput(flops_per_step, steps, ms_slowest, world):
    """Whole-job TFLOP/s of `world` independent replicas that each did `steps` steps; time = the slowest rank's."""
    return world * flops_per_step * steps / (ms_slowest * 1e-3) / 1e12


def oracle_sample(wl, host, target_seconds=12.0):
    """Times the CPU oracle on a row sample of the workload; returns (TFLOP/s, threads, description)."""
    import numpy as np

    import oracle

    wl.oracle_rows(host, np.arange(min(8, wl.rows), dtype=np.int64))            # page in, spin up the thread pool
    probe = np.linspace(0, wl.rows - 1, min(16, wl.rows)).astype(np.int64)
    t0 = time.perf_counter()
    wl.oracle_rows(host, probe)
    t = time.perf_counter() - t0
    n_rows = int(min(wl.rows, max(len(probe), len(probe) * target_seconds / max(t, 1e-4))))
    rows = np.linspace(0, wl.rows - 1, n_rows).astype(np.int64)
    t0 = time.perf_counter()
    wl.oracle_rows(host, rows)
    t = time.perf_counter() - t0
    return (wl.flops_for_rows(n_rows) / t / 1e12, oracle.num_threads(),
            f"{n_rows} of {wl.rows} {wl.unit}, {t:.1f} s")


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import numpy as np

    import oracle

    wl = Workload(args.workload)
    host = wl.host_inputs()
    # size the per-step sample from a short probe so that the whole run takes about a minute
    wl.oracle_rows(host, np.arange(min(8, wl.rows), dtype=np.int64))
    probe = np.linspace(0, wl.rows - 1, min(16, wl.rows)).astype(np.int64)
    t0 = time.perf_counter()
    wl.oracle_rows(host, probe)
    rows_per_s = len(probe) / max(time.perf_counter() - t0, 1e-5)
    rows_per_step = int(max(1, min(wl.rows, rows_per_s * 60.0 / max(1, args.steps + args.warmup))))
    rows = np.linspace(0, wl.rows - 1, rows_per_step).astype(np.int64)
    for _ in range(args.warmup):
        wl.oracle_rows(host, rows)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        wl.oracle_rows(host, rows)
    t = time.perf_counter() - t0
    value = wl.flops_for_rows(rows_per_step) * args.steps / t / 1e12
    sample = f"each step = {rows_per_step} of {wl.rows} {wl.unit} of the workload"
    cfg = dict(wl.config_dict(), workload=wl.w["label"], sample=sample)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": cfg,
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


class DeviceRun:
    """Device buffers and launchers of one workload: rotating buffer sets larger than L2, the step through the C entry
    point on raw device addresses, the host-buffer step, and the read-back of a set's output."""

    def __init__(self, wl, host, tdx, torch, stream, want_host_path=True):
        import numpy as np
        self.wl, self.host, self.tdx, self.torch, self.stream = wl, host, tdx, torch, stream
        w = wl.w

        def pinned(a):
            a = np.ascontiguousarray(a)
            return torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).pin_memory()

        self.h_in = [pinned(a) for a in host]
        out_dtype = torch.float32 if wl.dtype == "f32" else torch.int16
        self.h_out = torch.empty(wl.out_elems, dtype=out_dtype).pin_memory()
        # rotate over enough buffer sets that the cycled footprint exceeds L2 several times
        self.n_sets = int(min(512, max(2, -(-int(6 * L2_BYTES) // wl.algo_bytes))))
        sets = [([h.cuda(non_blocking=True) for h in self.h_in], torch.empty(wl.out_elems, dtype=out_dtype, device="cuda"))
                for _ in range(self.n_sets)]
        self.raw_stream = stream.cuda_stream          # the device launchers below take the raw handle
        DT = tdx.TDX_F32 if wl.dtype == "f32" else tdx.TDX_BF16
        self.in_place_input = None                    # index of the input the step overwrites, if any
        L = tdx.lib()
        if w["kind"] == "add_zero_pad":
            st_cfg, cfg = 1, None
            pd = w["pad"]
            sets = [(ins, ins[1]) for ins, _ in sets]        # in place: the output is the set's own y
            self.in_place_input = 1
            c_azp = L.tdx_add_zero_pad

            def launch(ins, out):
                return c_azp(w["N"], w["H"], w["W"], w["C"], pd, pd, pd, pd, DT, ins[0], out, out, self.raw_stream)

            h_y = self.h_in[1].clone().pin_memory()

            def launch_host():
                return tdx.tdx_add_zero_pad_host(w["N"], w["H"], w["W"], w["C"], pd, pd, pd, pd, DT, self.h_in[0], h_y, stream)
            kernel_name = "add_zero_pad_kernel<bf16>"
        elif w["kind"] == "gemm_batched":
            st_cfg, cfg = 1, None
            # the step accumulates into C (beta = 1); each buffer set carries its own copy of C, and the output IS that buffer
            sets = [(ins, ins[2]) for ins, _ in sets]
            self.in_place_input = 2
            c_batched = L.tdx_gemm_batched
            sa, sb, sc = w["M"] * w["K"], w["K"] * w["N"], w["M"] * w["N"]

            def launch(ins, out):
                return c_batched(w["batch"], w["M"], w["N"], w["K"], w["tA"], w["tB"], w["alpha"], w["beta"], DT,
                                 ins[0], sa, ins[1], sb, out, sc, self.raw_stream)

            def launch_host():
                self.h_out.copy_(self.h_in[2].reshape(-1))
                return tdx.tdx_gemm_batched_host(w["batch"], w["M"], w["N"], w["K"], w["tA"], w["tB"], w["alpha"], w["beta"], DT,
                                                 self.h_in[0], self.h_in[1], self.h_out, stream)
            kernel_name = ("umma_contract_kernel<false> on bf16 pieces (+ split_f32_bf16x3_kernel, splitk_reduce_f32_kernel)"
                           if wl.dtype == "f32" else "umma_contract_kernel<false> (+ pad_k_bf16_kernel, splitk_reduce_kernel)")
        elif w["kind"] == "gemm":
            st_cfg, cfg = tdx.tdx_default_gemm_config(w["M"], w["N"], w["K"], w["tA"], w["tB"], DT)
            c_gemm = L.tdx_gemm              # the C entry point itself: integers in, status out

            def launch(ins, out):
                return c_gemm(w["M"], w["N"], w["K"], w["tA"], w["tB"], w["alpha"], DT, ins[0], ins[1], out, self.raw_stream)

            def launch_host():
                return tdx.tdx_gemm_host(w["M"], w["N"], w["K"], w["tA"], w["tB"], w["alpha"], DT, self.h_in[0], self.h_in[1],
                                         self.h_out, stream)
            kernel_name = "sgemm_small_rowmajor_kernel" if wl.dtype == "f32" else "umma_contract_kernel<false>"
        else:
            cargs = (w["N"], w["H"], w["W"], w["Cin"], w["Cout"], w["R"], w["S"], w["pad"], w["stride"], DT)
            st_cfg, cfg = tdx.tdx_default_conv2d_config(*cargs)
            c_conv = L.tdx_conv2d_bias_relu

            def launch(ins, out):
                return c_conv(*cargs, ins[0], ins[1], ins[2], 1, out, self.raw_stream)

            def launch_host():
                return tdx.tdx_conv2d_bias_relu_host(*cargs, self.h_in[0], self.h_in[1], self.h_in[2], 1, self.h_out, stream)
            kernel_name = "umma_conv_halo_kernel" if (st_cfg == 0 and cfg.halo >= 2) else "umma_contract_kernel<true>"
        self.sets, self.launch, self.launch_host, self.kernel_name = sets, launch, launch_host, kernel_name
        self.tile_config = cfg.as_dict() if st_cfg == 0 else None
        # The timed loop passes raw device addresses and the raw stream handle (the binding takes integers as they are),
        # so that a step's host cost is the C call itself: the small workloads are otherwise bound by Python marshalling.
        self.ptr_sets = [(tuple(t.data_ptr() for t in ins), out.data_ptr()) for ins, out in sets]

    def step(self, i):
        ins, out = self.ptr_sets[i % self.n_sets]
        self.tdx.check(self.launch(ins, out))

    def timed(self, steps, first=0):
        """`steps` back-to-back steps between two events on the launching stream; milliseconds."""
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(self.stream)
        for i in range(steps):
            self.step(first + i)
        e1.record(self.stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    def per_launch(self, n, first=0):
        """Events around every single step: (min, median) milliseconds of a step launched onto an idle stream tail."""
        torch = self.torch
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        for i, (a, b) in enumerate(evs):
            a.record(self.stream)
            self.step(first + i)
            b.record(self.stream)
        torch.cuda.synchronize()
        t = sorted(a.elapsed_time(b) for a, b in evs)
        return t[0], statistics.median(t)

    def parity_of_step(self, last_index):
        """Output of step `last_index` against the oracle.  A step that accumulates in place is repeated once on a
        freshly uploaded copy of its input/output buffer, so that the compared result is one step's."""
        torch = self.torch
        k = last_index % self.n_sets
        ins, out = self.sets[k]
        if self.in_place_input is not None:
            ins[self.in_place_input].copy_(self.h_in[self.in_place_input], non_blocking=True)
            self.step(last_index)
        torch.cuda.synchronize()
        out_host = out.cpu().numpy()
        import numpy as np
        if out_host.dtype == np.int16:
            out_host = out_host.view(np.uint16)
        return self.wl.parity(self.host, out_host)

    def free(self):
        self.sets, self.ptr_sets, self.h_in, self.h_out = [], [], [], None
        self.torch.cuda.empty_cache()


def roofline_of(wl, kernel_ms, peaks, peak_kind, sm_count):
    """achieved / peak of one step taking kernel_ms, against the bound the workload names."""
    bound = wl.w["bound"]
    if bound == "tensor":
        achieved, unit = wl.flops / (kernel_ms * 1e-3) / 1e12, "TFLOP/s"
        peak, src = float(peaks["bf16_tflops"]), f"{peak_kind} bf16_tflops (burst)"
    elif bound == "hbm":
        achieved, unit = wl.algo_bytes / (kernel_ms * 1e-3) / 1e9, "GB/s"
        peak, src = float(peaks["hbm_gbs"]), f"{peak_kind} hbm_gbs"
    else:   # fp32 problems: 2 flops x 128 lanes x SMs x max SM clock
        achieved, unit = wl.flops / (kernel_ms * 1e-3) / 1e12, "TFLOP/s"
        peak = 2 * 128 * sm_count * float(peaks.get("sm_max_mhz", 1965.0)) * 1e6 / 1e12
        src = "derived: 2 x 128 fp32 lanes x SMs x max SM clock"
    return {"bound": bound, "achieved": achieved, "peak": peak, "unit": unit, "frac": achieved / peak, "peak_source": src}


def traffic_for(name, tile_config):
    """(bytes or None, provenance) -- the captured DRAM traffic only when the running tile configuration is the captured one."""
    t = TRAFFIC.get(name)
    if t is None:
        return None, None
    want = t["tile_config"]
    same = want is None or (tile_config is not None and all(tile_config.get(k) == v for k, v in want.items()))
    prov = {"profile": t["profile"], "captured_tile_config": want, "matches_running_config": bool(same)}
    return (t["bytes"] if same else None), prov


def table_entry(name, tdx, torch, stream, peaks, peak_kind, sm_count, sampler):
    """One row of `workloads`: short loops of one configuration, its roofline fraction, clocks and parity."""
    wl = Workload(name)
    host = wl.host_inputs()
    run = DeviceRun(wl, host, tdx, torch, stream)
    for i in range(5):
        run.step(i)
    torch.cuda.synchronize()
    est_ms = max(run.timed(3) / 3, 1e-3)
    steps = int(min(200, max(20, 30.0 / est_ms)))          # about 30 ms of back-to-back steps
    mark = sampler.mark()
    n0 = tdx.tdx_kernel_launch_count()
    ms = run.timed(steps)
    launches = tdx.tdx_kernel_launch_count() - n0
    t_min, t_med = run.per_launch(min(50, steps), first=steps)
    time.sleep(0.12)                                       # let the sampler see the region just timed
    clocks = sampler.summary(mark)
    par = run.parity_of_step(steps - 1)
    tdx.check(tdx.tdx_check_device_status(stream))
    kernel_ms = ms / steps
    entry = {"label": wl.w["label"], "us": 1e3 * kernel_ms, "us_min": 1e3 * t_min, "us_median": 1e3 * t_med,
             "tflops": wl.flops / (kernel_ms * 1e-3) / 1e12, "steps": steps, "launches_per_step": launches / steps,
             "kernel": run.kernel_name, "tile_config": run.tile_config, "clocks": clocks, "parity": par,
             "l2": f"rotating {run.n_sets} buffer sets ({run.n_sets * wl.algo_bytes / 1e6:.0f} MB)"}
    entry.update(roofline_of(wl, kernel_ms, peaks, peak_kind, sm_count))
    run.free()
    return entry


def run_tdx(args):
    import torch

    import paper_2409_03864_b200 as tdx

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
    wl = Workload(args.workload)
    w = wl.w
    host = wl.host_inputs()

    # CPU baseline first (rank 0, single-GPU runs only), before the GPU is busy
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, cores, desc = oracle_sample(wl, host)
        cpu_baseline = {"value": v, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": desc}

    stream = torch.cuda.current_stream()
    run = DeviceRun(wl, host, tdx, torch, stream)

    for i in range(args.warmup):
        run.step(i)
    torch.cuda.synchronize()
    if distributed:
        dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    n0 = tdx.tdx_kernel_launch_count()
    ms_total = run.timed(args.steps)
    launches = tdx.tdx_kernel_launch_count() - n0
    time.sleep(0.12)
    clocks = sampler.summary() if rank == 0 else None

    # the output of the last timed step against the oracle
    parity = run.parity_of_step(args.steps - 1) if rank == 0 else None

    # launch duration of the dominant kernel from events around single launches (at least 50), and around groups of 10
    n_single = max(50, min(args.steps, 200))
    t_min, t_med = run.per_launch(n_single, first=args.steps)
    group = 10
    n_groups = max(1, min(args.steps // group, 50))
    grouped_ms = statistics.mean(run.timed(group, first=g * group) for g in range(n_groups)) / group

    # sustained: back-to-back steps for at least two seconds, SM clock sampled meanwhile (the power cap bites here)
    sustained = None
    if rank == 0 and world == 1 and not args.no_sustained:
        n_sus = int(max(args.steps, 2200.0 / max(ms_total / args.steps, 1e-3)))
        mark = sampler.mark()
        ms_sus = run.timed(n_sus)
        time.sleep(0.12)
        sustained = {"steps": n_sus, "seconds": ms_sus * 1e-3, "ms_per_step": ms_sus / n_sus,
                     "tflops": wl.flops * n_sus / (ms_sus * 1e-3) / 1e12, "clocks": sampler.summary(mark)}

    # --graph: the same steps captured once into a CUDA graph and replayed, which takes the per-call host cost out
    # of a launch-bound step (the small workloads); reported beside the stream-of-calls figure, never instead of it
    graph_info = None
    if args.graph:
        side = torch.cuda.Stream()       # capture needs a stream of its own; the launchers read run.raw_stream when called
        saved_raw = run.raw_stream
        try:
            per_graph = max(1, min(args.steps, 60))
            replays = max(1, args.steps // per_graph)
            run.raw_stream = side.cuda_stream
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                for i in range(per_graph):
                    run.step(i)
            with torch.cuda.stream(side):
                g.replay()
                torch.cuda.synchronize()
                g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                g0.record(side)
                for _ in range(replays):
                    g.replay()
                g1.record(side)
                torch.cuda.synchronize()
            graph_info = {"ms_per_step": g0.elapsed_time(g1) / (replays * per_graph), "steps_per_graph": per_graph,
                          "replays": replays}
        except Exception as exc:      # capture refused: report it, the stream-of-calls figures stand
            graph_info = {"error": str(exc)[:200]}
        finally:
            run.raw_stream = saved_raw
    launches_per_step = launches / args.steps
    # average launch duration over the timed region (one dominant kernel per step; a split-K step also holds its
    # small reduction kernel, which this charges to the dominant kernel)
    kernel_ms = ms_total / args.steps
    tdx.check(tdx.tdx_check_device_status(stream))

    if distributed:
        ms_total = max_over_ranks(ms_total, "cuda")
        dist.barrier()
    value = replica_throughput(wl.flops, args.steps, ms_total, world)

    # end to end through the host-buffer entry point: H2D of the inputs, the kernels, D2H of the result, every step
    e2e_steps = max(3, min(args.steps, 20))
    for _ in range(3):
        tdx.check(run.launch_host())
    torch.cuda.synchronize()
    if distributed:
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        tdx.check(run.launch_host())
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    if distributed:
        e2e_s = max_over_ranks(e2e_s, "cuda")
    e2e_value = replica_throughput(wl.flops, e2e_steps, e2e_s * 1e3, world)

    line = None
    if rank == 0:
        peaks, peak_kind = measured_peaks()
        sm_count = torch.cuda.get_device_properties(local_rank).multi_processor_count
        roof = roofline_of(wl, kernel_ms, peaks, peak_kind, sm_count)
        traffic, prov = traffic_for(args.workload, run.tile_config)
        roof.update({"traffic": traffic, "traffic_source": prov, "kernel": run.kernel_name, "kernel_ms": kernel_ms,
                     "launches_per_step": launches_per_step, "kernel_ms_event_groups_of_10": grouped_ms,
                     "kernel_ms_single_launch_min": t_min, "kernel_ms_single_launch_median": t_med,
                     "single_launches_timed": n_single,
                     "hbm_gbs_algorithmic": wl.algo_bytes / (kernel_ms * 1e-3) / 1e9})
        if graph_info is not None:
            roof["cuda_graph"] = graph_info
        if w["bound"] == "tensor":
            roof["frac_of_sustained_peak"] = roof["achieved"] / float(peaks.get("bf16_tflops_sustained", roof["peak"]))
        if sustained is not None:
            sus_roof = roofline_of(wl, sustained["ms_per_step"], peaks, peak_kind, sm_count)
            sustained["frac_of_burst_peak"] = sus_roof["frac"]
            if w["bound"] == "tensor":
                sustained["frac_of_sustained_peak"] = sus_roof["achieved"] / float(peaks.get("bf16_tflops_sustained", sus_roof["peak"]))
            roof["sustained"] = sustained
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
            "config": dict(wl.config_dict(), workload=w["label"], accumulate="fp32", parallelism=f"replicas x{world}",
                           l2=f"rotating {run.n_sets} buffer sets ({run.n_sets * wl.algo_bytes / 1e6:.0f} MB) larger than L2",
                           tile_config=run.tile_config),
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": "TFLOP/s", "h2d_bytes_per_step": int(getattr(wl, "h2d_bytes", wl.in_bytes)),
                    "d2h_bytes_per_step": int(getattr(wl, "d2h_bytes", wl.out_bytes)), "steps": e2e_steps,
                    "api": "tdx_gemm_host / tdx_conv2d_bias_relu_host (pinned host buffers)"},
            "gpu_launches": int(launches),
            "parity": parity,
            "roofline": roof,
            "cpu_baseline": cpu_baseline,
        }
    run.free()

    # every other configuration, timed the same way with short loops (single-GPU runs of the headline workload only)
    if rank == 0 and world == 1 and not args.no_table:
        peaks, peak_kind = measured_peaks()
        sm_count = torch.cuda.get_device_properties(local_rank).multi_processor_count
        table = {}
        for name in TABLE_ORDER:
            if name == args.workload:
                table[name] = {"label": w["label"], "us": 1e3 * kernel_ms, "us_min": 1e3 * t_min, "us_median": 1e3 * t_med,
                               "tflops": line["roofline"]["achieved"] if w["bound"] != "hbm" else wl.flops / (kernel_ms * 1e-3) / 1e12,
                               "steps": args.steps, "launches_per_step": launches_per_step, "kernel": line["roofline"]["kernel"],
                               "tile_config": line["config"]["tile_config"], "clocks": clocks, "parity": parity,
                               **{k: line["roofline"][k] for k in ("bound", "achieved", "peak", "unit", "frac", "peak_source")}}
                continue
            try:
                table[name] = table_entry(name, tdx, torch, stream, peaks, peak_kind, sm_count, sampler)
            except Exception as exc:        # one configuration failing must not take the headline line with it
                table[name] = {"error": f"{type(exc).__name__}: {str(exc)[:200]}"}
        line["workloads"] = table
    if rank == 0:
        sampler.stop()
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
    ap.add_argument("--no-table", action="store_true", help="leave the per-configuration `workloads` table out")
    ap.add_argument("--no-sustained", action="store_true", help="leave the two-second sustained loop out")
    ap.add_argument("--graph", action="store_true",
                    help="also time the steps captured into a CUDA graph (roofline.cuda_graph)")
    ap.add_argument("--workload", default="c2", choices=sorted(WORKLOADS),
                    help="c2 (default) is the headline workload; the others are the remaining configurations")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_tdx(args)


if __name__ == "__main__":
    sys.exit(main())
