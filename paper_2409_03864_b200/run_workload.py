"""Run one named workload a few times on the current GPU and print its device time.

  python -m paper_2409_03864_b200.run_workload c4 [--iters 20] [--warmup 3] [--cfg tile_m=256,tile_n=256] [--flush]

Workloads: c1 (fp32 256^3), c2, c3, c4, c5a..c5e, or "gemm:M:N:K:transA:transB" /
"conv:N:H:W:Cin:Cout:R:S:pad:stride" (bf16).  Inputs are the seeded synthetic tensors of the workload
(run from the repository root so that seeded_inputs.py is importable).  Each launch is timed with CUDA
events on the launching stream; --flush writes a 256 MB buffer between launches so that operands are
not served from a warm L2.  This is the small, single-kernel command used for profiler captures.
"""
from __future__ import annotations

import argparse
import statistics
import sys

import numpy as np
import torch

from . import binding as tdx

NAMED = {
    "c1": ("gemm_f32", 256, 256, 256, 0, 0, 1.0, 0),
    "c2": ("gemm", 4096, 4096, 4096, 0, 1, -1.0, 1),
    "c3": ("conv", 4, 128, 128, 64, 64, 3, 3, 1, 1, 2),
    "c4": ("conv", 32, 56, 56, 256, 256, 3, 3, 1, 1, 3),
    "c5a": ("gemm", 1024, 1024, 1024, 0, 0, 1.0, 4),
    "c5b": ("gemm", 8192, 8192, 8192, 0, 0, 1.0, 4),
    "c5c": ("gemm", 128, 8192, 8192, 0, 0, 1.0, 4),
    "c5d": ("gemm", 8192, 128, 8192, 0, 0, 1.0, 4),
    "c5e": ("gemm", 4096, 4096, 512, 0, 0, 1.0, 4),
}


def parse(spec):
    if spec in NAMED:
        return NAMED[spec]
    f = spec.split(":")
    v = [int(x) for x in f[1:]]
    if f[0] == "gemm":
        return ("gemm", *v, 1.0, 4)
    if f[0] == "conv":
        return ("conv", *v, 3)
    raise SystemExit(f"unknown workload {spec!r}")


def dev(a):
    a = np.ascontiguousarray(a)
    return torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a).cuda()


def main(argv=None):
    import seeded_inputs as si

    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("workload")
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--cfg", default="", help="comma-separated tdx_config fields, e.g. tile_m=256,tile_n=128")
    ap.add_argument("--flush", action="store_true")
    args = ap.parse_args(argv)
    w = parse(args.workload)
    cfg = None
    if args.cfg:
        kw = {k: int(v) for k, v in (kv.split("=") for kv in args.cfg.split(","))}
        kw.setdefault("kernel", tdx.TDX_KERNEL_UMMA)
        cfg = tdx.tdx_config(**kw)
    stream = torch.cuda.current_stream()
    if w[0] in ("gemm", "gemm_f32"):
        _, M, N, K, tA, tB, alpha, seed = w
        if w[0] == "gemm_f32":
            A, B = si.gemm_f32_uniform(M, N, K, seed=seed)
            dt, out = tdx.TDX_F32, torch.empty(M * N, dtype=torch.float32, device="cuda")
        else:
            A, B = si.gemm_bf16_normal(M, N, K, seed=seed, transA=tA, transB=tB)
            dt, out = tdx.TDX_BF16, torch.empty(M * N, dtype=torch.int16, device="cuda")
        dA, dB = dev(A), dev(B)
        flops = 2.0 * M * N * K
        st, c = tdx.tdx_default_gemm_config(M, N, K, tA, tB, dt)

        def launch():
            tdx.check(tdx.tdx_gemm_ex(M, N, K, tA, tB, alpha, dt, dA, dB, out, stream, cfg, None, 0))
    else:
        _, Nb, H, W, Cin, Cout, R, S, pad, stride, seed = w
        x, wt, b = si.conv_bf16(Nb, H, W, Cin, Cout, R, S, seed=seed)
        dx, dw, db = dev(x), dev(wt), dev(b)
        P, Q = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - S) // stride + 1
        out = torch.empty(Nb * P * Q * Cout, dtype=torch.int16, device="cuda")
        flops = 2.0 * Nb * P * Q * Cout * R * S * Cin
        st, c = tdx.tdx_default_conv2d_config(Nb, H, W, Cin, Cout, R, S, pad, stride, tdx.TDX_BF16)

        def launch():
            tdx.check(tdx.tdx_conv2d_bias_relu_ex(Nb, H, W, Cin, Cout, R, S, pad, stride, tdx.TDX_BF16, dx, dw, db, 1,
                                                  out, stream, cfg))
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if args.flush else None
    for _ in range(args.warmup):
        launch()
    times = []
    for _ in range(args.iters):
        if flush is not None:
            flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        launch()
        e1.record(stream)
        e1.synchronize()
        times.append(e0.elapsed_time(e1) * 1e3)
    tdx.check(tdx.tdx_check_device_status(stream))
    med, best = statistics.median(times), min(times)
    print(f"{args.workload}: config {cfg if cfg is not None else c}  median {med:.2f} us  min {best:.2f} us  "
          f"{flops / med / 1e6:.1f} TFLOP/s (median)  {flops / best / 1e6:.1f} TFLOP/s (min)"
          f"{'  [L2 flushed]' if args.flush else ''}")
    return 0


if __name__ == "__main__":
    sys.exit(main())
