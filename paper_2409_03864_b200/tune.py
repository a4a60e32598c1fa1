"""Tile-configuration search over a list of workloads (command-line front end of tdx_tune_*).

  python -m paper_2409_03864_b200.tune [--iters 20] [--out tuned.json] [--top 5] [workload ...]

Workloads: c2 (4096^3 negated GEMM with transposed B), c3 / c4 (the two convolutions), c5 (the five
GEMM shapes of the search sweep), or explicit "gemm:M:N:K:transA:transB" /
"conv:N:H:W:Cin:Cout:R:S:pad:stride".  For each workload the search times every statically feasible
configuration on the device, prints the best few, and stores the winner in the tuning cache, which
--out saves as JSON (load it with tdx_tune_load).
"""
from __future__ import annotations

import argparse
import json
import sys

from . import binding as tdx

NAMED = {
    "c2": ["gemm:4096:4096:4096:0:1"],
    "c3": ["conv:4:128:128:64:64:3:3:1:1"],
    "c4": ["conv:32:56:56:256:256:3:3:1:1"],
    "c5": ["gemm:1024:1024:1024:0:0", "gemm:8192:8192:8192:0:0", "gemm:128:8192:8192:0:0",
           "gemm:8192:128:8192:0:0", "gemm:4096:4096:512:0:0"],
}


def expand(names):
    out = []
    for n in names or ["c2", "c3", "c4", "c5"]:
        out.extend(NAMED.get(n, [n]))
    return out


def flops(spec):
    f = spec.split(":")
    v = [int(x) for x in f[1:]]
    if f[0] == "gemm":
        return 2.0 * v[0] * v[1] * v[2]
    N, H, W, Cin, Cout, R, S, pad, stride = v
    P = (H + 2 * pad - R) // stride + 1
    Q = (W + 2 * pad - S) // stride + 1
    return 2.0 * N * P * Q * Cout * R * S * Cin


def tune_one(spec, iters, budget=0):
    f = spec.split(":")
    v = [int(x) for x in f[1:]]
    if f[0] == "gemm":
        if budget > 0:      # model-guided: time only the candidates the cost model ranks best
            return tdx.tdx_tune_gemm_guided(*v, tdx.TDX_BF16, budget, iters=iters, cap=8192)[:4]
        return tdx.tdx_tune_gemm(*v, tdx.TDX_BF16, iters=iters, cap=8192)
    if f[0] == "conv":
        return tdx.tdx_tune_conv2d(*v, tdx.TDX_BF16, iters=iters, cap=8192)
    raise SystemExit(f"unknown workload {spec!r}")


def brief(c):
    s = f"{'pair ' if c['cta_pair'] == 2 else ''}m{c['tile_m']} n{c['tile_n']} st{c['stages']} sk{c['split_k']} r{c['raster']} ks{c['k_stagger']} sm{c['store_mode']}"
    if c.get("fit"):
        s += f" fit{c['fit']}"
    if c["patch_w"]:
        s += f" p{c['patch_w']}x{c['patch_h']} h{c['halo']}"
    return s


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("workloads", nargs="*")
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--top", type=int, default=5)
    ap.add_argument("--budget", type=int, default=0,
                    help="GEMM: time only this many candidates, chosen by the cost model (0 = all)")
    ap.add_argument("--out", default=None, help="save the tuning cache (JSON) here")
    ap.add_argument("--json", default=None, help="also write every candidate's time to this file")
    args = ap.parse_args(argv)
    report = {}
    for spec in expand(args.workloads):
        st, best, best_us, tried = tune_one(spec, args.iters, args.budget)
        if st != tdx.TDX_OK:
            print(f"{spec}: status {st}: {tdx.tdx_last_error()}")
            continue
        fl = flops(spec)
        tried.sort(key=lambda t: t[1])
        print(f"{spec}: best {brief(best.as_dict())}  {best_us:9.2f} us  {fl / best_us / 1e6:8.1f} TFLOP/s"
              f"  ({len(tried)} candidates, slowest {tried[-1][1]:.1f} us)")
        for c, us in tried[:args.top]:
            print(f"      {brief(c):34s} {us:9.2f} us  {fl / us / 1e6:8.1f} TFLOP/s")
        report[spec] = {"best": best.as_dict(), "best_us": best_us, "tflops": fl / best_us / 1e6,
                        "tried": [{"cfg": c, "us": us} for c, us in tried]}
        sys.stdout.flush()
    if args.out:
        tdx.check(tdx.tdx_tune_save(args.out))
    if args.json:
        with open(args.json, "w") as f:
            json.dump(report, f, indent=1)
    return 0


if __name__ == "__main__":
    sys.exit(main())
