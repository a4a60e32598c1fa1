"""Host-side pieces of bench.py that need no GPU: the parity check it applies to a timed result, the traffic
provenance rule and the roofline arithmetic."""
import os
import sys

import numpy as np

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def _result_from_oracle(wl, host):
    """A full-size output buffer whose sampled units hold the oracle's values in the storage type (zeros elsewhere)."""
    units = wl.parity_units()
    ref = wl.oracle_rows(host, units)
    w = wl.w
    if wl.dtype == "f32":
        out = np.zeros(wl.out_elems, dtype=np.float32)
        conv = lambda v: v.astype(np.float32)          # noqa: E731
    else:
        out = np.zeros(wl.out_elems, dtype=np.uint16)
        conv = oracle.round_bf16
    if w["kind"] == "gemm":
        out.reshape(w["M"], w["N"])[units] = conv(ref)
    elif w["kind"] == "conv":
        out.reshape(wl.rows, w["Cout"])[units] = conv(ref)
    elif w["kind"] == "gemm_batched":
        out.reshape(w["batch"], w["M"], w["N"])[units] = conv(ref)
    else:
        out.reshape(w["N"], -1)[units] = conv(ref).reshape(len(units), -1)
    return out, units


def test_bench_parity_accepts_the_oracle_and_rejects_a_planted_error():
    for name in ("c1", "c3", "cs4", "cs4_bf16", "azp"):
        wl = bench.Workload(name)
        host = wl.host_inputs()
        out, units = _result_from_oracle(wl, host)
        par = wl.parity(host, out)
        assert par["ok"] and par["max_err"] < par["tol"] / 4, (name, par)
        assert par["tol"] == (1e-5 if wl.dtype == "f32" else 2e-2)
        # plant an error the size of the largest value in the first sampled unit
        bad = out.copy()
        w = wl.w
        first = {"gemm": lambda: units[0] * w["N"], "conv": lambda: units[0] * w["Cout"],
                 "gemm_batched": lambda: units[0] * w["M"] * w["N"],
                 "add_zero_pad": lambda: units[0] * (wl.out_elems // w["N"]) + (w["pad"] * (w["W"] + 2 * w["pad"]) + w["pad"]) * w["C"]}[w["kind"]]()
        if wl.dtype == "f32":
            bad[first] += np.abs(out).max()
        else:
            big = oracle.decode(out, "bf16")
            v = big[first] + np.abs(big).max()
            bad[first] = oracle.round_bf16(np.array([v]))[0]
        assert not wl.parity(host, bad)["ok"], name


def test_traffic_is_reported_only_for_the_captured_tile_configuration():
    cap = bench.TRAFFIC["c2"]["tile_config"]
    same = dict(cap, kernel=1, raster=0)
    b, prov = bench.traffic_for("c2", same)
    assert b == bench.TRAFFIC["c2"]["bytes"] and prov["matches_running_config"] and prov["profile"].startswith("profiles/")
    b, prov = bench.traffic_for("c2", dict(same, tile_n=128))
    assert b is None and not prov["matches_running_config"]
    assert bench.traffic_for("c2", None)[0] is None
    assert bench.traffic_for("c5a", same) == (None, None)
    assert bench.traffic_for("azp", None)[0] == bench.TRAFFIC["azp"]["bytes"]          # no tile configuration to differ


def test_roofline_fractions_use_the_bound_each_workload_names():
    peaks = {"bf16_tflops": 1600.0, "hbm_gbs": 6400.0, "sm_max_mhz": 1965.0}
    r = bench.roofline_of(bench.Workload("c2"), 0.1, peaks, "measured", 148)
    assert r["bound"] == "tensor" and abs(r["achieved"] - 2 * 4096 ** 3 / 1e-4 / 1e12) < 1e-6 and abs(r["frac"] - r["achieved"] / 1600.0) < 1e-12
    r = bench.roofline_of(bench.Workload("c5c"), 0.03, peaks, "measured", 148)
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and abs(r["achieved"] - 138412032 / 3e-5 / 1e9) < 1e-6
    # the paper's fp32 nest is an fp32 problem: reported against the fp32 ALU peak, not the bf16 tensor peak
    r = bench.roofline_of(bench.Workload("cs4"), 0.04, peaks, "measured", 148)
    assert r["bound"] == "alu" and abs(r["peak"] - 2 * 128 * 148 * 1965e6 / 1e12) < 1e-9
    assert bench.roofline_of(bench.Workload("cs4_bf16"), 0.04, peaks, "measured", 148)["bound"] == "tensor"
    assert set(bench.TABLE_ORDER) == set(bench.WORKLOADS)
