"""The device-side failure path, exercised without faulting the GPU: a wait that nothing satisfies runs into its
limit, the kernel returns normally with a code in the status word, the host reports it once, and the context is
still good for real work afterwards."""
import pytest

import paper_2409_03864_b200 as tdx
import seeded_inputs as si
from gpu_util import TIGHT, gemm_error, run_gemm

pytestmark = pytest.mark.gpu


def test_bounded_wait_times_out_and_reports_once():
    assert tdx.tdx_check_device_status() == tdx.TDX_OK
    assert tdx.tdx_selftest_bounded_wait(200) == tdx.TDX_OK          # the launch itself succeeds
    assert tdx.tdx_check_device_status() == tdx.TDX_ERR_TIMEOUT     # ... and the wait that ran out is reported
    assert "bounded wait" in tdx.tdx_last_error()
    assert tdx.tdx_check_device_status() == tdx.TDX_OK              # reported once, then cleared
    # the context is intact: a real GEMM still runs and is right
    M, N, K = 256, 256, 256
    A, B = si.gemm_bf16_normal(M, N, K, seed=95, transB=1)
    st, C, ok = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B)
    assert st == 0 and ok
    assert gemm_error(M, N, K, 0, 1, 1.0, "bf16", A, B, C) < TIGHT["bf16"]


def test_selftest_argument_check():
    assert tdx.tdx_selftest_bounded_wait(0) == tdx.TDX_ERR_INVALID_ARG
    assert tdx.tdx_selftest_bounded_wait(10 ** 7) == tdx.TDX_ERR_INVALID_ARG


def test_bounds_check_selftest_reports_once_and_skips_the_access():
    """The bounds-checked debug mode of the one-thread-per-output kernels: told an extent four elements short, the kernel
    refuses those indices (nothing outside the real buffers is touched), records it, and the host reports it once."""
    assert tdx.tdx_check_device_status() == tdx.TDX_OK
    assert tdx.tdx_selftest_bounds_check() == tdx.TDX_OK
    assert tdx.tdx_check_device_status() == tdx.TDX_ERR_BOUNDS
    assert "bounds" in tdx.tdx_last_error()
    assert tdx.tdx_check_device_status() == tdx.TDX_OK


_BOUNDS_CHILD = r"""
import numpy as np, torch
import paper_2409_03864_b200 as tdx, seeded_inputs as si, oracle
from gpu_util import run_gemm, run_conv, gemm_error, conv_error, TIGHT
cfg = tdx.tdx_config(kernel=tdx.TDX_KERNEL_GENERIC)
worst = 0.0
for (M, N, K, tA, tB) in [(67, 45, 131, 0, 0), (33, 130, 70, 1, 1), (129, 17, 64, 0, 1), (5, 7, 300, 1, 0)]:
    A, B = si.gemm_bf16_normal(M, N, K, seed=5, transA=tA, transB=tB)
    st, C, ok = run_gemm(M, N, K, tA, tB, -1.0, "bf16", A, B, cfg=cfg)
    assert st == 0 and ok, (st, tdx.tdx_last_error())
    worst = max(worst, gemm_error(M, N, K, tA, tB, -1.0, "bf16", A, B, C) / TIGHT["bf16"])
for (H, W, Cin, Cout, R, pad, stride) in [(9, 11, 5, 7, 3, 1, 1), (10, 9, 8, 16, 3, 1, 2), (6, 6, 3, 4, 1, 0, 1)]:
    x, w, b = si.conv_bf16(2, H, W, Cin, Cout, R, R, seed=6)
    st, y, ok = run_conv(2, H, W, Cin, Cout, R, R, pad, stride, "bf16", x, w, b, 1, cfg=cfg)
    assert st == 0 and ok, (st, tdx.tdx_last_error())
    worst = max(worst, conv_error(2, H, W, Cin, Cout, R, R, pad, stride, "bf16", x, w, b, 1, y) / TIGHT["bf16"])
assert tdx.tdx_check_device_status() == tdx.TDX_OK, tdx.tdx_last_error()
print("BOUNDS_OK", worst)
"""


def test_debug_bounds_mode_is_silent_on_valid_calls():
    """TDX_DEBUG_BOUNDS=1 checks every index of the one-thread-per-output kernels against the extent the shapes imply: on
    valid calls (all four layouts, ragged sizes, strided and 1 x 1 convolutions) nothing may fire and results are unchanged."""
    import os
    import subprocess
    import sys
    env = dict(os.environ, TDX_DEBUG_BOUNDS="1")
    here = os.path.dirname(os.path.abspath(__file__))
    env["PYTHONPATH"] = os.pathsep.join([os.path.dirname(here), here, env.get("PYTHONPATH", "")])
    out = subprocess.run([sys.executable, "-c", _BOUNDS_CHILD], env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stdout + out.stderr
    line = [l for l in out.stdout.splitlines() if l.startswith("BOUNDS_OK")][0]
    assert float(line.split()[1]) < 1.0
