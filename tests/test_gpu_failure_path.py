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
