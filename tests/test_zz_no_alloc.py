"""The allocation-free split-K GEMM entry point, tdx_gemm_splitk_static.

Some users of this library run where device allocation is not allowed once the program is set up:
a server that carved up its memory at start-up, or code that lives inside another framework's
memory pool.  For them the split-K partial sums live in a fixed 16 MiB array inside the library
instead of a cudaMalloc'ed workspace.  This test calls that entry point through the C ABI twice in
a row -- the second call on a different problem, so whatever the first call left in the shared
array must not leak into it -- and checks both results against tdx_gemm_ex with a caller-owned
workspace (same kernels, same fixed reduction order, so the bits must agree) and against the CPU
oracle within the tolerance of the other bf16 tests.

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test.
"""
import numpy as np
import pytest
import torch

import paper_2409_03864_b200 as tdx
import seeded_inputs as si
from gpu_util import TIGHT, GuardedOut, gemm_error, run_gemm, to_dev

pytestmark = pytest.mark.gpu


def run_static(M, N, K, transA, transB, alpha, A, B, tile_n, split_k):
    dA, dB = to_dev(A), to_dev(B)
    out = GuardedOut(M * N, "bf16")
    st = tdx.tdx_gemm_splitk_static(M, N, K, transA, transB, alpha, dA, dB, out.ptr, tile_n, split_k)
    torch.cuda.synchronize()
    return st, out.payload().reshape(M, N), out.guards_intact() if st == 0 else out.untouched()


def test_static_scratch_split_k_matches_workspace_split_k_twice_in_a_row():
    cases = [
        # M,   N,   K,   tA, tB, alpha, tile_n, split
        (264, 328, 1280, 0, 1, -1.0, 64, 3),      # first call: fills a good part of the array
        (136, 200, 1024, 0, 0, 0.5, 64, 2),       # second call: smaller, other layout, stale partials around it
    ]
    for i, (M, N, K, tA, tB, alpha, tile_n, split) in enumerate(cases):
        A, B = si.gemm_bf16_normal(M, N, K, seed=90 + i, transA=tA, transB=tB)
        st, got, ok = run_static(M, N, K, tA, tB, alpha, A, B, tile_n, split)
        assert st == 0 and ok, tdx.tdx_last_error()
        cfg = tdx.tdx_config(kernel=tdx.TDX_KERNEL_UMMA, tile_m=128, tile_n=tile_n, split_k=split)
        ws = torch.empty(split * M * N * 4, dtype=torch.uint8, device="cuda")
        st, ref, ok = run_gemm(M, N, K, tA, tB, alpha, "bf16", A, B, cfg=cfg, workspace=ws)
        assert st == 0 and ok, tdx.tdx_last_error()
        assert np.array_equal(got, ref), f"call {i}: static-scratch result differs from the workspace result"
        assert gemm_error(M, N, K, tA, tB, alpha, "bf16", A, B, got) < TIGHT["bf16"]
    assert tdx.tdx_check_device_status() == 0


def test_static_scratch_rejects_what_does_not_fit_and_leaves_output_untouched():
    M, N, K, split = 1024, 2048, 512, 4                   # 4 * 1024 * 2048 * 4 B = 32 MiB > 16 MiB
    assert split * M * N * 4 > tdx.TDX_STATIC_SCRATCH_BYTES
    A, B = si.gemm_bf16_normal(M, N, K, seed=92, transB=1)
    st, _, untouched = run_static(M, N, K, 0, 1, 1.0, A, B, 128, split)
    assert st == tdx.TDX_ERR_WORKSPACE and untouched
    assert "TDX_STATIC_SCRATCH_BYTES" in tdx.tdx_last_error()
    # a pitch that is not a multiple of 16 bytes is refused, not rerouted
    A, B = si.gemm_bf16_normal(64, 64, 100, seed=93, transB=1)
    st, _, untouched = run_static(64, 64, 100, 0, 1, 1.0, A, B, 64, 2)
    assert st == tdx.TDX_ERR_ALIGNMENT and untouched


def test_static_scratch_call_leaves_free_device_memory_unchanged():
    # the property the entry point exists for: once the library is warm on this device, a call takes no device
    # memory -- not from cudaMalloc, not from a growing cache.  All buffers are made before the measured calls.
    M, N, K, split = 392, 264, 2048, 4
    A, B = si.gemm_bf16_normal(M, N, K, seed=94, transB=1)
    dA, dB = to_dev(A), to_dev(B)
    out = GuardedOut(M * N, "bf16")
    assert tdx.tdx_gemm_splitk_static(M, N, K, 0, 1, 1.0, dA, dB, out.ptr, 64, split) == 0      # warm call
    torch.cuda.synchronize()
    first = out.payload().copy()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        assert tdx.tdx_gemm_splitk_static(M, N, K, 0, 1, 1.0, dA, dB, out.ptr, 64, split) == 0
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, (free0, free1)
    assert np.array_equal(out.payload(), first) and out.guards_intact()
    # a new shape on the warm library allocates nothing either (no per-shape cache behind this entry point)
    M2, N2 = 200, 136
    A2, B2 = si.gemm_bf16_normal(M2, N2, K, seed=95, transB=1)
    dA2, dB2 = to_dev(A2), to_dev(B2)
    out2 = GuardedOut(M2 * N2, "bf16")
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    assert tdx.tdx_gemm_splitk_static(M2, N2, K, 0, 1, 1.0, dA2, dB2, out2.ptr, 64, 2) == 0
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, (free0, free1)
    assert gemm_error(M2, N2, K, 0, 1, 1.0, "bf16", A2, B2, out2.payload().reshape(M2, N2)) < TIGHT["bf16"]
