"""Split-K summed inside a thread-block cluster (store_mode 3): the split_k CTAs of a tile exchange column slices of
their fp32 partial tiles through distributed shared memory; no workspace, no reduction launch.  The sum runs over the
K slices in ascending order, exactly as the reduction kernel of the workspace path does, so the two agree bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import paper_2409_03864_b200 as tdx
import seeded_inputs as si
from gpu_util import TIGHT, gemm_error, run_gemm

pytestmark = pytest.mark.gpu


def umma(**kw):
    return tdx.tdx_config(kernel=tdx.TDX_KERNEL_UMMA, **kw)


CASES = [
    # M, N, K, tile_n, split_k
    (128, 768, 2048, 192, 3),       # the skinny shape's configuration in small: three slices of 64 columns
    (300, 200, 1000, 128, 2),       # ragged M, N and K
    (256, 512, 4096, 256, 4),
    (128, 128, 8192, 256, 8),       # the largest cluster: eight slices of 32 columns, a tile wider than N
    (1000, 72, 1544, 64, 2),        # N % 8 == 0 but not a multiple of the slice
    (130, 250, 640, 128, 4),        # N % 8 != 0: element-wise stores
]


@pytest.mark.parametrize("transA,transB", [(0, 0), (0, 1), (1, 0), (1, 1)])
@pytest.mark.parametrize("case", CASES)
def test_cluster_reduction_matches_the_oracle_and_the_workspace_path(case, transA, transB):
    M, N, K, tn, sk = case
    if transB == 0 and (tn % 64 or N % 8):
        pytest.skip("N-major B needs 64-column tiles and a 16-byte row pitch")
    if transA == 1 and M % 8:
        pytest.skip("M-major A needs a 16-byte row pitch")
    A, B = si.gemm_bf16_normal(M, N, K, seed=91, transA=transA, transB=transB)
    before = tdx.tdx_kernel_launch_count()
    st, C, ok = run_gemm(M, N, K, transA, transB, -1.0, "bf16", A, B, cfg=umma(tile_m=128, tile_n=tn, split_k=sk, store_mode=3))
    assert st == 0 and ok, tdx.tdx_last_error()
    assert tdx.tdx_kernel_launch_count() - before == 1            # one launch: no reduction kernel
    assert gemm_error(M, N, K, transA, transB, -1.0, "bf16", A, B, C) < TIGHT["bf16"]
    st, need = tdx.tdx_gemm_workspace_size(M, N, K, tdx.TDX_BF16, umma(tile_m=128, tile_n=tn, split_k=sk, store_mode=3))
    assert st == 0 and need == 0
    # the same K slices summed by the reduction kernel from a workspace: same order, same bits
    ws = torch.empty(sk * M * N * 4, dtype=torch.uint8, device="cuda")
    st, C1, ok = run_gemm(M, N, K, transA, transB, -1.0, "bf16", A, B, workspace=ws,
                          cfg=umma(tile_m=128, tile_n=tn, split_k=sk, store_mode=1, stages=3))
    assert st == 0 and ok, tdx.tdx_last_error()
    assert np.array_equal(C, C1)
    assert tdx.tdx_check_device_status() == 0


def test_cluster_reduction_exact_integers():
    M, N, K = 256, 384, 64 * 12
    A = si.small_integers(92, 0, (M, K), "bf16", -1, 1)
    B = si.small_integers(92, 1, (K, N), "bf16", -1, 1)
    st, C, ok = run_gemm(M, N, K, 0, 0, 1.0, "bf16", A, B, cfg=umma(tile_m=128, tile_n=192, split_k=3, store_mode=3))
    assert st == 0 and ok, tdx.tdx_last_error()
    assert np.array_equal(C, oracle.round_bf16(oracle.gemm(M, N, K, 0, 0, 1.0, "bf16", A, B)))


def test_cluster_reduction_many_clusters():
    # more clusters than fit the device at once: they run in waves, one tile per cluster
    M, N, K = 128 * 40, 512, 512
    A, B = si.gemm_bf16_normal(M, N, K, seed=93, transA=0, transB=1)
    st, C, ok = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B, cfg=umma(tile_m=128, tile_n=128, split_k=2, store_mode=3))
    assert st == 0 and ok, tdx.tdx_last_error()
    assert gemm_error(M, N, K, 0, 1, 1.0, "bf16", A, B, C) < TIGHT["bf16"]


@pytest.mark.parametrize("cfg", [dict(tile_m=256, tile_n=128, split_k=2), dict(tile_m=128, tile_n=128, split_k=1),
                                 dict(tile_m=128, tile_n=192, split_k=4), dict(tile_m=128, tile_n=128, split_k=16),
                                 dict(tile_m=128, tile_n=256, split_k=2, fit=2)])
def test_cluster_reduction_constraints(cfg):
    M, N, K = 256, 768, 4096
    A, B = si.gemm_bf16_normal(M, N, K, seed=94, transA=0, transB=1)
    st, _, untouched = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B, cfg=umma(store_mode=3, **cfg))
    assert st == tdx.TDX_ERR_CONFIG and untouched, tdx.tdx_last_error()
