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
    # M, N, K, tile_n, split_k, tile_m
    (128, 768, 2048, 192, 3, 128),       # the skinny shape's configuration in small: three slices of 64 columns
    (300, 200, 1000, 128, 2, 128),       # ragged M, N and K
    (256, 512, 4096, 256, 4, 128),
    (128, 128, 8192, 256, 8, 128),       # the largest cluster: eight slices of 32 columns, a tile wider than N
    (1000, 72, 1544, 64, 2, 128),        # N % 8 == 0 but not a multiple of the slice
    (130, 250, 640, 128, 4, 128),        # N % 8 != 0: element-wise stores
    (700, 384, 2048, 128, 2, 256),       # 256-row tiles: two accumulator halves per CTA, ragged last tile
    (196, 256, 2368, 256, 4, 256),       # one 256-row tile taller than M
]


@pytest.mark.parametrize("transA,transB", [(0, 0), (0, 1), (1, 0), (1, 1)])
@pytest.mark.parametrize("case", CASES)
def test_cluster_reduction_matches_the_oracle_and_the_workspace_path(case, transA, transB):
    M, N, K, tn, sk, tm = case
    if transB == 0 and (tn % 64 or N % 8):
        pytest.skip("N-major B needs 64-column tiles and a 16-byte row pitch")
    if transA == 1 and M % 8:
        pytest.skip("M-major A needs a 16-byte row pitch")
    A, B = si.gemm_bf16_normal(M, N, K, seed=91, transA=transA, transB=transB)
    before = tdx.tdx_kernel_launch_count()
    st, C, ok = run_gemm(M, N, K, transA, transB, -1.0, "bf16", A, B, cfg=umma(tile_m=tm, tile_n=tn, split_k=sk, store_mode=3))
    assert st == 0 and ok, tdx.tdx_last_error()
    assert tdx.tdx_kernel_launch_count() - before == 1            # one launch: no reduction kernel
    assert gemm_error(M, N, K, transA, transB, -1.0, "bf16", A, B, C) < TIGHT["bf16"]
    st, need = tdx.tdx_gemm_workspace_size(M, N, K, tdx.TDX_BF16, umma(tile_m=tm, tile_n=tn, split_k=sk, store_mode=3))
    assert st == 0 and need == 0
    # the same K slices summed by the reduction kernel from a workspace: same order, same bits
    ws = torch.empty(sk * M * N * 4, dtype=torch.uint8, device="cuda")
    st, C1, ok = run_gemm(M, N, K, transA, transB, -1.0, "bf16", A, B, workspace=ws,
                          cfg=umma(tile_m=tm, tile_n=tn, split_k=sk, store_mode=1, stages=2 if tm == 256 and tn == 256 else 3))
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


@pytest.mark.parametrize("cfg", [dict(tile_m=256, tile_n=256, split_k=2, cta_pair=2), dict(tile_m=128, tile_n=128, split_k=1),
                                 dict(tile_m=128, tile_n=192, split_k=4), dict(tile_m=128, tile_n=128, split_k=16),
                                 dict(tile_m=128, tile_n=256, split_k=2, fit=2)])
def test_cluster_reduction_constraints(cfg):
    M, N, K = 256, 768, 4096
    A, B = si.gemm_bf16_normal(M, N, K, seed=94, transA=0, transB=1)
    st, _, untouched = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B, cfg=umma(store_mode=3, **cfg))
    assert st == tdx.TDX_ERR_CONFIG and untouched, tdx.tdx_last_error()


def test_cluster_reduction_fp32_result_from_bf16_pieces():
    # the fp32 GEMM on the tensor cores (three bf16 pieces per operand) with its K split summed inside clusters: the
    # summed slice leaves as 32 x 32 fp32 blocks through the copy engine; two launches (piece split, GEMM)
    M, N, K = 300, 200, 1000
    A = si.uniform(95, 0, (M, K), "f32")
    B = si.uniform(95, 1, (K, N), "f32")
    before = tdx.tdx_kernel_launch_count()
    st, C, ok = run_gemm(M, N, K, 0, 0, -0.5, "f32", A, B, cfg=umma(tile_m=128, tile_n=128, split_k=2, store_mode=3))
    assert st == 0 and ok, tdx.tdx_last_error()
    assert tdx.tdx_kernel_launch_count() - before == 2
    assert gemm_error(M, N, K, 0, 0, -0.5, "f32", A, B, C) < TIGHT["f32"]
    assert tdx.tdx_check_device_status() == 0


_FORCED_CHILD = r"""
import numpy as np, torch
import paper_2409_03864_b200 as tdx, seeded_inputs as si, oracle
from gpu_util import to_dev, TIGHT
batch, M, N, K = 3, 200, 256, 2048
A = si.normal(96, 0, (batch, M, K), "bf16"); B = si.normal(96, 1, (batch, N, K), "bf16"); C = si.normal(96, 2, (batch, M, N), "bf16")
dA, dB, dC = to_dev(A), to_dev(B), to_dev(C)
n0 = tdx.tdx_kernel_launch_count()
st = tdx.tdx_gemm_batched(batch, M, N, K, 0, 1, 0.5, -1.0, tdx.TDX_BF16, dA, dB, dC)
torch.cuda.synchronize()
assert st == 0, tdx.tdx_last_error()
launches = tdx.tdx_kernel_launch_count() - n0
got = dC.cpu().numpy().view(np.uint16).reshape(batch * M, N)
ref = oracle.gemm_batched(batch, M, N, K, 0, 1, 0.5, -1.0, "bf16", A, B, C).reshape(batch * M, N)
sc = oracle.gemm_batched_row_scales(batch, M, N, K, 0, 1, 0.5, -1.0, "bf16", A, B, C)
err = oracle.max_normalised_error(oracle.decode(got, "bf16"), ref, sc)
assert tdx.tdx_check_device_status() == 0
print("FORCED_OK", launches, err / TIGHT["bf16"])
"""


def test_cluster_reduction_batched_with_accumulate_term():
    """A batch with an accumulate term whose K split (pinned from the environment) is summed inside clusters: the batch
    offset and beta * C are applied where the slice is summed, one launch in all."""
    import os
    import subprocess
    import sys
    env = dict(os.environ, TDX_FORCE_CONFIG="tile_m=128,tile_n=128,split_k=2")
    here = os.path.dirname(os.path.abspath(__file__))
    env["PYTHONPATH"] = os.pathsep.join([os.path.dirname(here), here, env.get("PYTHONPATH", "")])
    out = subprocess.run([sys.executable, "-c", _FORCED_CHILD], env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stdout + out.stderr
    line = [l for l in out.stdout.splitlines() if l.startswith("FORCED_OK")][0].split()
    assert int(line[1]) == 1 and float(line[2]) < 1.0, line


@pytest.mark.parametrize("shape", [(384, 512, 2048, 0, 0), (520, 392, 1536, 1, 1), (128, 2048, 4096, 0, 1)])
def test_every_family_of_the_search_space_matches_the_oracle(shape):
    """Whatever the search may time must also be right: one candidate of every (tile, split, store mode, pair, fit,
    K order) family that the library enumerates for the shape runs and is compared with the oracle -- the in-cluster
    split-K of every legal cluster size among them."""
    M, N, K, tA, tB = shape
    st, cands = tdx.tdx_enum_gemm_configs(M, N, K, tA, tB, tdx.TDX_BF16)
    assert st == 0 and cands
    A, B = si.gemm_bf16_normal(M, N, K, seed=98, transA=tA, transB=tB)
    ref = oracle.gemm(M, N, K, tA, tB, 1.0, "bf16", A, B)
    sc = oracle.gemm_row_scales(M, N, K, tA, tB, 1.0, "bf16", A, B)
    seen, in_cluster = set(), 0
    for c in cands:
        fam = (c["tile_m"], c["tile_n"], c["split_k"], c["store_mode"], c["cta_pair"], c["fit"], c["k_stagger"])
        if fam in seen:
            continue
        seen.add(fam)
        cfg = tdx.tdx_config(**c)
        ws = None
        if c["split_k"] > 1 and c["store_mode"] != 3:
            ws = torch.empty(c["split_k"] * M * N * 4, dtype=torch.uint8, device="cuda")
        st, C, ok = run_gemm(M, N, K, tA, tB, 1.0, "bf16", A, B, cfg=cfg, workspace=ws)
        assert st == 0 and ok, (fam, tdx.tdx_last_error())
        err = oracle.max_normalised_error(oracle.decode(C, "bf16").reshape(M, N), ref, sc)
        assert err < TIGHT["bf16"], (fam, err)
        in_cluster += c["store_mode"] == 3
    assert len(seen) >= 10 and in_cluster >= 1
    assert tdx.tdx_check_device_status() == 0
