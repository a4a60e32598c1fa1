"""GPU parity of tdx_gemm against the CPU oracle (through the C ABI)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2409_03864_b200 as tdx
import seeded_inputs as si
from gpu_util import TIGHT, TOL, GuardedOut, gemm_error, run_gemm, structured_rows, to_dev

pytestmark = pytest.mark.gpu


def umma(**kw):
    return tdx.tdx_config(kernel=tdx.TDX_KERNEL_UMMA, **kw)


# ------------------------------------------------------------------ fp32 CUDA-core path

def test_fp32_gemm_256_cubed_uniform():
    M = N = K = 256
    A, B = si.gemm_f32_uniform(M, N, K, seed=0)
    st, C, ok = run_gemm(M, N, K, 0, 0, 1.0, "f32", A, B)
    assert st == 0, tdx.tdx_last_error()
    assert ok
    err = gemm_error(M, N, K, 0, 0, 1.0, "f32", A, B, C)
    assert err < TOL["f32"] and err < TIGHT["f32"], err


@pytest.mark.parametrize("transA,transB", [(0, 0), (0, 1), (1, 0), (1, 1)])
@pytest.mark.parametrize("shape", [(1, 1, 1), (33, 65, 17), (130, 70, 257), (64, 64, 64), (300, 500, 40), (100, 76, 204)])
def test_fp32_gemm_shapes_and_transposes(shape, transA, transB):
    M, N, K = shape
    A = si.uniform(10, 0, (K, M) if transA else (M, K), "f32")
    B = si.uniform(10, 1, (N, K) if transB else (K, N), "f32")
    st, C, ok = run_gemm(M, N, K, transA, transB, -0.5, "f32", A, B)
    assert st == 0 and ok, tdx.tdx_last_error()
    assert gemm_error(M, N, K, transA, transB, -0.5, "f32", A, B, C) < TOL["f32"]
    st, Cg, ok = run_gemm(M, N, K, transA, transB, -0.5, "f32", A, B, cfg=tdx.tdx_config(kernel=tdx.TDX_KERNEL_GENERIC))
    assert st == 0 and ok
    assert gemm_error(M, N, K, transA, transB, -0.5, "f32", A, B, Cg) < TOL["f32"]


# ------------------------------------------------------------------ bf16 tensor-core path

def test_umma_single_tile_exact_small_integers():
    # values in {-1, 0, 1} and K = 64: every output is an integer of magnitude <= 64, exact in bf16,
    # so the tensor-core result must equal the oracle bit for bit.
    M, N, K = 128, 128, 64
    A = si.small_integers(50, 0, (M, K), "bf16", -1, 1)
    B = si.small_integers(50, 1, (N, K), "bf16", -1, 1)
    st, C, ok = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B, cfg=umma(tile_n=128, stages=2))
    assert st == 0 and ok, tdx.tdx_last_error()
    ref = oracle.gemm(M, N, K, 0, 1, 1.0, "bf16", A, B)
    got = oracle.decode(C, "bf16")
    bad = np.argwhere(got != ref)
    assert bad.size == 0, f"first mismatches (row, col): {bad[:8].tolist()} got {got[tuple(bad[0])]} want {ref[tuple(bad[0])]}"


@pytest.mark.parametrize("transA,transB", [(0, 1), (0, 0), (1, 1), (1, 0)])
def test_umma_exact_integers_all_layouts(transA, transB):
    M, N, K = 256, 192, 192
    A = si.small_integers(51, 0, (K, M) if transA else (M, K), "bf16", -1, 1)
    B = si.small_integers(51, 1, (N, K) if transB else (K, N), "bf16", -1, 1)
    st, C, ok = run_gemm(M, N, K, transA, transB, 1.0, "bf16", A, B, cfg=umma(tile_n=64, stages=3))
    assert st == 0 and ok, tdx.tdx_last_error()
    ref = oracle.gemm(M, N, K, transA, transB, 1.0, "bf16", A, B)
    got = oracle.decode(C, "bf16")
    bad = np.argwhere(got != ref)
    assert bad.size == 0, f"{bad.shape[0]} mismatches, first (row, col): {bad[:8].tolist()}"


@pytest.mark.parametrize("transA,transB", [(0, 1), (0, 0), (1, 1), (1, 0)])
@pytest.mark.parametrize("shape", [(128, 128, 64), (384, 320, 448), (520, 264, 200), (136, 72, 1032), (8, 8, 8)])
def test_umma_shapes_transposes_and_tails(shape, transA, transB):
    M, N, K = shape
    A, B = si.gemm_bf16_normal(M, N, K, seed=52, transA=transA, transB=transB)
    st, C, ok = run_gemm(M, N, K, transA, transB, -1.0, "bf16", A, B, cfg=umma())
    assert st == 0 and ok, tdx.tdx_last_error()
    err = gemm_error(M, N, K, transA, transB, -1.0, "bf16", A, B, C)
    assert err < TOL["bf16"] and err < TIGHT["bf16"], err


@pytest.mark.parametrize("cfgkw", [
    dict(tile_n=32, stages=2), dict(tile_n=64, stages=8), dict(tile_n=96, stages=3), dict(tile_n=128, stages=7),
    dict(tile_n=256, stages=4), dict(tile_n=256, stages=2, raster=1), dict(tile_n=128, stages=4, raster=2),
    dict(tile_n=64, stages=4, raster=3),
])
def test_umma_explicit_tile_configs(cfgkw):
    M, N, K = 640, 520, 328          # 5 row tiles, ragged N and K tails
    A, B = si.gemm_bf16_normal(M, N, K, seed=53, transB=1)
    st, C, ok = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B, cfg=umma(**cfgkw))
    assert st == 0 and ok, tdx.tdx_last_error()
    err = gemm_error(M, N, K, 0, 1, 1.0, "bf16", A, B, C)
    assert err < TIGHT["bf16"], err


@pytest.mark.parametrize("transA,transB", [(0, 1), (0, 0), (1, 1), (1, 0)])
@pytest.mark.parametrize("cfgkw", [dict(tile_n=256, stages=3), dict(tile_n=128, stages=2), dict(tile_n=64, stages=5),
                                   dict(tile_n=192, stages=2, raster=2)])
def test_umma_256_row_tiles(cfgkw, transA, transB):
    # 256-row tiles: two 128-row halves share each B slice; 2 or 4 TMEM accumulator slots
    M, N, K = 904, 520, 328          # 4 row tiles with a ragged last one, ragged N and K tails
    A, B = si.gemm_bf16_normal(M, N, K, seed=62, transA=transA, transB=transB)
    st, C, ok = run_gemm(M, N, K, transA, transB, 1.0, "bf16", A, B, cfg=umma(tile_m=256, **cfgkw))
    assert st == 0 and ok, tdx.tdx_last_error()
    err = gemm_error(M, N, K, transA, transB, 1.0, "bf16", A, B, C)
    assert err < TIGHT["bf16"], err


@pytest.mark.parametrize("transA,transB", [(0, 1), (0, 0), (1, 1), (1, 0)])
@pytest.mark.parametrize("tile_m", [256, 128])
def test_umma_tile_widths_fitted_to_the_cta_count(tile_m, transA, transB):
    # fit = 2: 256- and 192-column tiles from a host-made table, B arriving in 64-row copies; ragged M, N and K tails
    M, N, K = 3304, 2840, 200
    A, B = si.gemm_bf16_normal(M, N, K, seed=64, transA=transA, transB=transB)
    _, rounds, _, _, _, _ = tdx.tdx_gemm_tile_plan(M, N, K, tile_m, 256, 2, torch.cuda.get_device_properties(0).multi_processor_count)
    assert rounds > 0, "this shape is meant to get a fitted plan"
    st, C, ok = run_gemm(M, N, K, transA, transB, -1.0, "bf16", A, B, cfg=umma(tile_m=tile_m, tile_n=256, raster=2, fit=2))
    assert st == 0 and ok, tdx.tdx_last_error()
    err = gemm_error(M, N, K, transA, transB, -1.0, "bf16", A, B, C)
    assert err < TIGHT["bf16"], err
    # same bits as the uniform grid: the reduction order inside an output element does not depend on the tile width
    st, C1, ok = run_gemm(M, N, K, transA, transB, -1.0, "bf16", A, B, cfg=umma(tile_m=tile_m, tile_n=256, raster=2, fit=1))
    assert st == 0 and ok, tdx.tdx_last_error()
    assert np.array_equal(C, C1)


def test_umma_cta_pairs_with_fitted_tile_widths():
    # the tile table dealt to CTA pairs: each CTA loads its half of a tile's B columns in 32-row copies
    M, N, K = 3304, 2840, 200
    A, B = si.gemm_bf16_normal(M, N, K, seed=66, transA=0, transB=1)
    st, C, ok = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B, cfg=umma(cta_pair=2, tile_n=256, fit=2))
    assert st == 0 and ok, tdx.tdx_last_error()
    err = gemm_error(M, N, K, 0, 1, 1.0, "bf16", A, B, C)
    assert err < TIGHT["bf16"], err
    st, C1, ok = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B, cfg=umma(cta_pair=2, tile_n=256, fit=1))
    assert st == 0 and ok, tdx.tdx_last_error()
    assert np.array_equal(C, C1)
    # exact integers, many tiles per pair
    M, N, K = 256 * 9, 64 * 37, 192
    Ai = si.small_integers(67, 0, (M, K), "bf16", -1, 1)
    Bi = si.small_integers(67, 1, (N, K), "bf16", -1, 1)
    st, C, ok = run_gemm(M, N, K, 0, 1, 1.0, "bf16", Ai, Bi, cfg=umma(cta_pair=2, tile_n=256, fit=2))
    assert st == 0 and ok, tdx.tdx_last_error()
    assert np.array_equal(oracle.decode(C, "bf16"), oracle.gemm(M, N, K, 0, 1, 1.0, "bf16", Ai, Bi))


def test_umma_fitted_tiles_exact_integers_and_direct_stores():
    M, N, K = 256 * 9, 64 * 37, 192
    A = si.small_integers(65, 0, (M, K), "bf16", -1, 1)
    B = si.small_integers(65, 1, (N, K), "bf16", -1, 1)
    ref = oracle.gemm(M, N, K, 0, 1, 1.0, "bf16", A, B)
    for sm in (1, 2):
        st, C, ok = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B, cfg=umma(tile_m=256, tile_n=256, fit=2, store_mode=sm))
        assert st == 0 and ok, tdx.tdx_last_error()
        assert np.array_equal(oracle.decode(C, "bf16"), ref), sm


def test_umma_256_row_tiles_exact_integers_many_tiles_per_cta():
    # more tiles than SMs, so every CTA walks several tiles and the accumulator slots wrap around
    M, N, K = 256 * 20, 64 * 16, 128
    A = si.small_integers(63, 0, (M, K), "bf16", -1, 1)
    B = si.small_integers(63, 1, (N, K), "bf16", -1, 1)
    for cfgkw in (dict(tile_m=256, tile_n=64), dict(tile_m=256, tile_n=256), dict(tile_m=128, tile_n=32)):
        st, C, ok = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B, cfg=umma(**cfgkw))
        assert st == 0 and ok, tdx.tdx_last_error()
        ref = oracle.gemm(M, N, K, 0, 1, 1.0, "bf16", A, B)
        assert np.array_equal(oracle.decode(C, "bf16"), ref), cfgkw


@pytest.mark.parametrize("store_mode", [1, 2])
@pytest.mark.parametrize("cfgkw", [dict(tile_m=128, tile_n=64), dict(tile_m=128, tile_n=256), dict(tile_m=256, tile_n=128),
                                   dict(tile_m=256, tile_n=256), dict(tile_m=128, tile_n=32), dict(tile_m=256, tile_n=96)])
def test_umma_store_modes(cfgkw, store_mode):
    # 1 = 16-byte stores from registers, 2 = staged in shared memory and written by the copy engine;
    # ragged M and N tails exercise the predicated stores / the copy engine's clipping
    M, N, K = 1000, 840, 264
    A, B = si.gemm_bf16_normal(M, N, K, seed=66, transB=1)
    st, C, ok = run_gemm(M, N, K, 0, 1, -1.0, "bf16", A, B, cfg=umma(store_mode=store_mode, **cfgkw))
    assert st == 0 and ok, tdx.tdx_last_error()
    assert gemm_error(M, N, K, 0, 1, -1.0, "bf16", A, B, C) < TIGHT["bf16"]
    if store_mode == 2:
        st, C1, _ = run_gemm(M, N, K, 0, 1, -1.0, "bf16", A, B, cfg=umma(store_mode=1, **cfgkw))
        assert np.array_equal(C, C1)                             # same arithmetic, different way out


@pytest.mark.parametrize("transA,transB", [(0, 1), (0, 0), (1, 1), (1, 0)])
@pytest.mark.parametrize("cfgkw", [dict(tile_n=256), dict(tile_n=128, stages=3), dict(tile_n=256, store_mode=1, raster=2)])
def test_umma_cta_pairs(cfgkw, transA, transB):
    # a cluster of two CTAs per 256-row tile: each stages half of the operands, one thread issues MMAs over both
    M, N, K = 1416, 1160, 392          # ragged last tile in M, N and K; more tiles than CTA pairs along the way
    A, B = si.gemm_bf16_normal(M, N, K, seed=69, transA=transA, transB=transB)
    st, C, ok = run_gemm(M, N, K, transA, transB, -1.0, "bf16", A, B, cfg=umma(cta_pair=2, **cfgkw))
    assert st == 0 and ok, tdx.tdx_last_error()
    assert gemm_error(M, N, K, transA, transB, -1.0, "bf16", A, B, C) < TIGHT["bf16"]
    assert tdx.tdx_check_device_status() == 0


def test_umma_cta_pairs_many_tiles_exact_and_deterministic():
    M, N, K = 256 * 40, 256 * 5, 192       # 200 pair tiles over 74 pairs: accumulator slots wrap around
    A = si.small_integers(70, 0, (M, K), "bf16", -1, 1)
    B = si.small_integers(70, 1, (N, K), "bf16", -1, 1)
    st, C, ok = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B, cfg=umma(cta_pair=2, tile_n=256))
    assert st == 0 and ok, tdx.tdx_last_error()
    rows = structured_rows(M, extra=2, max_blocks=20)
    assert np.array_equal(oracle.decode(C, "bf16")[rows], oracle.gemm(M, N, K, 0, 1, 1.0, "bf16", A, B, rows=rows))
    st, C2, _ = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B, cfg=umma(cta_pair=2, tile_n=256))
    assert np.array_equal(C, C2)
    # a pair needs 256-row tiles and has no split-K: refused, output untouched
    st, _, untouched = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B, cfg=umma(cta_pair=2, tile_m=128))
    assert st == tdx.TDX_ERR_CONFIG and untouched


@pytest.mark.parametrize("cfgkw", [dict(tile_m=128, tile_n=64, stages=3), dict(tile_m=256, tile_n=128, stages=2)])
def test_umma_staggered_k_order(cfgkw):
    # each CTA starts its K loop at a different block: same products, rotated order
    M, N, K = 1536, 1280, 712
    A, B = si.gemm_bf16_normal(M, N, K, seed=64, transB=1)
    st, C, ok = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B, cfg=umma(k_stagger=1, **cfgkw))
    assert st == 0 and ok, tdx.tdx_last_error()
    assert gemm_error(M, N, K, 0, 1, 1.0, "bf16", A, B, C) < TIGHT["bf16"]
    st, C2, _ = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B, cfg=umma(k_stagger=1, **cfgkw))
    assert np.array_equal(C, C2)                                  # still deterministic
    Ai = si.small_integers(65, 0, (M, K), "bf16", -1, 1)
    Bi = si.small_integers(65, 1, (N, K), "bf16", -1, 1)
    st, Ci, ok = run_gemm(M, N, K, 0, 1, 1.0, "bf16", Ai, Bi, cfg=umma(k_stagger=1, split_k=0, **cfgkw))
    assert st == 0 and ok
    assert np.array_equal(oracle.decode(Ci, "bf16"), oracle.gemm(M, N, K, 0, 1, 1.0, "bf16", Ai, Bi))


@pytest.mark.parametrize("split", [2, 3, 5])
@pytest.mark.parametrize("transB", [0, 1])
def test_umma_split_k_with_workspace(split, transB):
    M, N, K = 136, 320, 1280
    A, B = si.gemm_bf16_normal(M, N, K, seed=54, transB=transB)
    cfg = umma(tile_n=64, split_k=split)
    st, need = tdx.tdx_gemm_workspace_size(M, N, K, tdx.TDX_BF16, cfg)
    assert st == 0 and need == split * M * N * 4
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    st, C, ok = run_gemm(M, N, K, 0, transB, -1.0, "bf16", A, B, cfg=cfg, workspace=ws)
    assert st == 0 and ok, tdx.tdx_last_error()
    assert gemm_error(M, N, K, 0, transB, -1.0, "bf16", A, B, C) < TIGHT["bf16"]
    # too small a workspace is refused and leaves C untouched
    small = torch.empty(need - 256, dtype=torch.uint8, device="cuda")
    st, _, untouched = run_gemm(M, N, K, 0, transB, -1.0, "bf16", A, B, cfg=cfg, workspace=small)
    assert st == tdx.TDX_ERR_WORKSPACE and untouched


def test_umma_default_split_k_for_skinny_problem():
    M, N, K = 128, 512, 4096
    st, c = tdx.tdx_default_gemm_config(M, N, K, 0, 0, tdx.TDX_BF16)
    assert st == 0 and c.split_k > 1
    A, B = si.gemm_bf16_normal(M, N, K, seed=55)
    st, C, ok = run_gemm(M, N, K, 0, 0, 1.0, "bf16", A, B)
    assert st == 0 and ok, tdx.tdx_last_error()
    assert gemm_error(M, N, K, 0, 0, 1.0, "bf16", A, B, C) < TIGHT["bf16"]


def test_negate_is_bitwise_sign_flip_and_runs_are_deterministic():
    M, N, K = 384, 256, 512
    A, B = si.gemm_bf16_normal(M, N, K, seed=56, transB=1)
    _, pos, _ = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B)
    _, neg, _ = run_gemm(M, N, K, 0, 1, -1.0, "bf16", A, B)
    _, pos2, _ = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B)
    assert np.array_equal(pos, pos2)
    nz = (pos & 0x7FFF) != 0
    assert np.array_equal(neg[nz], pos[nz] ^ 0x8000)
    # negating A instead of the product gives the same bits (the negate commutes with the matmul)
    An = (A ^ np.uint16(0x8000)).astype(np.uint16)
    _, neg2, _ = run_gemm(M, N, K, 0, 1, 1.0, "bf16", An, B)
    assert np.array_equal(neg2[nz], neg[nz])


def test_transpose_flag_equals_materialised_transpose():
    # reading B^T through the descriptor and multiplying by a materialised copy agree to rounding
    # (bitwise when the hardware sums each K block in the same order, which is what is observed)
    M, N, K = 256, 256, 320
    A, Bt = si.gemm_bf16_normal(M, N, K, seed=57, transB=1)          # Bt stored N x K
    B = np.ascontiguousarray(Bt.T)                                     # stored K x N
    _, c1, _ = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, Bt, cfg=umma(tile_n=128))
    _, c0, _ = run_gemm(M, N, K, 0, 0, 1.0, "bf16", A, B, cfg=umma(tile_n=128))
    d = np.abs(oracle.decode(c1, "bf16") - oracle.decode(c0, "bf16"))
    sc = oracle.gemm_row_scales(M, N, K, 0, 1, 1.0, "bf16", A, Bt)
    assert (d.max(axis=1) / sc).max() < 4e-3
    At = np.ascontiguousarray(A.T)                                     # stored K x M
    _, c2, _ = run_gemm(M, N, K, 1, 1, 1.0, "bf16", At, Bt, cfg=umma(tile_n=128))
    d = np.abs(oracle.decode(c2, "bf16") - oracle.decode(c1, "bf16"))
    assert (d.max(axis=1) / sc).max() < 4e-3


@pytest.mark.parametrize("shape", [(37, 53, 71), (64, 100, 72), (100, 100, 101)])
def test_small_unaligned_shapes_use_the_generic_gpu_kernel(shape):
    # row pitches that are no multiple of 16 bytes, under 2^21 multiply-adds: one launch of the generic kernel
    M, N, K = shape
    A, B = si.gemm_bf16_normal(M, N, K, seed=58)
    n0 = tdx.tdx_kernel_launch_count()
    st, C, ok = run_gemm(M, N, K, 0, 0, 1.0, "bf16", A, B)
    assert st == 0 and ok, tdx.tdx_last_error()
    assert tdx.tdx_kernel_launch_count() == n0 + 1
    assert gemm_error(M, N, K, 0, 0, 1.0, "bf16", A, B, C) < TIGHT["bf16"]
    # asked for explicitly, the generic kernel also serves the large unaligned shape of the paper's Case Study 4
    M, N, K = 196, 256, 2305
    A, B = si.gemm_bf16_normal(M, N, K, seed=58)
    n0 = tdx.tdx_kernel_launch_count()
    st, C, ok = run_gemm(M, N, K, 0, 0, 1.0, "bf16", A, B, cfg=tdx.tdx_config(kernel=tdx.TDX_KERNEL_GENERIC))
    assert st == 0 and ok and tdx.tdx_kernel_launch_count() == n0 + 1
    assert gemm_error(M, N, K, 0, 0, 1.0, "bf16", A, B, C) < TIGHT["bf16"]


def test_n_not_multiple_of_8_takes_scalar_stores():
    M, N, K = 200, 100, 128           # transB=1: only K must be a multiple of 8
    A, B = si.gemm_bf16_normal(M, N, K, seed=59, transB=1)
    st, C, ok = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B, cfg=umma())
    assert st == 0 and ok, tdx.tdx_last_error()
    assert gemm_error(M, N, K, 0, 1, 1.0, "bf16", A, B, C) < TIGHT["bf16"]


def test_infeasible_config_leaves_output_untouched():
    M, N, K = 256, 256, 256
    A, B = si.gemm_bf16_normal(M, N, K, seed=60, transB=1)
    st, _, untouched = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B, cfg=umma(tile_n=48))
    assert st == tdx.TDX_ERR_CONFIG and untouched
    st, _, untouched = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B, cfg=umma(split_k=4))   # no workspace
    assert st == tdx.TDX_ERR_WORKSPACE and untouched


def test_k_zero_fills_zero_and_empty_is_noop():
    out = GuardedOut(12, "bf16")
    assert tdx.tdx_gemm(3, 4, 0, 0, 0, 1.0, tdx.TDX_BF16, None, None, out.ptr) == 0
    torch.cuda.synchronize()
    assert (out.payload() == 0).all() and out.guards_intact()
    out = GuardedOut(12, "bf16")
    assert tdx.tdx_gemm(0, 4, 8, 0, 0, 1.0, tdx.TDX_BF16, None, None, out.ptr) == 0
    torch.cuda.synchronize()
    assert out.untouched()


def test_host_buffer_entry_point():
    M, N, K = 256, 128, 192
    A, B = si.gemm_bf16_normal(M, N, K, seed=61, transB=1)
    C = np.zeros((M, N), dtype=np.uint16)
    st = tdx.tdx_gemm_host(M, N, K, 0, 1, -1.0, tdx.TDX_BF16, A, B, C)
    assert st == 0, tdx.tdx_last_error()
    assert gemm_error(M, N, K, 0, 1, -1.0, "bf16", A, B, C) < TIGHT["bf16"]


@pytest.mark.parametrize("shape", [(2304, 1024, 4096, 1), (4100, 512, 4096, 0)])
def test_host_buffer_entry_point_in_chunks(shape):
    # large enough for the rows to go up, be multiplied and come down chunk by chunk on three streams (two chunks of
    # 1280 + 1024 rows; four of 1280, 1280, 1280 and 260); called twice, the second call on the warm streams
    M, N, K, tB = shape
    A, B = si.gemm_bf16_normal(M, N, K, seed=62, transB=tB)
    ref = None
    for rep in range(2):
        C = np.zeros((M, N), dtype=np.uint16)
        st = tdx.tdx_gemm_host(M, N, K, 0, tB, -1.0, tdx.TDX_BF16, A, B, C)
        assert st == 0, tdx.tdx_last_error()
        if ref is None:
            assert gemm_error(M, N, K, 0, tB, -1.0, "bf16", A, B, C) < TIGHT["bf16"]
            ref = C
        else:
            assert np.array_equal(C, ref)


# ------------------------------------------------------------------ full-size workloads (every output element)

def full_gemm_error(M, N, K, tA, tB, alpha, A, B, C, chunk=1024):
    """Compares EVERY element of C with the oracle, 1024 rows at a time (bounds the fp64 reference's memory)."""
    worst = 0.0
    for r0 in range(0, M, chunk):
        rows = np.arange(r0, min(M, r0 + chunk), dtype=np.int64)
        worst = max(worst, gemm_error(M, N, K, tA, tB, alpha, "bf16", A, B, C, rows=rows))
    return worst


def test_full_size_negated_gemm_with_transposed_right_operand():
    # C = -(A . B^T), bf16, M = N = K = 4096, N(0,1) operands from seed 1, B stored N x K: all 4096 x 4096 outputs
    # of the configuration the benchmark times (the automatic choice) against the oracle
    M = N = K = 4096
    A, B = si.gemm_bf16_normal(M, N, K, seed=1, transB=1)
    st, C, ok = run_gemm(M, N, K, 0, 1, -1.0, "bf16", A, B)
    assert st == 0 and ok, tdx.tdx_last_error()
    err = full_gemm_error(M, N, K, 0, 1, -1.0, A, B, C)
    assert err < TOL["bf16"] and err < TIGHT["bf16"], err
    # property that holds at any size: entries have standard deviation sqrt(K)
    vals = oracle.decode(C[::37], "bf16")
    assert abs(vals.std() / 64.0 - 1.0) < 0.02
    assert tdx.tdx_check_device_status() == 0


@pytest.mark.parametrize("shape", [(1024, 1024, 1024), (128, 8192, 8192), (8192, 128, 8192), (4096, 4096, 512)])
def test_sweep_shapes_default_config(shape):
    # every output element (each shape is under 1e10 multiply-adds for the oracle)
    M, N, K = shape
    A, B = si.gemm_bf16_normal(M, N, K, seed=4)
    st, C, ok = run_gemm(M, N, K, 0, 0, 1.0, "bf16", A, B)
    assert st == 0 and ok, tdx.tdx_last_error()
    err = full_gemm_error(M, N, K, 0, 0, 1.0, A, B, C)
    assert err < TOL["bf16"] and err < TIGHT["bf16"], err
    assert tdx.tdx_check_device_status() == 0


def test_sweep_shape_8192_cubed():
    # 5.5e11 multiply-adds: rows {0, 1, 63, 64, 126, 127} and two seeded rows of EVERY 128-row block, all columns, so
    # that every CTA tile, every TMEM lane-quarter boundary and every column position is looked at (6 % of the output)
    M = N = K = 8192
    A, B = si.gemm_bf16_normal(M, N, K, seed=4)
    st, C, ok = run_gemm(M, N, K, 0, 0, 1.0, "bf16", A, B)
    assert st == 0 and ok, tdx.tdx_last_error()
    rows = structured_rows(M, extra=2, seed=8192)
    assert len(rows) >= 64 * 6
    err = gemm_error(M, N, K, 0, 0, 1.0, "bf16", A, B, C, rows=rows)
    assert err < TOL["bf16"] and err < TIGHT["bf16"], err
    assert tdx.tdx_check_device_status() == 0


# ------------------------------------------------------------------ fp32 on the tensor cores (three bf16 pieces per operand)

@pytest.mark.parametrize("transA,transB", [(0, 0), (0, 1), (1, 0), (1, 1)])
@pytest.mark.parametrize("shape", [(200, 136, 300), (520, 264, 70), (64, 64, 64)])
def test_fp32_gemm_from_bf16_pieces_all_layouts(shape, transA, transB):
    # explicit request (kernel = UMMA with fp32 data): ragged M, N and K; K not a multiple of the 64-deep K block
    M, N, K = shape
    A = si.uniform(68, 0, (K, M) if transA else (M, K), "f32")
    B = si.uniform(68, 1, (N, K) if transB else (K, N), "f32")
    st, C, ok = run_gemm(M, N, K, transA, transB, -1.5, "f32", A, B, cfg=umma())
    assert st == 0 and ok, tdx.tdx_last_error()
    err = gemm_error(M, N, K, transA, transB, -1.5, "f32", A, B, C)
    assert err < TOL["f32"] and err < TIGHT["f32"], err


def test_fp32_gemm_from_bf16_pieces_keeps_all_24_bits():
    # operands whose low significand bits matter: x = 1 + u * 2^-20 -- a two-piece split would lose them.  Compare with the
    # CUDA-core kernel's error on the same problem: the tensor-core path must be in the same class.
    M, N, K = 256, 192, 512
    A = (1.0 + si.uniform(69, 0, (M, K), "f32").astype(np.float64) * 2.0 ** -20).astype(np.float32)
    B = (1.0 + si.uniform(69, 1, (K, N), "f32").astype(np.float64) * 2.0 ** -20).astype(np.float32)
    st, C, ok = run_gemm(M, N, K, 0, 0, 1.0, "f32", A, B, cfg=umma())
    assert st == 0 and ok, tdx.tdx_last_error()
    ref = oracle.gemm(M, N, K, 0, 0, 1.0, "f32", A, B)
    rel = np.abs(C.astype(np.float64) - ref).max() / np.abs(ref).max()
    assert rel < 4e-7, rel                       # a few fp32 ulps of the result; two pieces would give ~1e-5
    st, Cs, ok = run_gemm(M, N, K, 0, 0, 1.0, "f32", A, B, cfg=tdx.tdx_config(kernel=tdx.TDX_KERNEL_SIMT))
    assert st == 0 and ok
    rel_simt = np.abs(Cs.astype(np.float64) - ref).max() / np.abs(ref).max()
    assert rel < 8 * max(rel_simt, 6e-8), (rel, rel_simt)


def test_fp32_gemm_large_takes_the_tensor_cores_automatically():
    M = N = K = 1024
    A, B = si.gemm_f32_uniform(M, N, K, seed=70)
    st, c = tdx.tdx_default_gemm_config(M, N, K, 0, 0, tdx.TDX_F32)
    assert st == 0 and c.kernel == tdx.TDX_KERNEL_UMMA
    st, c1 = tdx.tdx_default_gemm_config(256, 256, 256, 0, 0, tdx.TDX_F32)
    assert st == 0 and c1.kernel == tdx.TDX_KERNEL_SIMT      # the small configuration stays on the CUDA cores
    n0 = tdx.tdx_kernel_launch_count()
    st, C, ok = run_gemm(M, N, K, 0, 0, 1.0, "f32", A, B)
    assert st == 0 and ok, tdx.tdx_last_error()
    assert tdx.tdx_kernel_launch_count() - n0 in (2, 3)       # the piece kernel (both operands), the GEMM, and the fp32 reduction when K is split
    rows = structured_rows(M, max_blocks=4)
    err = gemm_error(M, N, K, 0, 0, 1.0, "f32", A, B, C, rows=rows)
    assert err < TIGHT["f32"], err
    # integer operands: exact
    Ai = si.small_integers(71, 0, (M, K), "f32", -8, 8)
    Bi = si.small_integers(71, 1, (K, N), "f32", -8, 8)
    st, Ci, ok = run_gemm(M, N, K, 0, 0, 1.0, "f32", Ai, Bi)
    assert st == 0 and ok
    assert np.array_equal(Ci[rows].astype(np.float64), oracle.gemm(M, N, K, 0, 0, 1.0, "f32", Ai, Bi, rows=rows))


# ------------------------------------------------------------------ bf16 operands, fp32 result

@pytest.mark.parametrize("transA,transB", [(0, 1), (0, 0), (1, 0), (1, 1)])
@pytest.mark.parametrize("shape", [(384, 320, 448), (130, 72, 1032), (136, 72, 1032), (128, 4096, 2048), (37, 53, 71)])
def test_bf16_gemm_with_fp32_result(shape, transA, transB):
    # the accumulator leaves as fp32: errors are those of fp32 accumulation, far below the bf16 rounding of tdx_gemm;
    # (128, 4096, 2048) takes split-K and the fp32 reduction, (37, 53, 71) the generic kernel (no 16-byte pitches)
    M, N, K = shape
    A, B = si.gemm_bf16_normal(M, N, K, seed=72, transA=transA, transB=transB)
    out = GuardedOut(M * N, "f32")
    st = tdx.tdx_gemm_f32out(M, N, K, transA, transB, -2.0, to_dev(A), to_dev(B), out.ptr)
    torch.cuda.synchronize()
    assert st == 0 and out.guards_intact(), tdx.tdx_last_error()
    err = oracle.max_normalised_error(out.payload().reshape(M, N).astype(np.float64),
                                      oracle.gemm(M, N, K, transA, transB, -2.0, "bf16", A, B),
                                      oracle.gemm_row_scales(M, N, K, transA, transB, -2.0, "bf16", A, B))
    assert err < TIGHT["f32"], err


def test_bf16_gemm_with_fp32_result_exact_integers():
    M, N, K = 520, 264, 320
    A = si.small_integers(73, 0, (M, K), "bf16", -8, 8)
    B = si.small_integers(73, 1, (N, K), "bf16", -8, 8)
    out = GuardedOut(M * N, "f32")
    assert tdx.tdx_gemm_f32out(M, N, K, 0, 1, 1.0, to_dev(A), to_dev(B), out.ptr) == 0
    torch.cuda.synchronize()
    assert out.guards_intact()
    assert np.array_equal(out.payload().reshape(M, N).astype(np.float64), oracle.gemm(M, N, K, 0, 1, 1.0, "bf16", A, B))


@pytest.mark.parametrize("transA,transB", [(0, 0), (0, 1), (1, 0), (1, 1)])
@pytest.mark.parametrize("shape", [(196, 256, 2305), (333, 515, 1001), (130, 70, 257)])
def test_bf16_gemm_with_odd_pitches_takes_the_tensor_cores_through_a_padded_copy(shape, transA, transB):
    # K (or M, N) not a multiple of 8: the copy engine cannot address the operands.  Large enough problems are repacked
    # K-major with K padded and run on the tensor cores (two launches); the smallest one stays on the generic kernel
    M, N, K = shape
    A, B = si.gemm_bf16_normal(M, N, K, seed=74, transA=transA, transB=transB)
    n0 = tdx.tdx_kernel_launch_count()
    st, C, ok = run_gemm(M, N, K, transA, transB, -1.0, "bf16", A, B)
    assert st == 0 and ok, tdx.tdx_last_error()
    launches = tdx.tdx_kernel_launch_count() - n0
    assert launches == (1 if M * N * K < 2 ** 21 else 2) or launches == 3       # 3: the cost model split K
    err = gemm_error(M, N, K, transA, transB, -1.0, "bf16", A, B, C)
    assert err < TIGHT["bf16"], err
    # a misaligned base pointer (2 bytes off a 16-byte boundary) takes the same route
    if M * N * K >= 2 ** 21:
        dA = to_dev(np.concatenate([np.zeros(1, np.uint16), A.ravel()]))
        dB = to_dev(np.concatenate([np.zeros(1, np.uint16), B.ravel()]))
        out = GuardedOut(M * N, "bf16")
        assert tdx.tdx_gemm(M, N, K, transA, transB, -1.0, tdx.TDX_BF16, dA.data_ptr() + 2, dB.data_ptr() + 2, out.ptr) == 0
        torch.cuda.synchronize()
        assert out.guards_intact() and np.array_equal(out.payload().reshape(M, N), C)


# ------------------------------------------------------------------ K blocks dealt evenly to all CTAs (fit = 3)

@pytest.mark.parametrize("transA,transB", [(0, 0), (0, 1), (1, 0), (1, 1)])
@pytest.mark.parametrize("case", [(128, 2048, 4096, 128, 192), (136, 1000, 4100 - 4, 128, 128), (520, 128, 8192, 128, 128),
                                  (256, 768, 2048, 256, 256), (128, 128, 576, 128, 128)])
def test_k_balanced_plan_matches_the_oracle(case, transA, transB):
    # few tiles, long reduction: every CTA gets an even run of (tile, K block) units; tiles cut by a CTA boundary are
    # completed from fp32 partial tiles in ascending K order.  Ragged M, N and K tails; all operand layouts.
    M, N, K, tm, tn = case
    A, B = si.gemm_bf16_normal(M, N, K, seed=75, transA=transA, transB=transB)
    cfg = umma(tile_m=tm, tile_n=tn, fit=3, split_k=1, store_mode=1)
    st, C, ok = run_gemm(M, N, K, transA, transB, -1.0, "bf16", A, B, cfg=cfg)       # the library's own workspace
    assert st == 0 and ok, tdx.tdx_last_error()
    err = gemm_error(M, N, K, transA, transB, -1.0, "bf16", A, B, C)
    assert err < TIGHT["bf16"], err
    # caller's workspace of the reported size: same bits (fixed reduction order); too small a one is refused
    st, need = tdx.tdx_gemm_workspace_size(M, N, K, tdx.TDX_BF16, cfg)
    assert st == 0 and need >= M * N * 4
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    st, C2, ok = run_gemm(M, N, K, transA, transB, -1.0, "bf16", A, B, cfg=cfg, workspace=ws)
    assert st == 0 and ok and np.array_equal(C, C2)
    st, _, untouched = run_gemm(M, N, K, transA, transB, -1.0, "bf16", A, B, cfg=cfg, workspace=ws[:need - 256])
    assert st == tdx.TDX_ERR_WORKSPACE and untouched
    assert tdx.tdx_check_device_status() == 0


def test_k_balanced_plan_exact_integers():
    M, N, K = 128, 1536, 192            # 12 tiles x 3 K blocks on 148 CTAs: pieces of one and two K blocks... snapped to whole tiles
    A = si.small_integers(76, 0, (M, K), "bf16", -1, 1)
    B = si.small_integers(76, 1, (K, N), "bf16", -1, 1)
    st, C, ok = run_gemm(M, N, K, 0, 0, 1.0, "bf16", A, B, cfg=umma(tile_m=128, tile_n=128, fit=3, split_k=1, store_mode=1))
    assert st == 0 and ok, tdx.tdx_last_error()
    assert np.array_equal(oracle.decode(C, "bf16"), oracle.gemm(M, N, K, 0, 0, 1.0, "bf16", A, B))
    M, N, K = 128, 640, 64 * 40         # 5 tiles x 40 K blocks: every tile cut into many pieces
    A = si.small_integers(77, 0, (M, K), "bf16", -1, 1)
    B = si.small_integers(77, 1, (N, K), "bf16", -1, 1)
    # sums of up to 2560 terms are not exact in bf16, so compare after the same single rounding
    st, C, ok = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B, cfg=umma(tile_m=128, tile_n=128, fit=3, split_k=1, store_mode=1))
    assert st == 0 and ok, tdx.tdx_last_error()
    assert np.array_equal(C, oracle.round_bf16(oracle.gemm(M, N, K, 0, 1, 1.0, "bf16", A, B)))
