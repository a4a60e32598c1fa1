"""GPU parity of tdx_gemm_batched (batch-matmul with accumulate) against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
import paper_2409_03864_b200 as tdx
import seeded_inputs as si
from gpu_util import TIGHT, TOL, to_dev

pytestmark = pytest.mark.gpu

DT = {"f32": tdx.TDX_F32, "bf16": tdx.TDX_BF16}


def operands(batch, M, N, K, dtype, seed, transA=0, transB=0, integers=False, span=2):
    gen = (lambda t, sh: si.small_integers(seed, t, sh, dtype, -span, span)) if integers else \
          (lambda t, sh: (si.uniform if dtype == "f32" else si.normal)(seed, t, sh, dtype))
    A = gen(0, (batch, K, M) if transA else (batch, M, K))
    B = gen(1, (batch, N, K) if transB else (batch, K, N))
    C = gen(2, (batch, M, N))
    return A, B, C


def run(batch, M, N, K, tA, tB, alpha, beta, dtype, A, B, C):
    dA, dB, dC = to_dev(A), to_dev(B), to_dev(C)
    st = tdx.tdx_gemm_batched(batch, M, N, K, tA, tB, alpha, beta, DT[dtype], dA, dB, dC)
    torch.cuda.synchronize()
    out = dC.cpu().numpy()
    return st, (out.view(np.uint16) if dtype == "bf16" else out).reshape(batch * M, N)


def error(batch, M, N, K, tA, tB, alpha, beta, dtype, A, B, C, got):
    ref = oracle.gemm_batched(batch, M, N, K, tA, tB, alpha, beta, dtype, A, B, C).reshape(batch * M, N)
    sc = oracle.gemm_batched_row_scales(batch, M, N, K, tA, tB, alpha, beta, dtype, A, B, C)
    return oracle.max_normalised_error(oracle.decode(got, dtype), ref, sc)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_the_papers_batch_matmul_workload(dtype):
    # Case Study 4's loop nest as printed: 6 batches of 196 x 256 x 2305, C += A . B.  K = 2305 breaks every 16-byte
    # rule of the copy engine, so both types first repack their operands K-major with K padded (fp32: as three bf16
    # pieces), then ONE tensor-core launch covers all batches; bf16 sums its K slices inside thread-block clusters, where
    # the old C is added too; fp32 in a reduction launch.
    batch, M, N, K = 6, 196, 256, 2305
    A, B, C = operands(batch, M, N, K, dtype, seed=90)
    n0 = tdx.tdx_kernel_launch_count()
    st, got = run(batch, M, N, K, 0, 0, 1.0, 1.0, dtype, A, B, C)
    assert st == 0, tdx.tdx_last_error()
    # repack, GEMM over all batches, and for fp32 (whose K split of six does not cut the 128 columns into 32-column
    # slices) a reduction launch: no generic kernel
    assert tdx.tdx_kernel_launch_count() - n0 == (2 if dtype == "bf16" else 3)
    err = error(batch, M, N, K, 0, 0, 1.0, 1.0, dtype, A, B, C, got)
    assert err < TOL[dtype] and err < TIGHT[dtype], err


@pytest.mark.parametrize("tA,tB", [(0, 0), (0, 1), (1, 0), (1, 1)])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_batched_exact_integers_all_layouts(dtype, tA, tB):
    # small integers: every path must return the oracle's values exactly (sums stay far below 2^8 .. 2^24)
    batch, M, N, K = 3, 136, 72, 40
    A, B, C = operands(batch, M, N, K, dtype, seed=91, transA=tA, transB=tB, integers=True)
    st, got = run(batch, M, N, K, tA, tB, 1.0, 1.0, dtype, A, B, C)
    assert st == 0, tdx.tdx_last_error()
    ref = oracle.gemm_batched(batch, M, N, K, tA, tB, 1.0, 1.0, dtype, A, B, C).reshape(batch * M, N)
    assert np.array_equal(oracle.decode(got, dtype), ref)


@pytest.mark.parametrize("shape", [(4, 384, 320, 448), (2, 128, 8192, 512), (5, 520, 264, 200), (37, 72, 136, 328)])
@pytest.mark.parametrize("alpha,beta", [(1.0, 1.0), (-0.5, 2.0), (1.0, 0.0)])
@pytest.mark.parametrize("tA,tB", [(0, 1), (0, 0), (1, 0), (1, 1)])
def test_batched_bf16_on_the_tensor_cores(shape, alpha, beta, tA, tB):
    # layouts the copy engine can address: ONE tensor-core launch over all batches straight from the caller's buffers
    # (3-D tensor maps, whatever the transposes); the accumulate term goes through the direct-store epilogue, or
    # through the batched reduction when K is split
    batch, M, N, K = shape
    A, B, C = operands(batch, M, N, K, "bf16", seed=92, transA=tA, transB=tB)
    n0 = tdx.tdx_kernel_launch_count()
    st, got = run(batch, M, N, K, tA, tB, alpha, beta, "bf16", A, B, C)
    assert st == 0, tdx.tdx_last_error()
    assert tdx.tdx_kernel_launch_count() - n0 <= 2
    err = error(batch, M, N, K, tA, tB, alpha, beta, "bf16", A, B, C, got)
    assert err < TIGHT["bf16"], err


@pytest.mark.parametrize("shape", [(3, 130, 70, 1101), (1, 196, 256, 2305), (5, 63, 190, 411), (2, 257, 129, 64)])
@pytest.mark.parametrize("tA,tB", [(0, 0), (0, 1), (1, 0), (1, 1)])
def test_batched_bf16_with_layouts_the_copy_engine_cannot_address(shape, tA, tB):
    # odd K, M or N: row pitches that are no multiple of 16 bytes.  The operands are repacked K-major with K padded
    # (one launch for both), then the same single tensor-core launch; output rows of odd length take scalar stores
    batch, M, N, K = shape
    A, B, C = operands(batch, M, N, K, "bf16", seed=96, transA=tA, transB=tB)
    n0 = tdx.tdx_kernel_launch_count()
    st, got = run(batch, M, N, K, tA, tB, -1.0, 0.5, "bf16", A, B, C)
    assert st == 0, tdx.tdx_last_error()
    assert tdx.tdx_kernel_launch_count() - n0 <= 3
    err = error(batch, M, N, K, tA, tB, -1.0, 0.5, "bf16", A, B, C, got)
    assert err < TIGHT["bf16"], err


@pytest.mark.parametrize("tA,tB", [(0, 0), (0, 1), (1, 0), (1, 1)])
@pytest.mark.parametrize("K", [200, 203])
def test_batched_bf16_exact_integers_on_the_tensor_cores(tA, tB, K):
    # values in {-1, 0, 1}: every sum (and the accumulate term) is an integer below 256, exact in bf16, so the result
    # must equal the oracle bit for bit -- directly addressed (K = 200) and repacked with zero padding (K = 203)
    batch, M, N = 3, 136, 72
    A, B, C = operands(batch, M, N, K, "bf16", seed=97, transA=tA, transB=tB, integers=True, span=1)
    st, got = run(batch, M, N, K, tA, tB, 1.0, 1.0, "bf16", A, B, C)
    assert st == 0, tdx.tdx_last_error()
    ref = oracle.gemm_batched(batch, M, N, K, tA, tB, 1.0, 1.0, "bf16", A, B, C).reshape(batch * M, N)
    bad = np.argwhere(oracle.decode(got, "bf16") != ref)
    assert bad.size == 0, f"{bad.shape[0]} mismatches, first (row, col): {bad[:8].tolist()}"


@pytest.mark.parametrize("gap_a,gap_c", [(16, 8), (7, 5)])
def test_batched_bf16_strides_shared_operand_and_gaps(gap_a, gap_c):
    # strideB = 0 shares one B among the batches; strideA / strideC larger than dense leave gaps that must stay
    # untouched.  Gaps of 16 and 8 elements keep every batch in the copy engine's layout; 7 and 5 do not (repack).
    batch, M, N, K = 4, 200, 136, 264
    A = si.normal(98, 0, (batch, M * K + gap_a), "bf16")
    Bm = si.normal(98, 1, (K, N), "bf16")
    C = si.normal(98, 2, (batch, M * N + gap_c), "bf16")
    dA, dB, dC = to_dev(A), to_dev(Bm), to_dev(C)
    st = tdx.tdx_gemm_batched(batch, M, N, K, 0, 0, 1.0, 1.0, tdx.TDX_BF16, dA, dB, dC, strideA=M * K + gap_a, strideB=0,
                              strideC=M * N + gap_c)
    torch.cuda.synchronize()
    assert st == 0, tdx.tdx_last_error()
    got = dC.cpu().numpy().view(np.uint16)
    assert np.array_equal(got[:, M * N:], C[:, M * N:])                       # gaps untouched
    Bt = np.tile(Bm.ravel(), batch)
    ref = oracle.gemm_batched(batch, M, N, K, 0, 0, 1.0, 1.0, "bf16", A, Bt, C, strideA=M * K + gap_a, strideC=M * N + gap_c)
    sc = oracle.gemm_batched_row_scales(batch, M, N, K, 0, 0, 1.0, 1.0, "bf16", np.ascontiguousarray(A[:, :M * K]), Bt,
                                        np.ascontiguousarray(C[:, :M * N]))
    err = oracle.max_normalised_error(oracle.decode(np.ascontiguousarray(got[:, :M * N]), "bf16").reshape(batch * M, N),
                                      ref.reshape(batch * M, N), sc)
    assert err < TIGHT["bf16"], err


def test_batched_strides_shared_operand_and_gaps():
    # strideB = 0 shares one B among the batches; strideA / strideC larger than dense leave gaps that must stay untouched
    batch, M, N, K = 3, 70, 50, 33
    A = si.uniform(93, 0, (batch, M * K + 7), "f32")
    Bm = si.uniform(93, 1, (K, N), "f32")
    C = si.uniform(93, 2, (batch, M * N + 5), "f32")
    dA, dB, dC = to_dev(A), to_dev(Bm), to_dev(C)
    st = tdx.tdx_gemm_batched(batch, M, N, K, 0, 0, 2.0, -1.0, tdx.TDX_F32, dA, dB, dC, strideA=M * K + 7, strideB=0,
                              strideC=M * N + 5)
    torch.cuda.synchronize()
    assert st == 0, tdx.tdx_last_error()
    got = dC.cpu().numpy()
    ref = oracle.gemm_batched(batch, M, N, K, 0, 0, 2.0, -1.0, "f32", A, np.tile(Bm.ravel(), batch), C,
                              strideA=M * K + 7, strideC=M * N + 5)
    assert np.array_equal(got[:, M * N:], C[:, M * N:])                       # gaps untouched
    sc = oracle.gemm_batched_row_scales(batch, M, N, K, 0, 0, 2.0, -1.0, "f32", A[:, :M * K], np.tile(Bm.ravel(), batch),
                                        C[:, :M * N])
    err = oracle.max_normalised_error(got[:, :M * N].reshape(batch * M, N).astype(np.float64), ref.reshape(batch * M, N), sc)
    assert err < TIGHT["f32"], err


def test_batched_edge_cases():
    M, N, K = 16, 24, 8
    A, B, C = operands(2, M, N, K, "f32", seed=94)
    dA, dB, dC = to_dev(A), to_dev(B), to_dev(C)
    # empty batch / empty output: no-op
    assert tdx.tdx_gemm_batched(0, M, N, K, 0, 0, 1.0, 1.0, tdx.TDX_F32, dA, dB, dC) == 0
    assert tdx.tdx_gemm_batched(2, 0, N, K, 0, 0, 1.0, 1.0, tdx.TDX_F32, dA, dB, dC) == 0
    torch.cuda.synchronize()
    assert np.array_equal(dC.cpu().numpy(), C)
    # K = 0: C = beta * C
    assert tdx.tdx_gemm_batched(2, M, N, 0, 0, 0, 1.0, 0.5, tdx.TDX_F32, dA, dB, dC) == 0
    torch.cuda.synchronize()
    assert np.array_equal(dC.cpu().numpy(), np.float32(0.5) * C)
    # overlapping outputs and negative strides are refused before anything runs
    assert tdx.tdx_gemm_batched(2, M, N, K, 0, 0, 1.0, 1.0, tdx.TDX_F32, dA, dB, dC, strideC=M * N - 1) == tdx.TDX_ERR_INVALID_ARG
    assert tdx.tdx_gemm_batched(2, M, N, K, 0, 0, 1.0, 1.0, tdx.TDX_F32, dA, dB, dC, strideA=-1) == tdx.TDX_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert np.array_equal(dC.cpu().numpy(), np.float32(0.5) * C)


@pytest.mark.parametrize("shape", [(6, 196, 256, 2305), (3, 130, 70, 1100), (5, 64, 192, 4100)])
@pytest.mark.parametrize("tA,tB", [(0, 0), (1, 1)])
def test_batched_fp32_on_the_tensor_cores_in_one_launch(shape, tA, tB):
    # fp32 batches large enough for the bf16-piece path: one piece kernel, ONE tensor-core launch over all batches
    # (3-D operands; rows past M or N of a batch must read as zero, not as the next batch) and one fp32 reduction
    batch, M, N, K = shape
    A, B, C = operands(batch, M, N, K, "f32", seed=95, transA=tA, transB=tB)
    n0 = tdx.tdx_kernel_launch_count()
    st, got = run(batch, M, N, K, tA, tB, 0.5, -1.0, "f32", A, B, C)
    assert st == 0, tdx.tdx_last_error()
    assert tdx.tdx_kernel_launch_count() - n0 <= 3
    err = error(batch, M, N, K, tA, tB, 0.5, -1.0, "f32", A, B, C, got)
    assert err < TIGHT["f32"], err


def test_one_batch_without_accumulate_takes_the_automatic_configuration():
    # batch = 1, beta = 0 is the plain GEMM: whatever configuration the library picks for tdx_gemm (for this shape,
    # which the shipped tuning cache does not list, the cost model's: a CTA pair) runs, in one launch, same bits
    batch, M, N, K = 1, 2048, 2048, 2048
    st, cfg = tdx.tdx_default_gemm_config(M, N, K, 0, 1, tdx.TDX_BF16)
    assert st == 0 and cfg.kernel == tdx.TDX_KERNEL_UMMA
    A, B, C = operands(batch, M, N, K, "bf16", seed=97, transB=1)
    n0 = tdx.tdx_kernel_launch_count()
    st, got = run(batch, M, N, K, 0, 1, 1.0, 0.0, "bf16", A, B, C)
    assert st == 0, tdx.tdx_last_error()
    assert tdx.tdx_kernel_launch_count() - n0 == 1
    dA, dB = to_dev(A), to_dev(B)
    dC = torch.zeros(M * N, dtype=torch.int16, device="cuda")
    assert tdx.tdx_gemm(M, N, K, 0, 1, 1.0, tdx.TDX_BF16, dA, dB, dC) == 0
    torch.cuda.synchronize()
    assert np.array_equal(got.reshape(-1), dC.cpu().numpy().view(np.uint16))
    rows = [0, 1, 127, 128, 1000, 2047]
    ref = oracle.gemm(M, N, K, 0, 1, 1.0, "bf16", A[0], B[0], rows=rows)
    sc = oracle.gemm_row_scales(M, N, K, 0, 1, 1.0, "bf16", A[0], B[0], rows=rows)
    assert oracle.max_normalised_error(oracle.decode(got, "bf16")[rows], ref, sc) < TIGHT["bf16"]
