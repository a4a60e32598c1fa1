"""Pins of the error-metric scales (oracle/metric.py) against plain Python loops.

The scales are the denominators of every GPU parity test: a scale that came out too large would loosen the
tests that divide by it without anything else noticing.  Each function is recomputed here element by element
from its definition -- scale_i = |alpha| * ||op(A)(i,:)|| * max_j ||op(B)(:,j)|| (+ the accumulate and residual
terms) -- with explicit index arithmetic on the flat storage, for every operand layout, stride and optional term.
"""
import math

import numpy as np
import pytest

import oracle
import seeded_inputs as si


def _val(flat, idx, dtype):
    return float(oracle.decode(np.asarray(flat).reshape(-1)[idx:idx + 1], dtype)[0])


def _gemm_scales_by_loops(M, N, K, tA, tB, alpha, dtype, A, B):
    a = oracle.decode(np.asarray(A).reshape(-1), dtype)
    b = oracle.decode(np.asarray(B).reshape(-1), dtype)
    a_norm = []
    for i in range(M):
        s = 0.0
        for k in range(K):
            v = a[k * M + i] if tA else a[i * K + k]
            s += v * v
        a_norm.append(math.sqrt(s))
    b_max = 0.0
    for j in range(N):
        s = 0.0
        for k in range(K):
            v = b[j * K + k] if tB else b[k * N + j]
            s += v * v
        b_max = max(b_max, math.sqrt(s))
    return np.array([abs(alpha) * an * b_max for an in a_norm])


@pytest.mark.parametrize("tA,tB", [(0, 0), (0, 1), (1, 0), (1, 1)])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_gemm_row_scales_every_layout(tA, tB, dtype):
    M, N, K, alpha = 5, 7, 11, -1.5       # all different: a swapped axis changes the answer's length or value
    if dtype == "bf16":
        A, B = si.gemm_bf16_normal(M, N, K, seed=60 + 2 * tA + tB, transA=tA, transB=tB)
    else:
        A = si.uniform(61, 0, (K, M) if tA else (M, K), "f32")
        B = si.uniform(61, 1, (N, K) if tB else (K, N), "f32")
    # make one row of op(A) and one column of op(B) stand out, so that a norm taken over the wrong axis differs
    got = oracle.gemm_row_scales(M, N, K, tA, tB, alpha, dtype, A, B)
    want = _gemm_scales_by_loops(M, N, K, tA, tB, alpha, dtype, A, B)
    assert got.shape == (M,)
    assert np.allclose(got, want, rtol=1e-13, atol=0.0)
    rows = [4, 0, 2]
    assert np.array_equal(oracle.gemm_row_scales(M, N, K, tA, tB, alpha, dtype, A, B, rows=rows), got[rows])
    # the scale bounds every |C[i,j]| (Cauchy-Schwarz) and is attained up to the angle: not a loose constant
    ref = oracle.gemm(M, N, K, tA, tB, alpha, dtype, A, B)
    assert (np.abs(ref) <= got[:, None] * (1 + 1e-12)).all()


def test_gemm_row_scales_axis_sensitivity():
    # A with one large row, B with one large column: the per-row scale must follow A's rows, not its columns
    M, N, K = 3, 4, 6
    A = np.ones((M, K), dtype=np.float32)
    A[1, :] = 10.0
    B = np.ones((K, N), dtype=np.float32)
    B[:, 2] = 3.0
    sc = oracle.gemm_row_scales(M, N, K, 0, 0, 1.0, "f32", A, B)
    assert np.allclose(sc, [math.sqrt(6) * 3 * math.sqrt(6), 10 * math.sqrt(6) * 3 * math.sqrt(6), math.sqrt(6) * 3 * math.sqrt(6)])
    # the same matrices stored transposed give the same scales
    sc_t = oracle.gemm_row_scales(M, N, K, 1, 1, 1.0, "f32", np.ascontiguousarray(A.T), np.ascontiguousarray(B.T))
    assert np.allclose(sc, sc_t, rtol=1e-14)


@pytest.mark.parametrize("tA,tB", [(0, 0), (0, 1), (1, 0), (1, 1)])
@pytest.mark.parametrize("beta", [0.0, 1.0, -0.5])
def test_gemm_batched_row_scales_by_loops(tA, tB, beta):
    batch, M, N, K, alpha = 3, 4, 5, 6, 2.0
    A = si.uniform(70, 0, (batch, K, M) if tA else (batch, M, K), "f32")
    B = si.uniform(70, 1, (batch, N, K) if tB else (batch, K, N), "f32")
    # batches of very different magnitude: a maximum taken over all batches instead of per batch would show
    B[1] *= 8.0
    C = si.uniform(70, 2, (batch, M, N), "f32")
    C[2] *= 5.0
    got = oracle.gemm_batched_row_scales(batch, M, N, K, tA, tB, alpha, beta, "f32", A, B, C)
    assert got.shape == (batch * M,)
    c = np.asarray(C, dtype=np.float64)
    for b in range(batch):
        one = _gemm_scales_by_loops(M, N, K, tA, tB, alpha, "f32", A[b], B[b])
        for i in range(M):
            want = one[i]
            if beta != 0.0:
                want += abs(beta) * max(abs(c[b, i, j]) for j in range(N))
            assert abs(got[b * M + i] - want) <= 1e-12 * max(1.0, want), (b, i)
    # one batch, no accumulate term: the plain GEMM scales
    assert np.allclose(oracle.gemm_batched_row_scales(1, M, N, K, tA, tB, alpha, 0.0, "f32", A[0], B[0]),
                       oracle.gemm_row_scales(M, N, K, tA, tB, alpha, "f32", A[0], B[0]), rtol=1e-14)
    # the scale bounds the result, accumulate term included
    ref = oracle.gemm_batched(batch, M, N, K, tA, tB, alpha, beta, "f32", A, B, C if beta != 0.0 else None)
    assert (np.abs(ref).reshape(batch * M, N) <= got[:, None] * (1 + 1e-12)).all()


def test_gemm_batched_row_scales_bf16_storage():
    batch, M, N, K = 2, 3, 4, 8
    A = si.normal(71, 0, (batch, M, K), "bf16")
    B = si.normal(71, 1, (batch, K, N), "bf16")
    C = si.normal(71, 2, (batch, M, N), "bf16")
    got = oracle.gemm_batched_row_scales(batch, M, N, K, 0, 0, 1.0, 1.0, "bf16", A, B, C)
    cd = oracle.decode(C, "bf16").reshape(batch, M, N)
    for b in range(batch):
        one = _gemm_scales_by_loops(M, N, K, 0, 0, 1.0, "bf16", A[b], B[b])
        for i in range(M):
            assert abs(got[b * M + i] - (one[i] + np.abs(cd[b, i]).max())) < 1e-12


def _conv_scales_by_loops(N, H, W, Cin, Cout, R, S, pad, stride, x, w, bias, residual):
    xd = oracle.decode(x, "bf16").reshape(N, H, W, Cin)
    wd = oracle.decode(w, "bf16").reshape(Cout, R * S * Cin)
    wmax = max(math.sqrt(float((wd[k] ** 2).sum())) for k in range(Cout))
    bmax = 0.0 if bias is None else max(abs(float(v)) for v in bias)
    P = (H + 2 * pad - R) // stride + 1
    Q = (W + 2 * pad - S) // stride + 1
    rd = None if residual is None else oracle.decode(residual, "bf16").reshape(N, P, Q, Cout)
    out = []
    for n in range(N):
        for p in range(P):
            for q in range(Q):
                e = 0.0
                for r in range(R):
                    for s in range(S):
                        h, ww = p * stride + r - pad, q * stride + s - pad
                        if 0 <= h < H and 0 <= ww < W:
                            for c in range(Cin):
                                e += float(xd[n, h, ww, c]) ** 2
                v = math.sqrt(e) * wmax + bmax
                if rd is not None:
                    v += max(abs(float(t)) for t in rd[n, p, q])
                out.append(v)
    return np.array(out)


@pytest.mark.parametrize("H,W,R,S,pad,stride", [
    (7, 6, 3, 3, 1, 2),      # stride 2, odd and even sizes
    (8, 9, 3, 3, 1, 3),      # stride 3
    (6, 7, 1, 1, 0, 2),      # 1 x 1, stride 2
    (5, 5, 3, 2, 2, 2),      # non-square filter, pad 2
    (5, 6, 3, 3, 1, 1),      # stride 1 (already pinned elsewhere; kept as the baseline of this loop)
])
@pytest.mark.parametrize("with_residual", [False, True])
@pytest.mark.parametrize("with_bias", [True, False])
def test_conv_row_scales_stride_and_residual(H, W, R, S, pad, stride, with_residual, with_bias):
    N, Cin, Cout = 2, 3, 4
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, R, S, seed=80 + stride)
    if not with_bias:
        b = None
    P = (H + 2 * pad - R) // stride + 1
    Q = (W + 2 * pad - S) // stride + 1
    res = si.normal(81, 3, (N * P * Q, Cout), "bf16") if with_residual else None
    got = oracle.conv_row_scales(N, H, W, Cin, Cout, R, S, pad, stride, "bf16", x, w, b, residual=res)
    want = _conv_scales_by_loops(N, H, W, Cin, Cout, R, S, pad, stride, x, w, b, res)
    assert got.shape == (N * P * Q,)
    assert np.allclose(got, want, rtol=1e-12, atol=1e-14)
    rows = [N * P * Q - 1, 0, 3]
    assert np.array_equal(oracle.conv_row_scales(N, H, W, Cin, Cout, R, S, pad, stride, "bf16", x, w, b, rows=rows,
                                                 residual=res), got[rows])
    # the scale bounds the result
    ref = oracle.conv2d(N, H, W, Cin, Cout, R, S, pad, stride, "bf16", x, w, b, 0, residual=res)
    assert (np.abs(ref) <= got[:, None] * (1 + 1e-12)).all()


def test_conv_row_scales_strided_window_positions():
    # one bright pixel: exactly the output pixels whose strided window covers it carry its energy
    N, H, W, Cin, Cout, R, S, pad, stride = 1, 7, 7, 1, 1, 3, 3, 1, 2
    x = np.zeros((N, H, W, Cin), dtype=np.float32)
    x[0, 4, 2, 0] = 2.0
    xb = si.f32_to_bf16_bits(x)
    w = si.f32_to_bf16_bits(np.ones((Cout, R, S, Cin), dtype=np.float32))
    sc = oracle.conv_row_scales(N, H, W, Cin, Cout, R, S, pad, stride, "bf16", xb, w, None).reshape(4, 4)
    for p in range(4):
        for q in range(4):
            covered = (p * 2 - 1 <= 4 <= p * 2 + 1) and (q * 2 - 1 <= 2 <= q * 2 + 1)
            assert sc[p, q] == pytest.approx(2.0 * 3.0 if covered else 0.0)
