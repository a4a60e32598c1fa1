"""Pins of the CPU oracle against things other than itself (CPU only).

Each test fixes one thing a plausible mistake would break: an index map, a
transposed operand, a dropped term, a sign, a flipped filter, the padding
offset, the stride, the bias/ReLU order.
"""
import math

import numpy as np
import pytest
from scipy.signal import correlate2d

import oracle
import seeded_inputs as si
from conftest import read_golden


def f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def bf(a):
    return si.f32_to_bf16_bits(f32(a))


# --------------------------------------------------------------------- GEMM

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("transA,transB", [(0, 0), (0, 1), (1, 0), (1, 1)])
def test_gemm_hand_computed_literals(dtype, transA, transB):
    g = read_golden("gemm_2x3x2.txt")
    A = np.array(g["A"]).reshape(2, 3)
    B = np.array(g["B"]).reshape(3, 2)
    C = np.array(g["C"]).reshape(2, 2)
    enc = f32 if dtype == "f32" else bf
    As = enc(A.T if transA else A)          # stored K x M when transA
    Bs = enc(B.T if transB else B)          # stored N x K when transB
    out = oracle.gemm(2, 2, 3, transA, transB, 1.0, dtype, As, Bs)
    assert np.array_equal(out, C)


def test_gemm_identity_and_closed_forms():
    M, K = 7, 5
    A = si.uniform(11, 0, (M, K), "f32")
    assert np.array_equal(oracle.gemm(M, K, K, 0, 0, 1.0, "f32", A, f32(np.eye(K))), A.astype(np.float64))
    assert np.array_equal(oracle.gemm(M, K, M, 0, 0, 1.0, "f32", f32(np.eye(M)), A), A.astype(np.float64))
    # all-ones operands: every entry equals K
    out = oracle.gemm(4, 6, 37, 0, 0, 1.0, "f32", f32(np.ones((4, 37))), f32(np.ones((37, 6))))
    assert np.array_equal(out, np.full((4, 6), 37.0))
    # A[i,k] = i, B[k,j] = j  =>  C[i,j] = K i j
    M, N, K = 5, 6, 9
    A = f32(np.repeat(np.arange(M)[:, None], K, axis=1))
    B = f32(np.repeat(np.arange(N)[None, :], K, axis=0))
    assert np.array_equal(oracle.gemm(M, N, K, 0, 0, 1.0, "f32", A, B), K * np.outer(np.arange(M), np.arange(N)))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("transA,transB", [(0, 0), (0, 1), (1, 0), (1, 1)])
def test_gemm_exact_integers_vs_library_matmul(dtype, transA, transB):
    # Small integers: all products and partial sums are exact in fp64, so the
    # oracle must agree with numpy's fp64 matmul bit for bit.
    M, N, K = 13, 9, 31
    A = si.bf16_bits_to_f32(si.small_integers(21, 0, (M, K), "bf16")).astype(np.float64)
    B = si.bf16_bits_to_f32(si.small_integers(21, 1, (K, N), "bf16")).astype(np.float64)
    enc = f32 if dtype == "f32" else bf
    out = oracle.gemm(M, N, K, transA, transB, -3.0, dtype,
                      enc(A.T if transA else A), enc(B.T if transB else B))
    assert np.array_equal(out, -3.0 * (A @ B))


def test_gemm_transpose_of_product():
    # (A.B)^T = B^T.A^T, exactly on integers: feed B as a transposed-left and
    # A as a transposed-right operand.
    M, N, K = 6, 10, 17
    A = si.small_integers(22, 0, (M, K), "f32")
    B = si.small_integers(22, 1, (K, N), "f32")
    AB = oracle.gemm(M, N, K, 0, 0, 1.0, "f32", A, B)
    BtAt = oracle.gemm(N, M, K, 1, 1, 1.0, "f32", B, A)     # op(A')=B^T (B stored K x N), op(B')=A^T (A stored M x K)
    assert np.array_equal(AB.T, BtAt)


def test_gemm_negate_is_exact_sign_flip_and_alpha_linear():
    M, N, K = 9, 8, 64
    A, B = si.gemm_bf16_normal(M, N, K, seed=3, transB=1)
    pos = oracle.gemm(M, N, K, 0, 1, 1.0, "bf16", A, B)
    neg = oracle.gemm(M, N, K, 0, 1, -1.0, "bf16", A, B)
    assert np.array_equal(neg, -pos)
    assert np.array_equal(oracle.gemm(M, N, K, 0, 1, 0.5, "bf16", A, B), 0.5 * pos)


def test_gemm_fp64_sum_within_error_bound_of_exact_sum():
    # Products of bf16 values are exact in fp64; math.fsum returns the
    # correctly rounded exact sum.  A sequential fp64 sum differs from it by at
    # most (K-1) * 2^-53 * sum|a b|.
    M, N, K = 3, 4, 4096
    A, B = si.gemm_bf16_normal(M, N, K, seed=4, transB=1)
    out = oracle.gemm(M, N, K, 0, 1, 1.0, "bf16", A, B)
    a = oracle.decode(A, "bf16").reshape(M, K)
    b = oracle.decode(B, "bf16").reshape(N, K)
    for i in range(M):
        for j in range(N):
            terms = [float(a[i, k]) * float(b[j, k]) for k in range(K)]
            exact = math.fsum(terms)
            bound = (K - 1) * 2.0 ** -53 * math.fsum(abs(t) for t in terms)
            assert abs(out[i, j] - exact) <= bound


def test_gemm_row_subset_matches_full():
    M, N, K = 40, 12, 33
    A, B = si.gemm_f32_uniform(M, N, K, seed=5)
    full = oracle.gemm(M, N, K, 0, 0, 1.0, "f32", A, B)
    rows = [0, 39, 7, 7, 21]
    assert np.array_equal(oracle.gemm(M, N, K, 0, 0, 1.0, "f32", A, B, rows=rows), full[rows])


def test_gemm_empty_reduction_gives_zero():
    out = oracle.gemm(3, 2, 0, 0, 0, 1.0, "f32", f32(np.zeros((3, 0))), f32(np.zeros((0, 2))))
    assert np.array_equal(out, np.zeros((3, 2)))


# --------------------------------------------------------------------- batch-matmul with accumulate

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_gemm_batched_hand_computed_literals(dtype):
    g = read_golden("gemm_batched_2x2x2x2.txt")
    enc = f32 if dtype == "f32" else bf
    A, B, Cin = enc(g["A"]), enc(g["B"]), enc(g["Cin"])
    out = oracle.gemm_batched(2, 2, 2, 2, 0, 0, 1.0, 1.0, dtype, A, B, Cin)       # the paper's nest: C += A . B
    assert np.array_equal(out.ravel(), np.array(g["C11"]))
    out = oracle.gemm_batched(2, 2, 2, 2, 0, 0, 2.0, -1.0, dtype, A, B, Cin)
    assert np.array_equal(out.ravel(), np.array(g["C2m1"]))


@pytest.mark.parametrize("transA,transB", [(0, 0), (0, 1), (1, 0), (1, 1)])
def test_gemm_batched_exact_integers_vs_library_einsum_with_gapped_strides(transA, transB):
    # small integers: exact in fp64, so the oracle must equal numpy's batched product bit for bit; the batches are
    # laid out with gaps (stride > dense size) filled with NaN, which a wrong stride or index map would pull in
    rng = np.random.default_rng(5)
    batch, M, N, K = 3, 5, 4, 7
    A = rng.integers(-4, 5, (batch, M, K)).astype(np.float64)
    B = rng.integers(-4, 5, (batch, K, N)).astype(np.float64)
    C = rng.integers(-9, 10, (batch, M, N)).astype(np.float64)
    sa, sb, sc = M * K + 3, K * N + 5, M * N + 2

    def lay(x, stride, transposed):
        buf = np.full(batch * stride, np.nan, dtype=np.float32)
        for b in range(batch):
            v = (x[b].T if transposed else x[b]).ravel()
            buf[b * stride: b * stride + v.size] = v
        return buf

    out = oracle.gemm_batched(batch, M, N, K, transA, transB, 3.0, -2.0, "f32", lay(A, sa, transA), lay(B, sb, transB),
                              lay(C, sc, False), strideA=sa, strideB=sb, strideC=sc)
    assert np.array_equal(out, 3.0 * np.einsum("bik,bkj->bij", A, B) - 2.0 * C)


def test_gemm_batched_closed_forms_and_special_cases():
    batch, M, N, K = 4, 3, 5, 11
    ones = lambda *sh: f32(np.ones(sh))                                    # noqa: E731
    # all-ones operands and C: every entry = alpha K + beta
    out = oracle.gemm_batched(batch, M, N, K, 0, 0, 0.5, 3.0, "f32", ones(batch, M, K), ones(batch, K, N), ones(batch, M, N))
    assert np.array_equal(out, np.full((batch, M, N), 0.5 * K + 3.0))
    # zero A: the result is beta C;  beta = 0: C is not read (NaNs in it do not matter, and it may be absent)
    Cin = si.uniform(12, 2, (batch, M, N), "f32")
    out = oracle.gemm_batched(batch, M, N, K, 0, 0, 1.0, -1.5, "f32", f32(np.zeros((batch, M, K))), ones(batch, K, N), Cin)
    assert np.array_equal(out, -1.5 * Cin.astype(np.float64))
    A, B = si.uniform(12, 0, (batch, M, K), "f32"), si.uniform(12, 1, (batch, K, N), "f32")
    nan_c = f32(np.full((batch, M, N), np.nan))
    out0 = oracle.gemm_batched(batch, M, N, K, 0, 0, 1.0, 0.0, "f32", A, B, nan_c)
    assert np.array_equal(out0, oracle.gemm_batched(batch, M, N, K, 0, 0, 1.0, 0.0, "f32", A, B))
    # each batch of the batched call is the single-matrix definition (pinned above) on that batch's operands
    for b in range(batch):
        assert np.array_equal(out0[b], oracle.gemm(M, N, K, 0, 0, 1.0, "f32", A[b], B[b]))
    # accumulating twice from zero doubles the product (integers: exact)
    Ai = f32(np.random.default_rng(6).integers(-3, 4, (batch, M, K)))
    Bi = f32(np.random.default_rng(7).integers(-3, 4, (batch, K, N)))
    once = oracle.gemm_batched(batch, M, N, K, 0, 0, 1.0, 1.0, "f32", Ai, Bi, f32(np.zeros((batch, M, N))))
    twice = oracle.gemm_batched(batch, M, N, K, 0, 0, 1.0, 1.0, "f32", Ai, Bi, f32(once))
    assert np.array_equal(twice, 2.0 * once)


# --------------------------------------------------------------------- add of zero pad

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_add_zero_pad_hand_computed_literals(dtype):
    g = read_golden("add_zero_pad_2x2_into_4x3.txt")
    enc = f32 if dtype == "f32" else bf
    out = oracle.add_zero_pad(1, 2, 2, 1, 1, 1, 0, 1, dtype, enc(g["x"]), enc(g["y"]))
    assert np.array_equal(out.ravel(), np.array(g["out"]))


@pytest.mark.parametrize("pads", [(0, 0, 0, 0), (1, 1, 1, 1), (2, 0, 1, 3), (0, 3, 0, 0)])
def test_add_zero_pad_vs_library_pad_and_closed_forms(pads):
    top, bottom, left, right = pads
    N, H, W, C = 2, 5, 4, 3
    x = si.uniform(21, 0, (N, H, W, C), "f32")
    y = si.uniform(21, 1, (N, H + top + bottom, W + left + right, C), "f32")
    ref = np.pad(x.astype(np.float64), ((0, 0), (top, bottom), (left, right), (0, 0))) + y.astype(np.float64)
    assert np.array_equal(oracle.add_zero_pad(N, H, W, C, top, bottom, left, right, "f32", x, y), ref)
    # all ones: 2 in the interior, 1 on the padding ring; the ring of the result is y's ring untouched
    one_x, one_y = f32(np.ones((N, H, W, C))), f32(np.ones(y.shape))
    out = oracle.add_zero_pad(N, H, W, C, top, bottom, left, right, "f32", one_x, one_y)
    interior = np.zeros(y.shape, dtype=bool)
    interior[:, top:top + H, left:left + W, :] = True
    assert np.array_equal(out, np.where(interior, 2.0, 1.0))
    assert np.array_equal(oracle.add_zero_pad(N, H, W, C, top, bottom, left, right, "f32", x, y)[~interior],
                          y.astype(np.float64)[~interior])


# --------------------------------------------------------------------- conv

def test_conv_hand_computed_literals():
    g = read_golden("conv_3x3_pad1.txt")
    x = f32(np.array(g["x"]).reshape(1, 3, 3, 1))
    w = f32(np.array(g["w"]).reshape(1, 3, 3, 1))
    out = oracle.conv2d(1, 3, 3, 1, 1, 3, 3, 1, 1, "f32", x, w, None, 0)
    assert np.array_equal(out.reshape(-1), np.array(g["y"]))


@pytest.mark.parametrize("R,S,pad", [(3, 3, 1), (5, 3, 0), (1, 1, 0), (3, 5, 2)])
def test_conv_vs_library_cross_correlation(R, S, pad):
    # Integer inputs, so everything is exact.  y[.,k] = sum_c correlate2d(x[.,c], w[k,.,.,c]).
    N, H, W, Cin, Cout = 2, 7, 9, 3, 4
    x = si.small_integers(31, 0, (N, H, W, Cin), "f32", -4, 4)
    w = si.small_integers(31, 1, (Cout, R, S, Cin), "f32", -4, 4)
    out = oracle.conv2d(N, H, W, Cin, Cout, R, S, pad, 1, "f32", x, w, None, 0)
    P, Q = H + 2 * pad - R + 1, W + 2 * pad - S + 1
    out = out.reshape(N, P, Q, Cout)
    xp = np.zeros((N, H + 2 * pad, W + 2 * pad, Cin))
    xp[:, pad:pad + H, pad:pad + W, :] = x
    for n in range(N):
        for k in range(Cout):
            ref = sum(correlate2d(xp[n, :, :, c], w[k, :, :, c].astype(np.float64), mode="valid")
                      for c in range(Cin))
            assert np.array_equal(out[n, :, :, k], ref)


def test_conv_1x1_reduces_to_gemm():
    N, H, W, Cin, Cout = 2, 4, 5, 16, 8
    x, w, _ = si.conv_bf16(N, H, W, Cin, Cout, 1, 1, seed=32)
    y = oracle.conv2d(N, H, W, Cin, Cout, 1, 1, 0, 1, "bf16", x, w, None, 0)
    g = oracle.gemm(N * H * W, Cout, Cin, 0, 1, 1.0, "bf16", x.reshape(-1, Cin), w.reshape(Cout, Cin))
    assert np.array_equal(y, g)


@pytest.mark.parametrize("r0,s0", [(0, 0), (0, 2), (1, 1), (2, 0), (2, 1)])
def test_conv_delta_filter_is_shifted_copy(r0, s0):
    # w[k, r0, s0, c] = delta(c, k): y[n,p,q,k] = X(n, p + r0 - pad, q + s0 - pad, k), zero outside.
    N, H, W, C, pad = 1, 5, 6, 3, 1
    x = si.uniform(33, 0, (N, H, W, C), "f32")
    w = np.zeros((C, 3, 3, C), dtype=np.float32)
    for k in range(C):
        w[k, r0, s0, k] = 1.0
    y = oracle.conv2d(N, H, W, C, C, 3, 3, pad, 1, "f32", x, w, None, 0).reshape(N, H, W, C)
    exp = np.zeros((N, H, W, C))
    for p in range(H):
        for q in range(W):
            h, ww = p + r0 - pad, q + s0 - pad
            if 0 <= h < H and 0 <= ww < W:
                exp[0, p, q] = x[0, h, ww]
    assert np.array_equal(y, exp)


def test_conv_zero_pad_border_counts():
    # all-ones image and 3x3 all-ones filter: interior 9, edges 6, corners 4
    H = W = 5
    y = oracle.conv2d(1, H, W, 1, 1, 3, 3, 1, 1, "f32", f32(np.ones((1, H, W, 1))), f32(np.ones((1, 3, 3, 1))),
                      None, 0).reshape(H, W)
    exp = np.full((H, W), 9.0)
    exp[0, :] = exp[-1, :] = exp[:, 0] = exp[:, -1] = 6.0
    exp[0, 0] = exp[0, -1] = exp[-1, 0] = exp[-1, -1] = 4.0
    assert np.array_equal(y, exp)


@pytest.mark.parametrize("stride", [1, 2])
def test_conv_padding_equals_explicit_zero_padded_copy(stride):
    N, H, W, Cin, Cout, pad = 2, 6, 7, 4, 3, 2
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, 3, 3, seed=34)
    y = oracle.conv2d(N, H, W, Cin, Cout, 3, 3, pad, stride, "bf16", x, w, b, 1)
    xp = np.zeros((N, H + 2 * pad, W + 2 * pad, Cin), dtype=np.uint16)
    xp[:, pad:pad + H, pad:pad + W, :] = x
    y2 = oracle.conv2d(N, H + 2 * pad, W + 2 * pad, Cin, Cout, 3, 3, 0, stride, "bf16", xp, w, b, 1)
    assert np.array_equal(y, y2)


def test_conv_stride_subsamples_stride1():
    N, H, W, Cin, Cout = 1, 9, 8, 2, 3
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, 3, 3, seed=35)
    y1 = oracle.conv2d(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 0).reshape(N, H, W, Cout)
    P2, Q2 = oracle.conv_out_dim(H, 3, 1, 2), oracle.conv_out_dim(W, 3, 1, 2)
    y2 = oracle.conv2d(N, H, W, Cin, Cout, 3, 3, 1, 2, "bf16", x, w, b, 0).reshape(N, P2, Q2, Cout)
    assert np.array_equal(y2, y1[:, ::2, ::2, :][:, :P2, :Q2, :])


def test_conv_bias_relu():
    N, H, W, Cin, Cout = 1, 4, 4, 3, 5
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, 3, 3, seed=36)
    zero_w = np.zeros_like(w)
    y = oracle.conv2d(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, zero_w, b, 1)
    assert np.array_equal(y, np.broadcast_to(np.maximum(b.astype(np.float64), 0.0), y.shape))
    lin = oracle.conv2d(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 0)
    act = oracle.conv2d(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1)
    assert (act >= 0).all() and np.array_equal(act, np.maximum(lin, 0.0))
    assert (lin < 0).any()                                   # the ReLU had something to clip
    nob = oracle.conv2d(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, None, 0)
    assert np.allclose(lin - nob, b.astype(np.float64)[None, :], rtol=0, atol=1e-12)


def test_conv_residual_joins_before_the_relu():
    N, H, W, Cin, Cout = 2, 5, 6, 3, 4
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, 3, 3, seed=19)
    xf, wf = si.bf16_bits_to_f32(x), si.bf16_bits_to_f32(w)
    res = si.uniform(19, 3, (N * H * W, Cout), "f32", scale=2.0)
    pre = oracle.conv2d(N, H, W, Cin, Cout, 3, 3, 1, 1, "f32", xf, wf, b, 0)
    # without ReLU the residual is a plain elementwise addend; with it, the ReLU sees the sum (not relu(conv) + residual)
    assert np.array_equal(oracle.conv2d(N, H, W, Cin, Cout, 3, 3, 1, 1, "f32", xf, wf, b, 0, residual=res),
                          pre + res.astype(np.float64))
    out = oracle.conv2d(N, H, W, Cin, Cout, 3, 3, 1, 1, "f32", xf, wf, b, 1, residual=res)
    assert np.array_equal(out, np.maximum(pre + res.astype(np.float64), 0.0)) and (out >= 0).all()
    assert not np.array_equal(out, np.maximum(pre, 0.0) + res.astype(np.float64))
    # zero weights and bias: y = relu(residual); a zero residual changes nothing
    z = np.zeros_like(wf)
    assert np.array_equal(oracle.conv2d(N, H, W, Cin, Cout, 3, 3, 1, 1, "f32", xf, z, None, 1, residual=res),
                          np.maximum(res.astype(np.float64), 0.0))
    assert np.array_equal(oracle.conv2d(N, H, W, Cin, Cout, 3, 3, 1, 1, "f32", xf, wf, b, 1, residual=np.zeros_like(res)),
                          oracle.conv2d(N, H, W, Cin, Cout, 3, 3, 1, 1, "f32", xf, wf, b, 1))
    # row subsets index the residual by output row
    rows = np.array([0, 7, 31, N * H * W - 1])
    assert np.array_equal(oracle.conv2d(N, H, W, Cin, Cout, 3, 3, 1, 1, "f32", xf, wf, b, 1, rows=rows, residual=res), out[rows])


def test_conv_linear_in_input_without_bias_and_relu():
    N, H, W, Cin, Cout = 1, 5, 5, 2, 2
    x1 = si.small_integers(37, 0, (N, H, W, Cin), "f32")
    x2 = si.small_integers(37, 3, (N, H, W, Cin), "f32")
    w = si.small_integers(37, 1, (Cout, 3, 3, Cin), "f32")
    f = lambda x: oracle.conv2d(N, H, W, Cin, Cout, 3, 3, 1, 1, "f32", x, w, None, 0)
    assert np.array_equal(f(f32(x1 + 2 * x2)), f(x1) + 2 * f(x2))


def test_conv_out_dim_brute_force():
    for H in range(1, 9):
        for R in range(1, 4):
            for pad in range(0, 3):
                for stride in (1, 2):
                    # valid p: window [p*stride - pad, p*stride - pad + R) inside the padded image
                    n = sum(1 for p in range(0, 64) if p * stride + R <= H + 2 * pad)
                    assert oracle.conv_out_dim(H, R, pad, stride) == n


def test_conv_row_subset_matches_full():
    N, H, W, Cin, Cout = 2, 5, 6, 4, 3
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, 3, 3, seed=38)
    full = oracle.conv2d(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1)
    rows = [0, 59, 30, 31, 5]
    assert np.array_equal(oracle.conv2d(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1, rows=rows), full[rows])


# --------------------------------------------------------- rounding, metric

def test_round_bf16_literals_and_independent_rounder():
    v = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -40, -2.5, 0.0, 3.0e-39])
    bits = oracle.round_bf16(v)
    assert [int(b) for b in bits[:6]] == [0x3F80, 0x3F80, 0x3F82, 0x3F81, 0xC020, 0x0000]
    # values that are exactly fp32: the generator module's integer-add rounder is an independent route
    x = si.normal(41, 0, (4096,), "f32")
    assert np.array_equal(oracle.round_bf16(x.astype(np.float64)), si.f32_to_bf16_bits(x))


def test_metric_returns_injected_perturbation():
    M, N, K = 6, 5, 32
    A, B = si.gemm_bf16_normal(M, N, K, seed=42, transB=1)
    ref = oracle.gemm(M, N, K, 0, 1, -1.0, "bf16", A, B)
    sc = oracle.gemm_row_scales(M, N, K, 0, 1, -1.0, "bf16", A, B)
    # scale is an upper bound on |C[i,j]| (Cauchy-Schwarz)
    assert (np.abs(ref) <= sc[:, None] * (1 + 1e-12)).all()
    a = oracle.decode(A, "bf16").reshape(M, K)
    b = oracle.decode(B, "bf16").reshape(N, K)
    exp_sc = np.array([np.linalg.norm(a[i]) for i in range(M)]) * max(np.linalg.norm(b[j]) for j in range(N))
    assert np.allclose(sc, exp_sc, rtol=1e-12)
    bad = ref.copy()
    bad[3, 2] += 1e-3 * sc[3]
    assert abs(oracle.max_normalised_error(bad, ref, sc) - 1e-3) < 1e-9
    assert oracle.max_normalised_error(ref, ref, sc) == 0.0


def test_conv_metric_scale_is_patch_norm():
    N, H, W, Cin, Cout, pad = 1, 4, 5, 3, 2, 1
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, 3, 3, seed=43)
    sc = oracle.conv_row_scales(N, H, W, Cin, Cout, 3, 3, pad, 1, "bf16", x, w, b).reshape(H, W)
    xd = oracle.decode(x, "bf16").reshape(H, W, Cin)
    wd = oracle.decode(w, "bf16").reshape(Cout, -1)
    wmax = max(np.linalg.norm(wd[k]) for k in range(Cout))
    for p in range(H):
        for q in range(W):
            e = 0.0
            for r in range(3):
                for s in range(3):
                    h, ww = p + r - pad, q + s - pad
                    if 0 <= h < H and 0 <= ww < W:
                        e += float((xd[h, ww] ** 2).sum())
            assert abs(sc[p, q] - (math.sqrt(e) * wmax + float(np.abs(b).max()))) < 1e-9
    # zero-scale rows must match exactly
    assert oracle.max_normalised_error(np.array([[1.0]]), np.array([[0.0]]), np.array([0.0])) == float("inf")
    assert oracle.max_normalised_error(np.array([[0.0]]), np.array([[0.0]]), np.array([0.0])) == 0.0


def test_statistical_sanity_of_normal_gemm():
    # entries of A.B^T with N(0,1) operands have variance K
    M, N, K = 64, 64, 1024
    A, B = si.gemm_bf16_normal(M, N, K, seed=1, transB=1)
    c = oracle.gemm(M, N, K, 0, 1, 1.0, "bf16", A, B)
    assert abs(c.std() / math.sqrt(K) - 1.0) < 0.05
