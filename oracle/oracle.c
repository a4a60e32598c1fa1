/*
 * CPU oracle for the dense-contraction payloads.  TEST INFRASTRUCTURE ONLY:
 * nothing on the product path may call this file; it shares no code with the
 * CUDA library and is compiled on its own with gcc.
 *
 * What it computes is the plain definition, written out:
 *   - GEMM: the (batch-)matmul loop nest of the paper's Case Study 4 (the
 *     OpenMP tiling figure), without the batch loop and overwriting instead of
 *     accumulating (oracle_gemm), and with both (oracle_gemm_batched), with the operand transposes that the `matmul_of_transpose`
 *     pattern of Case Study 3 folds into the matmul expressed as index maps,
 *     and the negate of `negate_of_transpose` expressed as alpha = -1.
 *   - conv2d + bias + ReLU: cross-correlation over a zero-padded NHWC input
 *     (the `add_of_zero_pad` pattern of Case Study 3: padded elements are
 *     zero and contribute nothing); the paper gives no formula for it, the
 *     definition below is the standard one.
 *
 * Arithmetic: inputs are decoded from their storage type (fp32 or bf16 bit
 * patterns) exactly into double; every output element is ONE sequential fp64
 * sum in ascending reduction index; no blocking, no reassociation.  OpenMP
 * parallelism is over output rows only.
 *
 * Pins: tests/test_oracle_pins.py (hand-computed literals, closed forms,
 * exact integer cases against a library matmul, delta-filter shifts, border
 * counts, explicit-padding equivalence, brute-force output-shape enumeration).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1 };

static inline double load_elem(const void *p, int64_t idx, int dtype)
{
    if (dtype == ORACLE_F32)
        return (double)((const float *)p)[idx];
    /* bf16: the 16 stored bits are the upper half of an fp32 pattern */
    uint32_t u = ((uint32_t)((const uint16_t *)p)[idx]) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * C_ref[r, j] = alpha * sum_{k<K} Aop(i_r, k) * Bop(k, j),   j < N
 *   Aop(i,k) = transA ? A[k*M + i] : A[i*K + k]
 *   Bop(k,j) = transB ? B[j*K + k] : B[k*N + j]
 * rows == NULL: i_r = r for r < M (nrows ignored); else i_r = rows[r], r < nrows.
 * out: nrows_eff x N doubles.
 */
int oracle_gemm(int64_t M, int64_t N, int64_t K, int transA, int transB, double alpha,
                int dtype, const void *A, const void *B,
                const int64_t *rows, int64_t nrows, double *out)
{
    if (M < 0 || N < 0 || K < 0) return 1;
    int64_t nr = rows ? nrows : M;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < nr; ++r) {
        int64_t i = rows ? rows[r] : r;
        double *c = out + r * N;
        if (transB) {
            for (int64_t j = 0; j < N; ++j) {
                double acc = 0.0;
                for (int64_t k = 0; k < K; ++k) {
                    double a = load_elem(A, transA ? k * M + i : i * K + k, dtype);
                    double b = load_elem(B, j * K + k, dtype);
                    acc += a * b;
                }
                c[j] = alpha * acc;
            }
        } else {
            /* same per-element order (k ascending); row of accumulators so
             * that B is walked along its contiguous dimension */
            for (int64_t j = 0; j < N; ++j) c[j] = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                double a = load_elem(A, transA ? k * M + i : i * K + k, dtype);
                for (int64_t j = 0; j < N; ++j)
                    c[j] += a * load_elem(B, k * N + j, dtype);
            }
            for (int64_t j = 0; j < N; ++j) c[j] = alpha * c[j];
        }
    }
    return 0;
}

/*
 * The batch-matmul loop nest of the paper's Case Study 4 (the OpenMP tiling figure) as it is printed, with the
 * accumulate:  C[b,i,j] += A[b,i,k] * B[b,k,j],  generalised by two scalars and the operand transposes:
 *   C_ref[b,i,j] = beta * C_in[b,i,j] + alpha * sum_{k<K} Aop(b,i,k) * Bop(b,k,j)
 *   Aop(b,i,k) = transA ? A[b*strideA + k*M + i] : A[b*strideA + i*K + k]
 *   Bop(b,k,j) = transB ? B[b*strideB + j*K + k] : B[b*strideB + k*N + j]
 *   C_in[b,i,j] = C[b*strideC + i*N + j]   (same storage type as A and B; not read when beta == 0)
 * (alpha = beta = 1 is the paper's nest).  Strides are in elements.  out: batch x M x N doubles, dense.
 */
int oracle_gemm_batched(int64_t batch, int64_t M, int64_t N, int64_t K, int transA, int transB,
                        double alpha, double beta, int dtype,
                        const void *A, int64_t strideA, const void *B, int64_t strideB,
                        const void *C, int64_t strideC, double *out)
{
    if (batch < 0 || M < 0 || N < 0 || K < 0) return 1;
    if (beta != 0.0 && C == NULL) return 2;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int64_t b = 0; b < batch; ++b) {
        for (int64_t i = 0; i < M; ++i) {
            for (int64_t j = 0; j < N; ++j) {
                double acc = 0.0;
                for (int64_t k = 0; k < K; ++k) {
                    double a = load_elem(A, b * strideA + (transA ? k * M + i : i * K + k), dtype);
                    double bb = load_elem(B, b * strideB + (transB ? j * K + k : k * N + j), dtype);
                    acc += a * bb;
                }
                double r = alpha * acc;
                if (beta != 0.0) r += beta * load_elem(C, b * strideC + i * N + j, dtype);
                out[(b * M + i) * N + j] = r;
            }
        }
    }
    return 0;
}

/* Output extent of a strided, symmetrically zero-padded window: floor((H + 2 pad - R) / stride) + 1. */
int64_t oracle_conv_out_dim(int64_t H, int64_t R, int64_t pad, int64_t stride)
{
    int64_t span = H + 2 * pad - R;
    if (span < 0 || stride <= 0) return 0;
    return span / stride + 1;
}

/*
 * y_ref[row, k] = relu?( bias[k] + sum_{r<R} sum_{s<S} sum_{c<Cin}
 *                        X(n, p*stride + r - pad, q*stride + s - pad, c) * w[k, r, s, c] )
 *   row = (n*P + p)*Q + q;  X = 0 outside 0<=h<H, 0<=w<W;  x is NHWC, w is KRSC.
 * bias may be NULL (treated as 0).  The sum starts from 0 and the bias is
 * added last, so it is independent of the reduction.
 * rows == NULL: all N*P*Q rows; else the listed rows.  out: nrows_eff x Cout.
 */
static int conv2d_impl(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S,
                       int64_t pad, int64_t stride, int dtype, const void *x, const void *w,
                       const float *bias, const void *residual, int relu,
                       const int64_t *rows, int64_t nrows, double *out);

int oracle_conv2d(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S,
                  int64_t pad, int64_t stride, int dtype, const void *x, const void *w,
                  const float *bias, int relu,
                  const int64_t *rows, int64_t nrows, double *out)
{
    return conv2d_impl(N, H, W, Cin, Cout, R, S, pad, stride, dtype, x, w, bias, NULL, relu, rows, nrows, out);
}

/*
 * The same with a residual term (the shortcut of a ResNet block, the network the paper's workload comes from):
 *   y_ref[row, k] = relu?( conv(x, w)[row, k] + bias[k] + residual[row, k] )
 * residual is N*P*Q x Cout in the storage type of x; it joins the sum after the bias and before the ReLU.
 */
int oracle_conv2d_residual(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S,
                           int64_t pad, int64_t stride, int dtype, const void *x, const void *w,
                           const float *bias, const void *residual, int relu,
                           const int64_t *rows, int64_t nrows, double *out)
{
    return conv2d_impl(N, H, W, Cin, Cout, R, S, pad, stride, dtype, x, w, bias, residual, relu, rows, nrows, out);
}

static int conv2d_impl(int64_t N, int64_t H, int64_t W, int64_t Cin, int64_t Cout, int64_t R, int64_t S,
                       int64_t pad, int64_t stride, int dtype, const void *x, const void *w,
                       const float *bias, const void *residual, int relu,
                       const int64_t *rows, int64_t nrows, double *out)
{
    int64_t P = oracle_conv_out_dim(H, R, pad, stride);
    int64_t Q = oracle_conv_out_dim(W, S, pad, stride);
    int64_t total = N * P * Q;
    int64_t nr = rows ? nrows : total;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t rr = 0; rr < nr; ++rr) {
        int64_t row = rows ? rows[rr] : rr;
        int64_t q = row % Q, p = (row / Q) % P, n = row / (Q * P);
        for (int64_t k = 0; k < Cout; ++k) {
            double acc = 0.0;
            for (int64_t r = 0; r < R; ++r) {
                int64_t h = p * stride + r - pad;
                for (int64_t s = 0; s < S; ++s) {
                    int64_t ww = q * stride + s - pad;
                    if (h < 0 || h >= H || ww < 0 || ww >= W) continue; /* zero tap */
                    for (int64_t c = 0; c < Cin; ++c) {
                        double xv = load_elem(x, ((n * H + h) * W + ww) * Cin + c, dtype);
                        double wv = load_elem(w, ((k * R + r) * S + s) * Cin + c, dtype);
                        acc += xv * wv;
                    }
                }
            }
            if (bias) acc += (double)bias[k];
            if (residual) acc += load_elem(residual, row * Cout + k, dtype);
            if (relu && acc < 0.0) acc = 0.0;
            out[rr * Cout + k] = acc;
        }
    }
    return 0;
}

/*
 * add(zero_pad(x), y): the expression that Case Study 3's `add_of_zero_pad` pattern rewrites, computed the
 * unrewritten way -- the padded tensor is materialised (zeros outside the interior) and then added elementwise.
 *   xp[n, h, w, c] = x[n, h - top, w - left, c]  if top <= h < top + H and left <= w < left + W, else 0
 *   out[n, h, w, c] = xp[n, h, w, c] + y[n, h, w, c]      (h < H + top + bottom, w < W + left + right)
 * x is N x H x W x C, y and out are N x Hp x Wp x C (NHWC, dense).  out: doubles.
 */
int oracle_add_zero_pad(int64_t N, int64_t H, int64_t W, int64_t C, int64_t top, int64_t bottom, int64_t left,
                        int64_t right, int dtype, const void *x, const void *y, double *out)
{
    if (N < 0 || H < 0 || W < 0 || C < 0 || top < 0 || bottom < 0 || left < 0 || right < 0) return 1;
    int64_t Hp = H + top + bottom, Wp = W + left + right;
    int64_t total = N * Hp * Wp * C;
    double *xp = (double *)calloc(total > 0 ? (size_t)total : 1, sizeof(double));   /* the padded copy */
    if (!xp) return 2;
    for (int64_t n = 0; n < N; ++n)
        for (int64_t h = 0; h < H; ++h)
            for (int64_t w = 0; w < W; ++w)
                for (int64_t c = 0; c < C; ++c)
                    xp[((n * Hp + h + top) * Wp + w + left) * C + c] = load_elem(x, ((n * H + h) * W + w) * C + c, dtype);
    for (int64_t i = 0; i < total; ++i) out[i] = xp[i] + load_elem(y, i, dtype);
    free(xp);
    return 0;
}

/* double -> bf16 bit pattern, round to nearest, ties to even, in one rounding
 * (diagnostics only: distance in bf16 ulps between a result and the reference). */
void oracle_round_bf16(const double *in, int64_t n, uint16_t *out)
{
    for (int64_t i = 0; i < n; ++i) {
        double v = in[i];
        if (v == 0.0 || isnan(v) || isinf(v)) {
            float f = (float)v; uint32_t u; memcpy(&u, &f, 4);
            out[i] = (uint16_t)(u >> 16);
            continue;
        }
        int e;
        double m = frexp(fabs(v), &e);          /* |v| = m * 2^e, m in [0.5, 1) */
        /* bf16 has 8 significant bits: scale so that the integer part has 8 bits */
        int ee = e - 8;
        if (e - 1 < -126) ee = -126 - 7;        /* subnormal range of the format */
        double scaled = ldexp(fabs(v), -ee);
        double fl = floor(scaled);
        double frac = scaled - fl;
        if (frac > 0.5 || (frac == 0.5 && fmod(fl, 2.0) == 1.0)) fl += 1.0;
        float f = (float)ldexp(fl, ee);         /* exact: <= 9 significant bits */
        if (v < 0) f = -f;
        uint32_t u; memcpy(&u, &f, 4);
        out[i] = (uint16_t)(u >> 16);
        (void)m;
    }
}
