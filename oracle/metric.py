"""Error metric of the parity tests (test infrastructure, CPU only, numpy fp64).

A result C^ is compared with the fp64 reference C per output row i:

    err = max_i max_j |C^[i,j] - C[i,j]| / scale_i

GEMM:  scale_i = |alpha| * ||Aop(i,:)||_2 * max_j ||Bop(:,j)||_2
batched GEMM with accumulate: scale_(b,i) = the GEMM scale of batch b + |beta| * max_j |C_in[b,i,j]|
conv:  scale_i = ||patch_i||_2 * max_k ||w_k||_2 + max_k |bias_k|
       (patch_i = the R*S*Cin input window of output pixel i, zero taps included;
        ReLU is 1-Lipschitz so the same bound carries through it)

By Cauchy-Schwarz |C[i,j]| <= scale_i, so err is a relative error against the
largest value the row could hold.  A row whose scale is 0 must match exactly.
"""
from __future__ import annotations

import numpy as np


def decode(arr: np.ndarray, dtype) -> np.ndarray:
    """Storage (fp32 array, or uint16 bf16 bit patterns) -> exact float64 values."""
    if dtype in ("f32", 0):
        return np.asarray(arr, dtype=np.float32).astype(np.float64)
    u = np.asarray(arr, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def gemm_row_scales(M, N, K, transA, transB, alpha, dtype, A, B, rows=None) -> np.ndarray:
    a = decode(A, dtype).reshape((K, M) if transA else (M, K))
    b = decode(B, dtype).reshape((N, K) if transB else (K, N))
    a_norm = np.sqrt((a * a).sum(axis=0 if transA else 1))          # per row i of op(A)
    b_norm = np.sqrt((b * b).sum(axis=1 if transB else 0))          # per column j of op(B)
    bmax = b_norm.max() if b_norm.size else 0.0
    s = abs(float(alpha)) * a_norm * bmax
    return s if rows is None else s[np.asarray(rows, dtype=np.int64)]


def gemm_batched_row_scales(batch, M, N, K, transA, transB, alpha, beta, dtype, A, B, C=None) -> np.ndarray:
    """Scales of the batch * M output rows of a dense batched GEMM (row b*M + i), accumulate term included."""
    a = decode(A, dtype).reshape((batch, K, M) if transA else (batch, M, K))
    b = decode(B, dtype).reshape((batch, N, K) if transB else (batch, K, N))
    a_norm = np.sqrt((a * a).sum(axis=1 if transA else 2))          # batch x M
    b_norm = np.sqrt((b * b).sum(axis=2 if transB else 1))          # batch x N
    bmax = b_norm.max(axis=1, keepdims=True) if N else np.zeros((batch, 1))
    s = abs(float(alpha)) * a_norm * bmax
    if beta != 0.0 and C is not None:
        s = s + abs(float(beta)) * np.abs(decode(C, dtype).reshape(batch, M, N)).max(axis=2)
    return s.reshape(-1)


def conv_row_scales(N, H, W, Cin, Cout, R, S, pad, stride, dtype, x, w, bias, rows=None, residual=None) -> np.ndarray:
    xe = decode(x, dtype).reshape(N, H, W, Cin)
    energy = (xe * xe).sum(axis=3)                                   # per input pixel
    ep = np.zeros((N, H + 2 * pad, W + 2 * pad))
    ep[:, pad:pad + H, pad:pad + W] = energy
    P = (H + 2 * pad - R) // stride + 1
    Q = (W + 2 * pad - S) // stride + 1
    acc = np.zeros((N, P, Q))
    for r in range(R):
        for s in range(S):
            acc += ep[:, r:r + (P - 1) * stride + 1:stride, s:s + (Q - 1) * stride + 1:stride]
    wd = decode(w, dtype).reshape(Cout, -1)
    wmax = np.sqrt((wd * wd).sum(axis=1)).max()
    bmax = 0.0 if bias is None else float(np.abs(np.asarray(bias, dtype=np.float64)).max())
    sc = (np.sqrt(acc) * wmax + bmax).reshape(-1)
    if residual is not None:                                          # + max_k |residual[row, k]|
        sc = sc + np.abs(decode(residual, dtype).reshape(-1, Cout)).max(axis=1)
    return sc if rows is None else sc[np.asarray(rows, dtype=np.int64)]


def max_normalised_error(result: np.ndarray, ref: np.ndarray, scales: np.ndarray) -> float:
    """max over rows of max_j |result - ref| / scale_row (inf if a zero-scale row differs)."""
    result = np.asarray(result, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    if result.shape != ref.shape:
        raise ValueError(f"shape mismatch {result.shape} vs {ref.shape}")
    if result.size == 0:
        return 0.0
    if not np.isfinite(result).all():
        return float("inf")
    d = np.abs(result - ref).max(axis=1)
    scales = np.asarray(scales, dtype=np.float64)
    zero = scales == 0.0
    if (d[zero] != 0.0).any():
        return float("inf")
    safe = np.where(zero, 1.0, scales)
    return float((d / safe).max())
