"""CPU oracle (test infrastructure, NOT a product path).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It wraps `oracle.c` (plain fp64 loops, compiled here with gcc)
and adds the error metric used to compare a result with the reference.

The oracle never imports the CUDA package and the CUDA package never imports
the oracle.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "oracle.c"
_LIB = _HERE / "liboracle.so"

F32 = 0
BF16 = 1
_DT = {"f32": F32, "bf16": BF16, F32: F32, BF16: BF16}

_lib = None


def build(force: bool = False) -> Path:
    """Compile oracle.c into liboracle.so (gcc -O2 -fopenmp, no fast-math)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        cmd = ["gcc", "-O2", "-fopenmp", "-fno-fast-math", "-ffp-contract=off", "-shared", "-fPIC",
               "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_LIB))
        i64, p = ctypes.c_int64, ctypes.c_void_p
        lib.oracle_gemm.argtypes = [i64, i64, i64, ctypes.c_int, ctypes.c_int, ctypes.c_double,
                                    ctypes.c_int, p, p, p, i64, p]
        lib.oracle_gemm.restype = ctypes.c_int
        lib.oracle_gemm_batched.argtypes = [i64, i64, i64, i64, ctypes.c_int, ctypes.c_int, ctypes.c_double,
                                            ctypes.c_double, ctypes.c_int, p, i64, p, i64, p, i64, p]
        lib.oracle_gemm_batched.restype = ctypes.c_int
        lib.oracle_add_zero_pad.argtypes = [i64] * 8 + [ctypes.c_int, p, p, p]
        lib.oracle_add_zero_pad.restype = ctypes.c_int
        lib.oracle_conv2d.argtypes = [i64] * 9 + [ctypes.c_int, p, p, p, ctypes.c_int, p, i64, p]
        lib.oracle_conv2d.restype = ctypes.c_int
        lib.oracle_conv2d_residual.argtypes = [i64] * 9 + [ctypes.c_int, p, p, p, p, ctypes.c_int, p, i64, p]
        lib.oracle_conv2d_residual.restype = ctypes.c_int
        lib.oracle_conv_out_dim.argtypes = [i64] * 4
        lib.oracle_conv_out_dim.restype = i64
        lib.oracle_round_bf16.argtypes = [p, i64, p]
        lib.oracle_round_bf16.restype = None
        lib.oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _check(arr: np.ndarray, dtype: int, n: int, name: str) -> np.ndarray:
    want = np.float32 if dtype == F32 else np.uint16
    a = np.ascontiguousarray(arr)
    if a.dtype != want:
        raise TypeError(f"{name}: expected {want.__name__} storage, got {a.dtype}")
    if a.size != n:
        raise ValueError(f"{name}: expected {n} elements, got {a.size}")
    return a


def gemm(M, N, K, transA, transB, alpha, dtype, A, B, rows=None) -> np.ndarray:
    """fp64 reference of C = alpha * op(A) . op(B); returns (len(rows) or M) x N doubles.

    A is stored K x M when transA else M x K; B is stored N x K when transB else
    K x N (all row-major).  bf16 tensors are uint16 bit patterns.
    """
    lib, dt = _load(), _DT[dtype]
    A = _check(A, dt, M * K, "A")
    B = _check(B, dt, K * N, "B")
    if rows is None:
        nr, rp, rows_arr = M, None, None
    else:
        rows_arr = np.ascontiguousarray(rows, dtype=np.int64)
        if rows_arr.size and (rows_arr.min() < 0 or rows_arr.max() >= M):
            raise ValueError("row index out of range")
        nr, rp = rows_arr.size, rows_arr.ctypes.data
    out = np.empty((nr, N), dtype=np.float64)
    rc = lib.oracle_gemm(M, N, K, int(transA), int(transB), float(alpha), dt,
                         A.ctypes.data, B.ctypes.data, rp, nr, out.ctypes.data)
    if rc:
        raise RuntimeError(f"oracle_gemm failed ({rc})")
    return out


def gemm_batched(batch, M, N, K, transA, transB, alpha, beta, dtype, A, B, C=None, strideA=None, strideB=None,
                 strideC=None) -> np.ndarray:
    """fp64 reference of C[b] = beta * C[b] + alpha * op(A[b]) . op(B[b]); returns batch x M x N doubles.

    Strides are in elements and default to the dense ones (M*K, K*N, M*N); C is only read when beta != 0.
    """
    lib, dt = _load(), _DT[dtype]
    sa = M * K if strideA is None else strideA
    sb = K * N if strideB is None else strideB
    sc = M * N if strideC is None else strideC
    need = lambda stride, dense: (batch - 1) * stride + dense if batch > 0 else 0   # noqa: E731
    want = np.float32 if dt == F32 else np.uint16
    A = np.ascontiguousarray(A)
    B = np.ascontiguousarray(B)
    if A.dtype != want or B.dtype != want:
        raise TypeError(f"expected {want.__name__} storage")
    if A.size < need(sa, M * K) or B.size < need(sb, K * N):
        raise ValueError("operand smaller than its strides imply")
    cp = None
    if beta != 0.0:
        if C is None:
            raise ValueError("beta != 0 needs C")
        C = np.ascontiguousarray(C)
        if C.dtype != want or C.size < need(sc, M * N):
            raise ValueError("bad C")
        cp = C.ctypes.data
    out = np.empty((batch, M, N), dtype=np.float64)
    rc = lib.oracle_gemm_batched(batch, M, N, K, int(transA), int(transB), float(alpha), float(beta), dt,
                                 A.ctypes.data, sa, B.ctypes.data, sb, cp, sc, out.ctypes.data)
    if rc:
        raise RuntimeError(f"oracle_gemm_batched failed ({rc})")
    return out


def add_zero_pad(N, H, W, C, top, bottom, left, right, dtype, x, y) -> np.ndarray:
    """fp64 reference of zero_pad(x) + y; x is N x H x W x C, y is N x (H+top+bottom) x (W+left+right) x C."""
    lib, dt = _load(), _DT[dtype]
    Hp, Wp = H + top + bottom, W + left + right
    x = _check(x, dt, N * H * W * C, "x")
    y = _check(y, dt, N * Hp * Wp * C, "y")
    out = np.empty((N, Hp, Wp, C), dtype=np.float64)
    rc = lib.oracle_add_zero_pad(N, H, W, C, top, bottom, left, right, dt, x.ctypes.data, y.ctypes.data, out.ctypes.data)
    if rc:
        raise RuntimeError(f"oracle_add_zero_pad failed ({rc})")
    return out


def conv_out_dim(H, R, pad, stride) -> int:
    return int(_load().oracle_conv_out_dim(H, R, pad, stride))


def conv2d(N, H, W, Cin, Cout, R, S, pad, stride, dtype, x, w, bias, relu, rows=None, residual=None) -> np.ndarray:
    """fp64 reference of y = relu?(conv(x, w) + bias [+ residual]); returns (rows or N*P*Q) x Cout.
    residual, if given, is N*P*Q x Cout in the storage type of x."""
    lib, dt = _load(), _DT[dtype]
    x = _check(x, dt, N * H * W * Cin, "x")
    w = _check(w, dt, Cout * R * S * Cin, "w")
    bp = None
    if bias is not None:
        bias = _check(bias, F32, Cout, "bias")
        bp = bias.ctypes.data
    P, Q = conv_out_dim(H, R, pad, stride), conv_out_dim(W, S, pad, stride)
    if rows is None:
        nr, rp, rows_arr = N * P * Q, None, None
    else:
        rows_arr = np.ascontiguousarray(rows, dtype=np.int64)
        if rows_arr.size and (rows_arr.min() < 0 or rows_arr.max() >= N * P * Q):
            raise ValueError("row index out of range")
        nr, rp = rows_arr.size, rows_arr.ctypes.data
    out = np.empty((nr, Cout), dtype=np.float64)
    if residual is not None:
        residual = _check(residual, dt, N * P * Q * Cout, "residual")
        rc = lib.oracle_conv2d_residual(N, H, W, Cin, Cout, R, S, pad, stride, dt, x.ctypes.data, w.ctypes.data,
                                        bp, residual.ctypes.data, int(relu), rp, nr, out.ctypes.data)
    else:
        rc = lib.oracle_conv2d(N, H, W, Cin, Cout, R, S, pad, stride, dt, x.ctypes.data, w.ctypes.data,
                               bp, int(relu), rp, nr, out.ctypes.data)
    if rc:
        raise RuntimeError(f"oracle_conv2d failed ({rc})")
    return out


def round_bf16(v: np.ndarray) -> np.ndarray:
    """fp64 -> bf16 bit patterns with a single round-to-nearest-even."""
    v = np.ascontiguousarray(v, dtype=np.float64)
    out = np.empty(v.shape, dtype=np.uint16)
    _load().oracle_round_bf16(v.ctypes.data, v.size, out.ctypes.data)
    return out


from .metric import (decode, gemm_row_scales, gemm_batched_row_scales, conv_row_scales, max_normalised_error)  # noqa: E402,F401
