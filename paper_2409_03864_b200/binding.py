"""ctypes binding of libtdx.so: argument marshalling only, same names as include/tdx.h.

Pointers may be given as torch tensors (their data_ptr() is used), numpy arrays (for the *_host
entry points), integers or None.  Streams may be a torch.cuda.Stream, an integer handle or None.
Every function returns the library's status code unless stated otherwise; `check()` turns a
non-zero status into a TdxError carrying tdx_last_error().
"""
from __future__ import annotations

import ctypes
import os
from pathlib import Path

_LIB_PATH = Path(__file__).resolve().parent / "libtdx.so"

TDX_OK = 0
TDX_ERR_INVALID_ARG = 1
TDX_ERR_UNSUPPORTED = 2
TDX_ERR_ALIGNMENT = 3
TDX_ERR_CONFIG = 4
TDX_ERR_WORKSPACE = 5
TDX_ERR_CUDA = 16
TDX_ERR_TIMEOUT = 17
TDX_ERR_NO_DEVICE = 18
TDX_ERR_BOUNDS = 19

TDX_F32 = 0
TDX_BF16 = 1

TDX_KERNEL_AUTO = 0
TDX_KERNEL_UMMA = 1
TDX_KERNEL_SIMT = 2
TDX_KERNEL_GENERIC = 3


class TdxError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"tdx status {status}: {message}")
        self.status = status


class tdx_config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in
                ("kernel", "tile_m", "tile_n", "tile_k", "stages", "cta_pair", "split_k", "store_mode", "raster",
                 "patch_w", "patch_h", "k_stagger", "halo", "fit")]

    def as_dict(self) -> dict:
        return {n: int(getattr(self, n)) for n, _ in self._fields_}

    def __repr__(self) -> str:
        return "tdx_config(" + ", ".join(f"{k}={v}" for k, v in self.as_dict().items()) + ")"


_lib = None


def lib() -> ctypes.CDLL:
    """Load libtdx.so (built in-tree by paper_2409_03864_b200.build).  Fails loudly if it is missing."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise FileNotFoundError(
                f"{_LIB_PATH} is missing: run `python -m paper_2409_03864_b200.build` (there is no fallback path)")
        L = ctypes.CDLL(str(_LIB_PATH))
        i64, ci, cf, vp, sz = ctypes.c_int64, ctypes.c_int, ctypes.c_float, ctypes.c_void_p, ctypes.c_size_t
        cfgp = ctypes.POINTER(tdx_config)
        fp = ctypes.POINTER(ctypes.c_float)
        ip = ctypes.POINTER(ctypes.c_int)
        gemm_args = [i64, i64, i64, ci, ci, cf, ci, vp, vp, vp, vp]
        conv_args = [i64] * 7 + [ci, ci, ci, vp, vp, vp, ci, vp, vp]
        L.tdx_gemm.argtypes = gemm_args
        L.tdx_gemm_ex.argtypes = gemm_args + [cfgp, vp, sz]
        L.tdx_gemm_batched.argtypes = [i64, i64, i64, i64, ci, ci, cf, cf, ci, vp, i64, vp, i64, vp, i64, vp]
        L.tdx_gemm_batched_host.argtypes = [i64, i64, i64, i64, ci, ci, cf, cf, ci, vp, vp, vp, vp]
        L.tdx_add_zero_pad.argtypes = [i64, i64, i64, i64, ci, ci, ci, ci, ci, vp, vp, vp, vp]
        L.tdx_add_zero_pad_host.argtypes = [i64, i64, i64, i64, ci, ci, ci, ci, ci, vp, vp, vp]
        L.tdx_gemm_f32out.argtypes = [i64, i64, i64, ci, ci, cf, vp, vp, vp, vp]
        L.tdx_gemm_workspace_size.argtypes = [i64, i64, i64, ci, cfgp, ctypes.POINTER(sz)]
        L.tdx_conv2d_bias_relu.argtypes = conv_args
        L.tdx_conv2d_bias_relu_ex.argtypes = conv_args + [cfgp]
        L.tdx_conv2d_bias_add_relu.argtypes = [i64] * 7 + [ci, ci, ci, vp, vp, vp, vp, ci, vp, vp, cfgp]
        L.tdx_gemm_host.argtypes = gemm_args
        L.tdx_conv2d_bias_relu_host.argtypes = conv_args
        L.tdx_tune_gemm.argtypes = [i64, i64, i64, ci, ci, ci, ci, cfgp, fp, cfgp, fp, ci, ip, vp]
        L.tdx_tune_gemm_guided.argtypes = [i64, i64, i64, ci, ci, ci, ci, ci, cfgp, fp, cfgp, fp, ci, ip, ip, vp]
        L.tdx_model_gemm_us.argtypes = [i64, i64, i64, ci, ci, ci, cfgp, ci, ctypes.POINTER(ctypes.c_double)]
        L.tdx_tune_conv2d.argtypes = [i64] * 7 + [ci, ci, ci, ci, cfgp, fp, cfgp, fp, ci, ip, vp]
        L.tdx_enum_gemm_configs.argtypes = [i64, i64, i64, ci, ci, ci, cfgp, ci, ip]
        L.tdx_enum_conv2d_configs.argtypes = [i64] * 7 + [ci, ci, ci, cfgp, ci, ip]
        L.tdx_default_gemm_config.argtypes = [i64, i64, i64, ci, ci, ci, cfgp]
        L.tdx_default_conv2d_config.argtypes = [i64] * 7 + [ci, ci, ci, cfgp]
        L.tdx_tune_save.argtypes = [ctypes.c_char_p]
        L.tdx_tune_load.argtypes = [ctypes.c_char_p]
        L.tdx_tune_clear.argtypes = []
        L.tdx_set_autotune.argtypes = [ci]
        dp = ctypes.POINTER(ctypes.c_double)
        L.tdx_gemm_tile_plan.argtypes = [i64, i64, i64, ci, ci, ci, ci, ip, ci, ip, ip, dp, dp]
        L.tdx_tune_conv2d_guided.argtypes = [i64] * 7 + [ci, ci, ci, ci, ci, cfgp, fp, cfgp, fp, ci, ip, ip, vp]
        L.tdx_model_conv2d_us.argtypes = [i64] * 7 + [ci, ci, ci, cfgp, ci, ctypes.POINTER(ctypes.c_double)]
        L.tdx_enum_gemm_space.argtypes = [i64, i64, i64, ci, ci, ci, ctypes.c_char_p, cfgp, ci, ip, ctypes.POINTER(i64), ctypes.POINTER(i64)]
        L.tdx_tune_gemm_space.argtypes = [i64, i64, i64, ci, ci, ci, ctypes.c_char_p, ci, ci, cfgp, fp, cfgp, fp, ci, ip, ip, vp]
        L.tdx_gemm_k_balanced_plan.argtypes = [i64, i64, i64, ci, ci, ci, ip, ci, ip, ip, ip]
        L.tdx_gemm_splitk_static.argtypes = [i64, i64, i64, ci, ci, cf, vp, vp, vp, ci, ci, vp]
        L.tdx_check_device_status.argtypes = [vp]
        L.tdx_selftest_bounded_wait.argtypes = [ci, vp]
        L.tdx_selftest_bounds_check.argtypes = [vp]
        L.tdx_kernel_launch_count.argtypes = []
        L.tdx_kernel_launch_count.restype = i64
        L.tdx_last_error.restype = ctypes.c_char_p
        L.tdx_version.restype = ctypes.c_char_p
        for name in EXPORTS:
            fn = getattr(L, name)
            if name not in ("tdx_kernel_launch_count", "tdx_last_error", "tdx_version"):
                fn.restype = ci
        _lib = L
        # Tuned tile configurations measured on B200 ship next to the library; TDX_TUNE_CACHE names another
        # file, or "0" for none.  A missing or unreadable file only means the library's automatic choice is used.
        cache = os.environ.get("TDX_TUNE_CACHE", str(_LIB_PATH.parent / "tuned_b200.json"))
        if cache != "0" and os.path.exists(cache):
            L.tdx_tune_load(cache.encode())
    return _lib


# every symbol include/tdx.h declares
EXPORTS = (
    "tdx_gemm", "tdx_gemm_f32out", "tdx_add_zero_pad", "tdx_add_zero_pad_host", "tdx_gemm_batched", "tdx_gemm_batched_host", "tdx_gemm_ex", "tdx_gemm_workspace_size", "tdx_conv2d_bias_relu", "tdx_conv2d_bias_add_relu", "tdx_conv2d_bias_relu_ex",
    "tdx_gemm_host", "tdx_conv2d_bias_relu_host", "tdx_tune_gemm", "tdx_tune_gemm_guided", "tdx_model_gemm_us", "tdx_tune_conv2d", "tdx_enum_gemm_configs",
    "tdx_enum_conv2d_configs", "tdx_default_gemm_config", "tdx_default_conv2d_config", "tdx_tune_save",
    "tdx_tune_load", "tdx_tune_clear", "tdx_set_autotune", "tdx_gemm_tile_plan", "tdx_gemm_k_balanced_plan", "tdx_enum_gemm_space", "tdx_tune_gemm_space", "tdx_tune_conv2d_guided", "tdx_model_conv2d_us", "tdx_gemm_splitk_static", "tdx_check_device_status", "tdx_selftest_bounded_wait", "tdx_selftest_bounds_check", "tdx_kernel_launch_count", "tdx_last_error",
    "tdx_version",
)


def _ptr(x):
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if hasattr(x, "ctypes"):
        return x.ctypes.data
    raise TypeError(f"cannot take a pointer from {type(x)}")


def _stream(s):
    if s is None:
        return None
    if isinstance(s, int):
        return s
    return s.cuda_stream


def _cfg(c):
    return None if c is None else ctypes.byref(c)


def tdx_last_error() -> str:
    return lib().tdx_last_error().decode()


def tdx_version() -> str:
    return lib().tdx_version().decode()


def check(status: int) -> int:
    if status != TDX_OK:
        raise TdxError(status, tdx_last_error())
    return status


def tdx_gemm(M, N, K, transA, transB, alpha, dtype, A, B, C, stream=None) -> int:
    return lib().tdx_gemm(M, N, K, transA, transB, alpha, dtype, _ptr(A), _ptr(B), _ptr(C), _stream(stream))


def tdx_gemm_ex(M, N, K, transA, transB, alpha, dtype, A, B, C, stream=None, cfg=None, workspace=None,
                workspace_bytes=0) -> int:
    return lib().tdx_gemm_ex(M, N, K, transA, transB, alpha, dtype, _ptr(A), _ptr(B), _ptr(C), _stream(stream),
                             _cfg(cfg), _ptr(workspace), workspace_bytes)


def tdx_gemm_batched(batch, M, N, K, transA, transB, alpha, beta, dtype, A, B, C, strideA=None, strideB=None,
                     strideC=None, stream=None) -> int:
    """C[b] = beta * C[b] + alpha * op(A[b]) . op(B[b]); strides in elements, dense by default."""
    sa = M * K if strideA is None else strideA
    sb = K * N if strideB is None else strideB
    sc = M * N if strideC is None else strideC
    return lib().tdx_gemm_batched(batch, M, N, K, transA, transB, alpha, beta, dtype, _ptr(A), sa, _ptr(B), sb, _ptr(C),
                                  sc, _stream(stream))


def tdx_gemm_batched_host(batch, M, N, K, transA, transB, alpha, beta, dtype, A, B, C, stream=None) -> int:
    """A, B, C are dense host arrays (numpy, or pinned torch CPU tensors)."""
    return lib().tdx_gemm_batched_host(batch, M, N, K, transA, transB, alpha, beta, dtype, _ptr(A), _ptr(B), _ptr(C),
                                       _stream(stream))


def tdx_add_zero_pad(N, H, W, C, pad_top, pad_bottom, pad_left, pad_right, dtype, x, y, out, stream=None) -> int:
    """out = zero_pad(x) + y without building the padded copy; out may be y (in place: the ring is untouched)."""
    return lib().tdx_add_zero_pad(N, H, W, C, pad_top, pad_bottom, pad_left, pad_right, dtype, _ptr(x), _ptr(y), _ptr(out),
                                  _stream(stream))


def tdx_add_zero_pad_host(N, H, W, C, pad_top, pad_bottom, pad_left, pad_right, dtype, x, y, stream=None) -> int:
    """In place on host arrays: y = zero_pad(x) + y."""
    return lib().tdx_add_zero_pad_host(N, H, W, C, pad_top, pad_bottom, pad_left, pad_right, dtype, _ptr(x), _ptr(y),
                                       _stream(stream))


def tdx_gemm_f32out(M, N, K, transA, transB, alpha, A, B, C, stream=None) -> int:
    """bf16 A and B, fp32 C = alpha * op(A) . op(B) (the accumulator without the rounding to bf16)."""
    return lib().tdx_gemm_f32out(M, N, K, transA, transB, alpha, _ptr(A), _ptr(B), _ptr(C), _stream(stream))


def tdx_gemm_workspace_size(M, N, K, dtype, cfg):
    """Returns (status, bytes)."""
    out = ctypes.c_size_t(0)
    st = lib().tdx_gemm_workspace_size(M, N, K, dtype, _cfg(cfg), ctypes.byref(out))
    return st, int(out.value)


def tdx_conv2d_bias_relu(N, H, W, Cin, Cout, R, S, pad, stride, dtype, x, w, bias, relu, y, stream=None) -> int:
    return lib().tdx_conv2d_bias_relu(N, H, W, Cin, Cout, R, S, pad, stride, dtype, _ptr(x), _ptr(w), _ptr(bias),
                                      relu, _ptr(y), _stream(stream))


def tdx_conv2d_bias_add_relu(N, H, W, Cin, Cout, R, S, pad, stride, dtype, x, w, bias, residual, relu, y, stream=None,
                             cfg=None) -> int:
    """y = relu?(conv(x, w) + bias + residual); residual is N*P*Q x Cout in the type of y, or None."""
    return lib().tdx_conv2d_bias_add_relu(N, H, W, Cin, Cout, R, S, pad, stride, dtype, _ptr(x), _ptr(w), _ptr(bias),
                                          _ptr(residual), relu, _ptr(y), _stream(stream), _cfg(cfg))


def tdx_conv2d_bias_relu_ex(N, H, W, Cin, Cout, R, S, pad, stride, dtype, x, w, bias, relu, y, stream=None,
                            cfg=None) -> int:
    return lib().tdx_conv2d_bias_relu_ex(N, H, W, Cin, Cout, R, S, pad, stride, dtype, _ptr(x), _ptr(w), _ptr(bias),
                                         relu, _ptr(y), _stream(stream), _cfg(cfg))


def tdx_gemm_host(M, N, K, transA, transB, alpha, dtype, A_host, B_host, C_host, stream=None) -> int:
    return lib().tdx_gemm_host(M, N, K, transA, transB, alpha, dtype, _ptr(A_host), _ptr(B_host), _ptr(C_host),
                               _stream(stream))


def tdx_conv2d_bias_relu_host(N, H, W, Cin, Cout, R, S, pad, stride, dtype, x_host, w_host, bias_host, relu, y_host,
                              stream=None) -> int:
    return lib().tdx_conv2d_bias_relu_host(N, H, W, Cin, Cout, R, S, pad, stride, dtype, _ptr(x_host), _ptr(w_host),
                                           _ptr(bias_host), relu, _ptr(y_host), _stream(stream))


def _tune(call, cap):
    best, best_us = tdx_config(), ctypes.c_float(0)
    tried = (tdx_config * cap)()
    tried_us = (ctypes.c_float * cap)()
    n = ctypes.c_int(0)
    st = call(ctypes.byref(best), ctypes.byref(best_us), tried, tried_us, cap, ctypes.byref(n))
    k = min(int(n.value), cap)
    return st, best, float(best_us.value), [(tried[i].as_dict(), float(tried_us[i])) for i in range(k)]


def tdx_tune_gemm(M, N, K, transA, transB, dtype, iters=20, stream=None, cap=512):
    """Returns (status, best tdx_config, best microseconds, [(config dict, microseconds), ...])."""
    L = lib()
    return _tune(lambda b, bu, t, tu, c, n: L.tdx_tune_gemm(M, N, K, transA, transB, dtype, iters, b, bu, t, tu, c, n,
                                                            _stream(stream)), cap)


def tdx_tune_gemm_guided(M, N, K, transA, transB, dtype, budget, iters=20, stream=None, cap=512):
    """Returns (status, best tdx_config, best microseconds, [(config dict, microseconds), ...], size of the full space)."""
    L = lib()
    n_cand = ctypes.c_int(0)
    st, best, us, tried = _tune(lambda b, bu, t, tu, c, n: L.tdx_tune_gemm_guided(
        M, N, K, transA, transB, dtype, iters, budget, b, bu, t, tu, c, n, ctypes.byref(n_cand), _stream(stream)), cap)
    return st, best, us, tried, int(n_cand.value)


def tdx_set_autotune(budget: int) -> int:
    """Search on first use: 0 off (default), > 0 guided search with that budget, < 0 exhaustive."""
    return lib().tdx_set_autotune(int(budget))


def tdx_model_gemm_us(M, N, K, transA, transB, dtype, cfg, ctas=148):
    """Returns (status, predicted microseconds) of the cost model that ranks the guided search (host only)."""
    us = ctypes.c_double(0.0)
    st = lib().tdx_model_gemm_us(M, N, K, transA, transB, dtype, _cfg(cfg), ctas, ctypes.byref(us))
    return st, float(us.value)


def tdx_tune_conv2d(N, H, W, Cin, Cout, R, S, pad, stride, dtype, iters=20, stream=None, cap=512):
    L = lib()
    return _tune(lambda b, bu, t, tu, c, n: L.tdx_tune_conv2d(N, H, W, Cin, Cout, R, S, pad, stride, dtype, iters, b,
                                                              bu, t, tu, c, n, _stream(stream)), cap)


def tdx_tune_conv2d_guided(N, H, W, Cin, Cout, R, S, pad, stride, dtype, budget, iters=20, stream=None, cap=512):
    """Returns (status, best tdx_config, best microseconds, [(config dict, microseconds), ...], size of the full space)."""
    L = lib()
    n_cand = ctypes.c_int(0)
    st, best, us, tried = _tune(lambda b, bu, t, tu, c, n: L.tdx_tune_conv2d_guided(
        N, H, W, Cin, Cout, R, S, pad, stride, dtype, iters, budget, b, bu, t, tu, c, n, ctypes.byref(n_cand), _stream(stream)), cap)
    return st, best, us, tried, int(n_cand.value)


def tdx_model_conv2d_us(N, H, W, Cin, Cout, R, S, pad, stride, dtype, cfg, ctas=148):
    """Returns (status, predicted microseconds) of the convolution cost model (host only)."""
    us = ctypes.c_double(0.0)
    st = lib().tdx_model_conv2d_us(N, H, W, Cin, Cout, R, S, pad, stride, dtype, _cfg(cfg), ctas, ctypes.byref(us))
    return st, float(us.value)


def _enum(call, cap=8192):
    out = (tdx_config * cap)()
    n = ctypes.c_int(0)
    st = call(out, cap, ctypes.byref(n))
    return st, [out[i].as_dict() for i in range(min(cap, int(n.value)))]


def tdx_enum_gemm_configs(M, N, K, transA, transB, dtype):
    """Returns (status, [config dict, ...])."""
    L = lib()
    return _enum(lambda o, c, n: L.tdx_enum_gemm_configs(M, N, K, transA, transB, dtype, o, c, n))


def tdx_enum_conv2d_configs(N, H, W, Cin, Cout, R, S, pad, stride, dtype):
    L = lib()
    return _enum(lambda o, c, n: L.tdx_enum_conv2d_configs(N, H, W, Cin, Cout, R, S, pad, stride, dtype, o, c, n))


def tdx_enum_gemm_space(M, N, K, transA, transB, dtype, space: str, cap=8192):
    """Returns (status, [config dict, ...], size of the cross product, how many pass the stated rules)."""
    out = (tdx_config * cap)()
    n, prod, kept = ctypes.c_int(0), ctypes.c_int64(0), ctypes.c_int64(0)
    st = lib().tdx_enum_gemm_space(M, N, K, transA, transB, dtype, space.encode(), out, cap, ctypes.byref(n), ctypes.byref(prod),
                                   ctypes.byref(kept))
    return st, [out[i].as_dict() for i in range(min(cap, int(n.value)))], int(prod.value), int(kept.value)


def tdx_tune_gemm_space(M, N, K, transA, transB, dtype, space: str, budget=0, iters=20, stream=None, cap=512):
    """Searches the stated space; returns (status, best, best microseconds, [(config dict, microseconds), ...], candidates)."""
    L = lib()
    n_cand = ctypes.c_int(0)
    st, best, us, tried = _tune(lambda b, bu, t, tu, c, n: L.tdx_tune_gemm_space(
        M, N, K, transA, transB, dtype, space.encode(), iters, budget, b, bu, t, tu, c, n, ctypes.byref(n_cand), _stream(stream)), cap)
    return st, best, us, tried, int(n_cand.value)


def tdx_default_gemm_config(M, N, K, transA, transB, dtype):
    """Returns (status, tdx_config)."""
    c = tdx_config()
    return lib().tdx_default_gemm_config(M, N, K, transA, transB, dtype, ctypes.byref(c)), c


def tdx_default_conv2d_config(N, H, W, Cin, Cout, R, S, pad, stride, dtype):
    c = tdx_config()
    return lib().tdx_default_conv2d_config(N, H, W, Cin, Cout, R, S, pad, stride, dtype, ctypes.byref(c)), c


def tdx_tune_save(path: str) -> int:
    return lib().tdx_tune_save(str(path).encode())


def tdx_tune_load(path: str) -> int:
    return lib().tdx_tune_load(str(path).encode())


def tdx_tune_clear() -> int:
    return lib().tdx_tune_clear()


def tdx_gemm_tile_plan(M, N, K, tile_m=256, tile_n=256, raster=0, ctas=148, cap_tiles=1 << 16):
    """-> (status, rounds, ctas_used, tiles, model_cycles, model_cycles_uniform); tiles[round][cta] =
    (row block, first column, width), width 0 = no tile; rounds = 0 when the uniform grid is kept."""
    table = (ctypes.c_int * (3 * cap_tiles))()
    rounds, used = ctypes.c_int(0), ctypes.c_int(0)
    fit, uni = ctypes.c_double(0.0), ctypes.c_double(0.0)
    st = lib().tdx_gemm_tile_plan(M, N, K, tile_m, tile_n, raster, ctas, table, cap_tiles, ctypes.byref(rounds),
                                  ctypes.byref(used), ctypes.byref(fit), ctypes.byref(uni))
    tiles = [[(table[3 * (r * used.value + c)], table[3 * (r * used.value + c) + 1], table[3 * (r * used.value + c) + 2])
              for c in range(used.value)] for r in range(rounds.value)]
    return st, rounds.value, used.value, tiles, fit.value, uni.value


def tdx_gemm_k_balanced_plan(M, N, K, tile_m=128, tile_n=128, ctas=148, cap_entries=1 << 14):
    """-> (status, rounds, ctas_used, entries, max_slots); entries[round][cta] = (row block, first column, width,
    first K block, end K block, partial slot), width 0 = no entry."""
    table = (ctypes.c_int * (6 * cap_entries))()
    rounds, used, slots = ctypes.c_int(0), ctypes.c_int(0), ctypes.c_int(0)
    st = lib().tdx_gemm_k_balanced_plan(M, N, K, tile_m, tile_n, ctas, table, cap_entries, ctypes.byref(rounds), ctypes.byref(used),
                                        ctypes.byref(slots))
    ent = [[tuple(table[6 * (r * used.value + c) + i] for i in range(6)) for c in range(used.value)] for r in range(rounds.value)]
    return st, rounds.value, used.value, ent, slots.value


TDX_STATIC_SCRATCH_BYTES = 16 * 1024 * 1024


def tdx_gemm_splitk_static(M, N, K, transA, transB, alpha, A, B, C, tile_n=0, split_k=2, stream=None) -> int:
    """bf16 split-K GEMM that allocates no device memory: its partial sums live in a fixed
    TDX_STATIC_SCRATCH_BYTES array inside the library, for callers that may not call cudaMalloc
    (fixed memory budgets, code living inside another allocator's pool).  Calls that can overlap
    on the GPU race on that array; keep them ordered on one stream."""
    return lib().tdx_gemm_splitk_static(M, N, K, transA, transB, alpha, _ptr(A), _ptr(B), _ptr(C), tile_n, split_k,
                                        _stream(stream))


def tdx_check_device_status(stream=None) -> int:
    return lib().tdx_check_device_status(_stream(stream))


def tdx_selftest_bounded_wait(limit_us=200, stream=None) -> int:
    return lib().tdx_selftest_bounded_wait(limit_us, _stream(stream))


def tdx_selftest_bounds_check(stream=None) -> int:
    return lib().tdx_selftest_bounds_check(_stream(stream))


def tdx_kernel_launch_count() -> int:
    return int(lib().tdx_kernel_launch_count())
