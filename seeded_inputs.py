"""Seeded synthetic input tensors for the dense-contraction workloads.

This module only *generates data*: it holds no matmul, convolution, epilogue or
error-metric arithmetic.  Both the CPU oracle's tests and the CUDA path's tests
draw their inputs from here so that the two sides see byte-identical buffers.

Generator (stateless, counter based):
    key   = mix64(seed * GOLDEN + tensor_id + 1)
    bits  = mix64(key + (e + 1) * GOLDEN)            for element index e
where mix64 is the finaliser of the splitmix64 generator (Steele, Lea, Flood,
"Fast splittable pseudorandom number generators", OOPSLA 2014):
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9
    z = (z ^ (z >> 27)) * 0x94D049BB133111EB
    z =  z ^ (z >> 31)

uniform[-1, 1): the top 24 bits r give u = 2 * (r / 2**24) - 1, exact in fp32.
normal(0, sigma): Box-Muller in fp64 on the two 32-bit halves of `bits`,
    u1 = (hi + 1) / 2**32 in (0, 1],  u2 = lo / 2**32 in [0, 1),
    z  = sqrt(-2 ln u1) * cos(2 pi u2) * sigma,
rounded to fp32 and then to the storage type.

Storage types: "f32" -> numpy float32; "bf16" -> numpy uint16 holding the
upper 16 bits of the fp32 pattern after round-to-nearest-even.

Tensor ids inside one workload: 0 = left operand / activations,
1 = right operand / filter, 2 = bias.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_CHUNK = 1 << 22


def _each_chunk(n: int, fill) -> None:
    """Calls fill(start, count) for every _CHUNK-sized piece of n elements; large tensors spread the pieces over a
    few threads (each piece depends only on its own element counters, so the result is the same either way)."""
    pieces = [(s, min(_CHUNK, n - s)) for s in range(0, n, _CHUNK)]
    workers = min(len(pieces), 8, len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else 4)
    if workers <= 1:
        for s, c in pieces:
            fill(s, c)
        return
    with ThreadPoolExecutor(max_workers=workers) as pool:
        list(pool.map(lambda sc: fill(*sc), pieces))


def mix64(z: np.ndarray) -> np.ndarray:
    """splitmix64 output finaliser on a uint64 array (wrapping arithmetic)."""
    z = np.asarray(z, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        z = z ^ (z >> np.uint64(31))
    return z


def stream_key(seed: int, tensor_id: int) -> np.uint64:
    with np.errstate(over="ignore"):
        k = np.uint64(seed) * GOLDEN + np.uint64(tensor_id + 1)
    return mix64(np.array([k], dtype=np.uint64))[0]


def raw_bits(seed: int, tensor_id: int, start: int, count: int) -> np.ndarray:
    """64 random bits for elements start .. start+count-1 of one tensor."""
    key = stream_key(seed, tensor_id)
    e = np.arange(start + 1, start + count + 1, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return mix64(key + e * GOLDEN)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round to nearest even. Finite inputs."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> the fp32 values they denote (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _store(x32: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "f32":
        return x32
    if dtype == "bf16":
        return f32_to_bf16_bits(x32)
    raise ValueError(f"unknown storage dtype {dtype!r}")


def uniform(seed: int, tensor_id: int, shape, dtype: str = "f32", scale: float = 1.0) -> np.ndarray:
    """i.i.d. uniform[-scale, scale) values; scale is applied in fp32."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.float32 if dtype == "f32" else np.uint16)

    def fill(s, c):
        r24 = (raw_bits(seed, tensor_id, s, c) >> np.uint64(40)).astype(np.float32)
        u = np.float32(2.0) * (r24 * np.float32(2.0 ** -24)) - np.float32(1.0)
        if scale != 1.0:
            u = u * np.float32(scale)
        out[s:s + c] = _store(u.astype(np.float32), dtype)

    _each_chunk(n, fill)
    return out.reshape(shape)


def normal(seed: int, tensor_id: int, shape, dtype: str = "f32", sigma: float = 1.0) -> np.ndarray:
    """i.i.d. normal(0, sigma) values (sigma is the standard deviation)."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.float32 if dtype == "f32" else np.uint16)

    def fill(s, c):
        b = raw_bits(seed, tensor_id, s, c)
        hi = (b >> np.uint64(32)).astype(np.float64)
        lo = (b & np.uint64(0xFFFFFFFF)).astype(np.float64)
        u1 = (hi + 1.0) * 2.0 ** -32
        u2 = lo * 2.0 ** -32
        z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2) * float(sigma)
        out[s:s + c] = _store(z.astype(np.float32), dtype)

    _each_chunk(n, fill)
    return out.reshape(shape)


def small_integers(seed: int, tensor_id: int, shape, dtype: str = "f32", lo: int = -8, hi: int = 8) -> np.ndarray:
    """Integers in [lo, hi] (exact in bf16 and fp32) for exact-arithmetic tests."""
    n = int(np.prod(shape))
    span = np.uint64(hi - lo + 1)
    v = (raw_bits(seed, tensor_id, 0, n) >> np.uint64(33)) % span
    x = (v.astype(np.int64) + lo).astype(np.float32)
    return _store(x, dtype).reshape(shape)


# ---------------------------------------------------------------------------
# The named workloads (shapes, distributions and seeds of the five configs).
# ---------------------------------------------------------------------------

def gemm_f32_uniform(M: int, N: int, K: int, seed: int = 0):
    """fp32 A (M x K) and B (K x N), uniform[-1, 1), row-major, no transpose."""
    return uniform(seed, 0, (M, K), "f32"), uniform(seed, 1, (K, N), "f32")


def gemm_bf16_normal(M: int, N: int, K: int, seed: int, transA: int = 0, transB: int = 0):
    """bf16 N(0,1) operands in the storage layout the flags imply:
    A stored K x M if transA else M x K; B stored N x K if transB else K x N."""
    a_shape = (K, M) if transA else (M, K)
    b_shape = (N, K) if transB else (K, N)
    return normal(seed, 0, a_shape, "bf16"), normal(seed, 1, b_shape, "bf16")


def conv_bf16(N: int, H: int, W: int, Cin: int, Cout: int, R: int, S: int, seed: int):
    """NHWC bf16 activations N(0,1); KRSC bf16 filter N(0, sigma = 1/sqrt(Cin*R*S));
    fp32 bias uniform[-0.1, 0.1)."""
    x = normal(seed, 0, (N, H, W, Cin), "bf16")
    w = normal(seed, 1, (Cout, R, S, Cin), "bf16", sigma=1.0 / np.sqrt(Cin * R * S))
    bias = uniform(seed, 2, (Cout,), "f32", scale=0.1)
    return x, w, bias


def fnv1a64(buf: np.ndarray) -> int:
    """FNV-1a hash (64 bit) of an array's bytes; used to pin generated inputs."""
    data = np.ascontiguousarray(buf).view(np.uint8).ravel()
    h = 0xCBF29CE484222325
    for byte in data.tolist():
        h = ((h ^ byte) * 0x100000001B3) & 0xFFFFFFFFFFFFFFFF
    return h
