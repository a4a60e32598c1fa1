"""Pins of the seeded input generator (CPU only)."""
import numpy as np

import seeded_inputs as si

UNIFORM_256_HASH = 0xC0D27F2CFF202114


def test_mix64_matches_published_splitmix64_stream():
    # splitmix64 seeded with 0 produces these first three outputs (test vector
    # distributed with the public-domain reference implementation).
    e = np.arange(1, 4, dtype=np.uint64)
    with np.errstate(over="ignore"):
        got = si.mix64(e * si.GOLDEN)
    assert [int(v) for v in got] == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]


def test_counter_based_and_deterministic():
    a = si.uniform(5, 0, (1000,), "f32")
    b = si.uniform(5, 0, (1000,), "f32")
    assert np.array_equal(a, b)
    # element e does not depend on how many elements are drawn
    assert np.array_equal(si.uniform(5, 0, (10,), "f32"), a[:10])
    # chunk boundary is invisible
    big = si.uniform(7, 1, (si._CHUNK + 5,), "f32")
    tail = (si.raw_bits(7, 1, si._CHUNK, 5) >> np.uint64(40)).astype(np.float64)
    assert np.array_equal(big[-5:].astype(np.float64), 2.0 * tail / 2.0 ** 24 - 1.0)
    # tensors and seeds give different streams
    assert not np.array_equal(a, si.uniform(5, 1, (1000,), "f32"))
    assert not np.array_equal(a, si.uniform(6, 0, (1000,), "f32"))


def test_uniform_range_and_moments():
    u = si.uniform(0, 0, (1 << 20,), "f32").astype(np.float64)
    assert u.min() >= -1.0 and u.max() < 1.0
    assert abs(u.mean()) < 3e-3
    assert abs(u.var() - 1.0 / 3.0) < 3e-3
    b = si.uniform(2, 2, (4096,), "f32", scale=0.1)
    assert b.min() >= -0.1 and b.max() < 0.1 and b.dtype == np.float32


def test_uniform_hash_pin():
    # integer-exact arithmetic, so the bytes are the same on every machine
    # (the expected values below are re-derived with Python integers)
    first = si.uniform(0, 0, (3,), "f32").astype(np.float64)
    key = int(si.stream_key(0, 0))
    exp = []
    for e in range(3):
        z = (key + (e + 1) * 0x9E3779B97F4A7C15) & 0xFFFFFFFFFFFFFFFF
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & 0xFFFFFFFFFFFFFFFF
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & 0xFFFFFFFFFFFFFFFF
        z ^= z >> 31
        exp.append(2.0 * ((z >> 40) / 2.0 ** 24) - 1.0)
    assert list(first) == exp
    # FNV-1a over bytes 01 02 03, worked by hand from the offset basis and prime
    assert si.fnv1a64(np.array([1, 2, 3], dtype=np.uint8)) == 0xD0AA6218672CF5AB
    # fingerprint of the first 256 uniform values of (seed 0, tensor 0)
    assert si.fnv1a64(si.uniform(0, 0, (256,), "f32")) == UNIFORM_256_HASH


def test_normal_moments_and_sigma():
    z = si.bf16_bits_to_f32(si.normal(1, 0, (1 << 20,), "bf16")).astype(np.float64)
    assert abs(z.mean()) < 4e-3
    assert abs(z.std() - 1.0) < 4e-3
    assert abs((z ** 4).mean() - 3.0) < 0.05          # kurtosis of a normal
    w = si.bf16_bits_to_f32(si.normal(2, 1, (1 << 18,), "bf16", sigma=1.0 / 24.0)).astype(np.float64)
    assert abs(w.std() * 24.0 - 1.0) < 1e-2


def test_bf16_rounding_ties_to_even():
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, -2.5, 0.0],
                 dtype=np.float32)
    bits = si.f32_to_bf16_bits(x)
    assert [int(b) for b in bits] == [0x3F80, 0x3F80, 0x3F82, 0x3F81, 0xC020, 0x0000]
    assert np.array_equal(si.bf16_bits_to_f32(bits[:1]), np.array([1.0], dtype=np.float32))


def test_workload_shapes():
    a, b = si.gemm_bf16_normal(16, 24, 32, seed=1, transB=1)
    assert a.shape == (16, 32) and b.shape == (24, 32) and a.dtype == np.uint16
    a, b = si.gemm_bf16_normal(16, 24, 32, seed=1, transA=1)
    assert a.shape == (32, 16) and b.shape == (32, 24)
    x, w, bias = si.conv_bf16(2, 5, 6, 8, 4, 3, 3, seed=2)
    assert x.shape == (2, 5, 6, 8) and w.shape == (4, 3, 3, 8) and bias.shape == (4,)
    assert bias.dtype == np.float32 and abs(bias).max() < 0.1
    v = si.small_integers(3, 0, (1000,), "bf16")
    f = si.bf16_bits_to_f32(v)
    assert f.min() >= -8 and f.max() <= 8 and np.array_equal(f, np.round(f))
