"""GPU parity of tdx_add_zero_pad (add(zero_pad(x), y) without the padded copy) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2409_03864_b200 as tdx
import seeded_inputs as si
from gpu_util import to_dev

pytestmark = pytest.mark.gpu

DT = {"f32": tdx.TDX_F32, "bf16": tdx.TDX_BF16}
# one rounding of an exact-or-fp32 sum: half an ulp of the output type, relative to |x| + |y|
EPS = {"f32": 2.0 ** -24, "bf16": 2.0 ** -8}

CASES = [
    # N, H,  W,  C,  top, bottom, left, right
    (2, 14, 14, 64, 1, 1, 1, 1),       # 16-byte rows: vector path
    (3, 7, 9, 24, 2, 0, 1, 3),         # asymmetric pads
    (1, 5, 6, 7, 1, 2, 3, 1),          # C = 7: scalar path
    (2, 8, 8, 32, 0, 0, 0, 0),         # no padding: plain add
    (1, 1, 1, 8, 3, 3, 3, 3),          # one pixel in a wide ring
    (2, 6, 5, 12, 0, 1, 0, 0),         # bf16 rows of 120 bytes: not 16-byte multiples
]


def host(a, dtype):
    return a.view(np.uint16) if dtype == "bf16" else a


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("in_place", [False, True])
def test_add_zero_pad_vs_oracle(case, dtype, in_place):
    N, H, W, C, top, bottom, left, right = case
    Hp, Wp = H + top + bottom, W + left + right
    gen = si.uniform if dtype == "f32" else si.normal
    x, y = gen(30, 0, (N, H, W, C), dtype), gen(30, 1, (N, Hp, Wp, C), dtype)
    dx, dy = to_dev(x), to_dev(y)
    dout = dy if in_place else to_dev(np.full_like(y, 0x7FC0 if dtype == "bf16" else np.nan))   # NaN canvas
    st = tdx.tdx_add_zero_pad(N, H, W, C, top, bottom, left, right, DT[dtype], dx, dy, dout)
    torch.cuda.synchronize()
    assert st == 0, tdx.tdx_last_error()
    got = oracle.decode(host(dout.cpu().numpy(), dtype), dtype).reshape(N, Hp, Wp, C)
    ref = oracle.add_zero_pad(N, H, W, C, top, bottom, left, right, dtype, x, y)
    xd = np.pad(oracle.decode(x, dtype).reshape(N, H, W, C), ((0, 0), (top, bottom), (left, right), (0, 0)))
    yd = oracle.decode(y, dtype).reshape(N, Hp, Wp, C)
    assert np.all(np.abs(got - ref) <= EPS[dtype] * (np.abs(xd) + np.abs(yd)))
    # the padding ring is y, bit for bit
    ring = np.ones((N, Hp, Wp, C), dtype=bool)
    ring[:, top:top + H, left:left + W, :] = False
    assert np.array_equal(got[ring], yd[ring])
    if not in_place:
        assert np.array_equal(host(dy.cpu().numpy(), dtype), y)          # y itself unchanged


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_add_zero_pad_exact_on_small_integers(dtype):
    N, H, W, C, p = 2, 9, 11, 16, 2
    x = si.small_integers(31, 0, (N, H, W, C), dtype, -8, 8)
    y = si.small_integers(31, 1, (N, H + 2 * p, W + 2 * p, C), dtype, -8, 8)
    dx, dy = to_dev(x), to_dev(y)
    assert tdx.tdx_add_zero_pad(N, H, W, C, p, p, p, p, DT[dtype], dx, dy, dy) == 0
    torch.cuda.synchronize()
    got = oracle.decode(host(dy.cpu().numpy(), dtype), dtype).reshape(y.shape)
    assert np.array_equal(got, oracle.add_zero_pad(N, H, W, C, p, p, p, p, dtype, x, y))


def test_add_zero_pad_in_place_launches_one_kernel_and_arguments_are_checked():
    N, H, W, C = 4, 56, 56, 64
    x, y = si.normal(32, 0, (N, H, W, C), "bf16"), si.normal(32, 1, (N, H + 2, W + 2, C), "bf16")
    dx, dy = to_dev(x), to_dev(y)
    n0 = tdx.tdx_kernel_launch_count()
    assert tdx.tdx_add_zero_pad(N, H, W, C, 1, 1, 1, 1, tdx.TDX_BF16, dx, dy, dy) == 0
    assert tdx.tdx_kernel_launch_count() - n0 == 1           # no pass over the ring, no padded copy
    torch.cuda.synchronize()
    assert tdx.tdx_add_zero_pad(N, H, W, C, -1, 1, 1, 1, tdx.TDX_BF16, dx, dy, dy) == tdx.TDX_ERR_INVALID_ARG
    assert tdx.tdx_add_zero_pad(N, H, W, C, 1, 1, 1, 1, 5, dx, dy, dy) == tdx.TDX_ERR_INVALID_ARG
    assert tdx.tdx_add_zero_pad(N, H, W, C, 1, 1, 1, 1, tdx.TDX_BF16, None, dy, dy) == tdx.TDX_ERR_INVALID_ARG
    assert tdx.tdx_add_zero_pad(0, H, W, C, 1, 1, 1, 1, tdx.TDX_BF16, None, None, None) == 0
