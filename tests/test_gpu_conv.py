"""GPU parity of tdx_conv2d_bias_relu against the CPU oracle (through the C ABI)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2409_03864_b200 as tdx
import seeded_inputs as si
from gpu_util import TIGHT, TOL, GuardedOut, conv_error, run_conv, structured_rows, to_dev

pytestmark = pytest.mark.gpu


def umma(**kw):
    return tdx.tdx_config(kernel=tdx.TDX_KERNEL_UMMA, **kw)


def test_conv_delta_filter_is_exact_shifted_copy():
    # w[k, r0, s0, c] = delta(c, k): the output is the input shifted by (r0 - pad, s0 - pad) with zeros
    # shifted in from the padding -- exact in bf16, so the comparison is bitwise.
    N, H, W, C, pad = 2, 12, 20, 64, 1
    x = si.normal(70, 0, (N, H, W, C), "bf16")
    for r0, s0 in [(0, 0), (1, 1), (2, 0), (0, 2)]:
        w = np.zeros((C, 3, 3, C), dtype=np.float32)
        for k in range(C):
            w[k, r0, s0, k] = 1.0
        wb = si.f32_to_bf16_bits(w)
        st, y, ok = run_conv(N, H, W, C, C, 3, 3, pad, 1, "bf16", x, wb, None, 0, cfg=umma())
        assert st == 0 and ok, tdx.tdx_last_error()
        exp = np.zeros((N, H, W, C), dtype=np.uint16)
        dh, dw = r0 - pad, s0 - pad
        hs, ws = slice(max(0, -dh), min(H, H - dh)), slice(max(0, -dw), min(W, W - dw))
        hd, wd = slice(max(0, dh), min(H, H + dh)), slice(max(0, dw), min(W, W + dw))
        exp[:, hs, ws, :] = x[:, hd, wd, :]
        y = y.reshape(N, H, W, C)
        nz = (exp & 0x7FFF) != 0
        assert np.array_equal(y[nz], exp[nz]) and ((y[~nz] & 0x7FFF) == 0).all(), (r0, s0)


CASES = [
    # N, H,  W,  Cin, Cout, R, S, pad
    (1, 8, 8, 64, 64, 3, 3, 1),
    (2, 14, 14, 128, 96, 3, 3, 1),       # 14 x 14 maps: ragged 8 x 8 patches; tile_n = 96 or 128 with a tail
    (3, 7, 7, 64, 32, 3, 3, 1),          # patches spanning several images in one tile
    (1, 20, 36, 72, 40, 3, 3, 1),        # Cin not a multiple of 64: zero-filled channel tail
    (2, 9, 17, 8, 8, 1, 1, 0),           # 1 x 1 filter, tiny channel count
    (1, 16, 16, 64, 64, 5, 5, 2),
    (1, 16, 24, 64, 72, 3, 5, 0),        # no padding, non-square filter
    (1, 10, 130, 64, 64, 3, 3, 1),       # wide rows: 128-wide patches with a ragged tail
    (1, 6, 6, 64, 36, 3, 3, 2),          # pad larger than the usual (R - 1) / 2; Cout % 8 != 0 -> scalar stores
]


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("bias_relu", [(True, 1), (False, 0)])
def test_conv_small_cases_vs_oracle(case, bias_relu):
    N, H, W, Cin, Cout, R, S, pad = case
    use_bias, relu = bias_relu
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, R, S, seed=71)
    bias = b if use_bias else None
    st, y, ok = run_conv(N, H, W, Cin, Cout, R, S, pad, 1, "bf16", x, w, bias, relu, cfg=umma())
    assert st == 0 and ok, tdx.tdx_last_error()
    err = conv_error(N, H, W, Cin, Cout, R, S, pad, 1, "bf16", x, w, bias, relu, y)
    assert err < TOL["bf16"] and err < TIGHT["bf16"], err


@pytest.mark.parametrize("patch", [(8, 8), (16, 8), (8, 16), (32, 4), (128, 1), (8, 1), (16, 2)])
def test_conv_patch_shapes(patch):
    N, H, W, Cin, Cout = 2, 24, 40, 64, 64
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, 3, 3, seed=72)
    st, y, ok = run_conv(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1,
                         cfg=umma(patch_w=patch[0], patch_h=patch[1], tile_n=64, stages=3))
    assert st == 0 and ok, tdx.tdx_last_error()
    assert conv_error(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1, y) < TIGHT["bf16"]


@pytest.mark.parametrize("cfgkw", [dict(tile_n=64, patch_w=8, patch_h=8), dict(tile_n=128, patch_w=16, patch_h=8),
                                   dict(tile_n=256, patch_w=128, patch_h=1)])
def test_conv_256_row_tiles(cfgkw):
    N, H, W, Cin, Cout = 3, 24, 40, 128, 200
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, 3, 3, seed=77)
    st, y, ok = run_conv(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1, cfg=umma(tile_m=256, **cfgkw))
    assert st == 0 and ok, tdx.tdx_last_error()
    assert conv_error(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1, y) < TIGHT["bf16"]


@pytest.mark.parametrize("patch", [(8, 8), (32, 1), (16, 4), (64, 2), (128, 1), (8, 4)])
def test_conv_store_modes_agree(patch):
    # ragged 30 x 44 maps: patches hang over the right and bottom edges and over the last image
    N, H, W, Cin, Cout = 3, 30, 44, 64, 128
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, 3, 3, seed=79)
    outs = []
    for sm in (1, 2):
        st, y, ok = run_conv(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1,
                             cfg=umma(patch_w=patch[0], patch_h=patch[1], tile_n=64, store_mode=sm))
        assert st == 0 and ok, tdx.tdx_last_error()
        assert conv_error(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1, y) < TIGHT["bf16"]
        outs.append(y)
    assert np.array_equal(outs[0], outs[1])


HALO_CASES = [
    # N, H,  W,  Cin, Cout, R, S, pad
    (2, 16, 8, 64, 64, 3, 3, 1),          # exactly one 8 x 16 patch per image
    (3, 56, 56, 128, 96, 3, 3, 1),        # 56 = 3.5 patches high: ragged last patch row
    (1, 20, 36, 72, 40, 3, 3, 1),         # channel tail, ragged both ways
    (2, 30, 44, 64, 128, 5, 5, 2),        # 5 x 5 window
    (1, 24, 24, 64, 64, 3, 5, 0),         # no padding, non-square filter
    (1, 7, 7, 256, 256, 3, 3, 1),         # image smaller than a patch
    (1, 33, 17, 64, 72, 1, 3, 1),         # single filter row
    (5, 9, 12, 64, 32, 3, 3, 1),          # stacked: 10 rows per image, patches straddle up to three images
    (3, 12, 8, 64, 64, 3, 3, 2),          # padding wider than R - 1 - pad: more output rows than H + pad
    (4, 20, 16, 64, 64, 5, 3, 0),         # no padding: the rows between images are R - 1 discarded outputs
]


@pytest.mark.parametrize("case", HALO_CASES)
@pytest.mark.parametrize("tile_m", [128, 256])
@pytest.mark.parametrize("halo", [2, 3])
def test_conv_halo_reuse_vs_oracle(case, tile_m, halo):
    # the input window of a patch is loaded once per channel chunk and every filter tap reads it from shared memory;
    # halo 3 cuts the patches from the column of all images, so a patch may cover the seam between two images
    N, H, W, Cin, Cout, R, S, pad = case
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, R, S, seed=80)
    st, y, ok = run_conv(N, H, W, Cin, Cout, R, S, pad, 1, "bf16", x, w, b, 1, cfg=umma(halo=halo, tile_m=tile_m))
    assert st == 0 and ok, tdx.tdx_last_error()
    err = conv_error(N, H, W, Cin, Cout, R, S, pad, 1, "bf16", x, w, b, 1, y)
    assert err < TOL["bf16"] and err < TIGHT["bf16"], err


def test_conv_halo_reuse_equals_per_tap_loads_bitwise_for_one_channel_chunk():
    # with Cin <= 64 both kernels add the taps in the same order
    N, H, W, Cin, Cout = 2, 40, 24, 64, 64
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, 3, 3, seed=81)
    _, y1, _ = run_conv(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1, cfg=umma(halo=1, patch_w=8, patch_h=16))
    st, y2, ok = run_conv(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1, cfg=umma(halo=2, tile_n=64, stages=2))
    assert st == 0 and ok, tdx.tdx_last_error()
    assert np.array_equal(y1, y2)
    st, y3, ok = run_conv(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1, cfg=umma(halo=3, tile_n=64, stages=2))
    assert st == 0 and ok, tdx.tdx_last_error()
    assert np.array_equal(y1, y3)
    # a 1 x 1 filter has nothing to reuse: the halo kernel is refused, output untouched
    st, _, untouched = run_conv(N, H, W, Cin, Cout, 1, 1, 0, 1, "bf16", x, si.normal(82, 1, (Cout, 1, 1, Cin), "bf16"), b, 1,
                                cfg=umma(halo=2))
    assert st == tdx.TDX_ERR_CONFIG and untouched


def test_conv_staggered_k_order():
    N, H, W, Cin, Cout = 8, 28, 28, 192, 128
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, 3, 3, seed=78)
    for tm in (128, 256):
        st, y, ok = run_conv(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1, cfg=umma(tile_m=tm, k_stagger=1))
        assert st == 0 and ok, tdx.tdx_last_error()
        assert conv_error(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1, y) < TIGHT["bf16"]


def test_conv_padding_equals_explicit_zero_padded_copy_bitwise():
    # the copy engine's zero fill and explicit zeros feed the same products in the same order
    N, H, W, Cin, Cout, pad = 2, 16, 24, 64, 64, 1
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, 3, 3, seed=73)
    _, y1, _ = run_conv(N, H, W, Cin, Cout, 3, 3, pad, 1, "bf16", x, w, b, 1, cfg=umma(patch_w=8, patch_h=8))
    xp = np.zeros((N, H + 2 * pad, W + 2 * pad, Cin), dtype=np.uint16)
    xp[:, pad:pad + H, pad:pad + W, :] = x
    _, y2, _ = run_conv(N, H + 2 * pad, W + 2 * pad, Cin, Cout, 3, 3, 0, 1, "bf16", xp, w, b, 1,
                        cfg=umma(patch_w=8, patch_h=8))
    assert np.array_equal(y1, y2)


STRIDED_CASES = [
    # N, H,  W,  Cin, Cout, R, S, pad, stride
    (2, 56, 56, 64, 128, 3, 3, 1, 2),        # a ResNet-style down-sampling 3 x 3
    (3, 57, 41, 72, 40, 3, 3, 1, 2),         # odd sizes: ragged patches, channel tail
    (2, 28, 28, 128, 256, 1, 1, 0, 2),       # strided 1 x 1 (projection shortcut)
    (1, 40, 40, 64, 64, 5, 5, 2, 3),         # stride 3, 5 x 5
    (2, 17, 23, 64, 32, 2, 4, 0, 2),         # no padding, even filter
]


@pytest.mark.parametrize("case", STRIDED_CASES)
@pytest.mark.parametrize("tile_m", [128, 256])
def test_conv_strided_on_the_tensor_cores(case, tile_m):
    # per-tap loads whose copies walk the image with the convolution's stride
    N, H, W, Cin, Cout, R, S, pad, stride = case
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, R, S, seed=83)
    st, y, ok = run_conv(N, H, W, Cin, Cout, R, S, pad, stride, "bf16", x, w, b, 1, cfg=umma(tile_m=tile_m))
    assert st == 0 and ok, tdx.tdx_last_error()
    err = conv_error(N, H, W, Cin, Cout, R, S, pad, stride, "bf16", x, w, b, 1, y)
    assert err < TOL["bf16"] and err < TIGHT["bf16"], err
    # the automatic choice takes the tensor-core path too
    n0 = tdx.tdx_kernel_launch_count()
    st, y0, ok = run_conv(N, H, W, Cin, Cout, R, S, pad, stride, "bf16", x, w, b, 1)
    assert st == 0 and ok, tdx.tdx_last_error()
    st_cfg, c = tdx.tdx_default_conv2d_config(N, H, W, Cin, Cout, R, S, pad, stride, tdx.TDX_BF16)
    assert st_cfg == 0 and c.kernel == tdx.TDX_KERNEL_UMMA and c.halo == 1
    assert conv_error(N, H, W, Cin, Cout, R, S, pad, stride, "bf16", x, w, b, 1, y0) < TIGHT["bf16"]


def test_conv_strided_delta_filter_is_subsampled_shift():
    # exact: a delta filter at tap (r0, s0) with stride 2 copies every second pixel of the shifted input
    N, H, W, C = 2, 20, 24, 64
    x = si.small_integers(84, 0, (N, H, W, C), "bf16", -8, 8)
    wf = np.zeros((C, 3, 3, C), dtype=np.float32)
    for k in range(C):
        wf[k, 2, 0, k] = 1.0
    w = si.f32_to_bf16_bits(wf)
    st, y, ok = run_conv(N, H, W, C, C, 3, 3, 1, 2, "bf16", x, w, None, 0)
    assert st == 0 and ok, tdx.tdx_last_error()
    ref = oracle.conv2d(N, H, W, C, C, 3, 3, 1, 2, "bf16", x, w, None, 0)
    assert np.array_equal(oracle.decode(y, "bf16"), ref)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("stride", [1, 2])
def test_conv_generic_kernel(dtype, stride):
    N, H, W, Cin, Cout = 2, 11, 13, 5, 7
    xb, wb, b = si.conv_bf16(N, H, W, Cin, Cout, 3, 3, seed=74)
    if dtype == "f32":
        x, w = si.bf16_bits_to_f32(xb), si.bf16_bits_to_f32(wb)
    else:
        x, w = xb, wb
    st, y, ok = run_conv(N, H, W, Cin, Cout, 3, 3, 1, stride, dtype, x, w, b, 1)
    assert st == 0 and ok, tdx.tdx_last_error()
    assert conv_error(N, H, W, Cin, Cout, 3, 3, 1, stride, dtype, x, w, b, 1, y) < TOL[dtype]


def test_conv_infeasible_config_leaves_output_untouched():
    N, H, W, Cin, Cout = 1, 8, 8, 64, 64
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, 3, 3, seed=75)
    st, _, untouched = run_conv(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1, cfg=umma(patch_w=4, patch_h=4))
    assert st == tdx.TDX_ERR_CONFIG and untouched
    st, _, untouched = run_conv(N, H, W, Cin, Cout, 3, 3, 1, 2, "bf16", x, w, b, 1, cfg=umma(halo=2))   # halo reuse is stride 1 only
    assert st == tdx.TDX_ERR_CONFIG and untouched
    st, _, untouched = run_conv(N, H, W, Cin, Cout, 3, 3, 1, 9, "bf16", x, w, b, 1, cfg=umma())   # stride 9
    assert st == tdx.TDX_ERR_ALIGNMENT and untouched


def test_conv_host_buffer_entry_point():
    N, H, W, Cin, Cout = 1, 16, 16, 64, 64
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, 3, 3, seed=76)
    y = np.zeros((N * H * W, Cout), dtype=np.uint16)
    st = tdx.tdx_conv2d_bias_relu_host(N, H, W, Cin, Cout, 3, 3, 1, 1, tdx.TDX_BF16, x, w, b, 1, y)
    assert st == 0, tdx.tdx_last_error()
    assert conv_error(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1, y) < TIGHT["bf16"]


def test_conv_host_buffer_entry_point_in_chunks():
    # 5 images of 96 x 96 x 128: enough bytes for two groups of images (3 + 2) on the three-stream path
    N, H, W, Cin, Cout = 5, 96, 96, 128, 128
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, 3, 3, seed=77)
    y = np.zeros((N * H * W, Cout), dtype=np.uint16)
    st = tdx.tdx_conv2d_bias_relu_host(N, H, W, Cin, Cout, 3, 3, 1, 1, tdx.TDX_BF16, x, w, b, 1, y)
    assert st == 0, tdx.tdx_last_error()
    assert conv_error(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1, y) < TIGHT["bf16"]


# ------------------------------------------------------------------ full-size workloads

def test_full_size_conv_128x128x64():
    # N=4, H=W=128, Cin=Cout=64, 3x3, stride 1, pad 1, bias + ReLU, seed 2 -- full oracle
    N, H, W, Cin, Cout = 4, 128, 128, 64, 64
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, 3, 3, seed=2)
    st, y, ok = run_conv(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1)
    assert st == 0 and ok, tdx.tdx_last_error()
    err = conv_error(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1, y)
    assert err < TOL["bf16"] and err < TIGHT["bf16"], err
    assert (oracle.decode(y, "bf16") >= 0).all()
    assert tdx.tdx_check_device_status() == 0


def test_full_size_conv_56x56x256():
    # N=32, H=W=56, Cin=Cout=256, seed 3 -- every output element (5.9e10 multiply-adds for the oracle), in the
    # configuration the benchmark times (the automatic choice)
    N, H, W, Cin, Cout = 32, 56, 56, 256, 256
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, 3, 3, seed=3)
    st, y, ok = run_conv(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1)
    assert st == 0 and ok, tdx.tdx_last_error()
    M = N * H * W
    worst = 0.0
    for r0 in range(0, M, 12544):                  # four images at a time bounds the fp64 reference's memory
        rows = np.arange(r0, min(M, r0 + 12544), dtype=np.int64)
        worst = max(worst, conv_error(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1, y, rows=rows))
    assert worst < TOL["bf16"] and worst < TIGHT["bf16"], worst
    assert (oracle.decode(y[::53], "bf16") >= 0).all()
    assert tdx.tdx_check_device_status() == 0


RESIDUAL_CASES = [
    # N, H,  W,  Cin, Cout, R, S, pad, stride, cfg
    (2, 56, 56, 64, 64, 3, 3, 1, 1, None),                          # automatic: halo reuse over stacked images
    (3, 20, 36, 72, 40, 3, 3, 1, 1, dict(halo=2, tile_m=256)),      # ragged patches, channel tail
    (2, 28, 28, 128, 256, 1, 1, 0, 1, None),                        # 1 x 1: per-tap kernel
    (2, 30, 30, 64, 128, 3, 3, 1, 2, None),                         # strided
    (2, 16, 24, 64, 64, 3, 3, 1, 1, dict(store_mode=1)),            # direct-store epilogue
    (1, 9, 11, 5, 7, 3, 3, 1, 1, None),                             # generic kernel (Cin % 8 != 0)
]


@pytest.mark.parametrize("case", RESIDUAL_CASES)
@pytest.mark.parametrize("relu", [0, 1])
def test_conv_with_residual_term_vs_oracle(case, relu):
    N, H, W, Cin, Cout, R, S, pad, stride, cfgkw = case
    P, Q = oracle.conv_out_dim(H, R, pad, stride), oracle.conv_out_dim(W, S, pad, stride)
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, R, S, seed=85)
    res = si.normal(85, 3, (N * P * Q, Cout), "bf16", sigma=2.0)
    dx, dw, db, dres = to_dev(x), to_dev(w), to_dev(b), to_dev(res)
    out = GuardedOut(N * P * Q * Cout, "bf16")
    st = tdx.tdx_conv2d_bias_add_relu(N, H, W, Cin, Cout, R, S, pad, stride, tdx.TDX_BF16, dx, dw, db, dres, relu, out.ptr,
                                      cfg=None if cfgkw is None else umma(**cfgkw))
    torch.cuda.synchronize()
    assert st == 0 and out.guards_intact(), tdx.tdx_last_error()
    got = oracle.decode(out.payload().reshape(N * P * Q, Cout), "bf16")
    ref = oracle.conv2d(N, H, W, Cin, Cout, R, S, pad, stride, "bf16", x, w, b, relu, residual=res)
    sc = oracle.conv_row_scales(N, H, W, Cin, Cout, R, S, pad, stride, "bf16", x, w, b, residual=res)
    err = oracle.max_normalised_error(got, ref, sc)
    assert err < TIGHT["bf16"], err
    if relu:
        assert (got >= 0).all()
    # the residual really entered: the result differs from the plain convolution
    st, y_plain, _ = run_conv(N, H, W, Cin, Cout, R, S, pad, stride, "bf16", x, w, b, relu)
    assert st == 0 and not np.array_equal(oracle.decode(y_plain, "bf16"), got)


@pytest.mark.parametrize("tile_m", [128, 256])
def test_conv_halo_with_tile_widths_fitted_to_the_cta_count(tile_m):
    # fit = 2 on the halo kernel: some row blocks are cut into two 128-column tiles; filter slices arrive in 64-row copies
    N, H, W, Cin, Cout = 8, 56, 56, 64, 256
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, 3, 3, seed=86)
    st, y, ok = run_conv(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1, cfg=umma(halo=3, tile_m=tile_m, tile_n=256, fit=2))
    assert st == 0 and ok, tdx.tdx_last_error()
    rows = structured_rows(N * H * W, max_blocks=24)
    err = conv_error(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1, y, rows=rows)
    assert err < TIGHT["bf16"], err
    st, y1, ok = run_conv(N, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1, cfg=umma(halo=3, tile_m=tile_m, tile_n=256, fit=1))
    assert st == 0 and ok, tdx.tdx_last_error()
    assert np.array_equal(y, y1)          # the reduction order inside an output does not depend on the tile width


@pytest.mark.parametrize("case", [(8, 56, 56, 64, 512, 3, 3, 1, 2), (4, 28, 28, 128, 384, 1, 1, 0, 1), (6, 30, 26, 64, 256, 3, 3, 1, 2)])
@pytest.mark.parametrize("tile_m", [128, 256])
def test_conv_per_tap_with_tile_widths_fitted_to_the_cta_count(case, tile_m):
    # fit = 2 on the per-tap kernel (strided layers, 1 x 1 filters): some row blocks are cut into narrower tiles so that
    # all CTAs finish together; filter slices arrive in 64-row copies.  Same bits as the uniform grid.
    N, H, W, Cin, Cout, R, S, pad, stride = case
    x, w, b = si.conv_bf16(N, H, W, Cin, Cout, R, S, seed=87)
    st, y, ok = run_conv(N, H, W, Cin, Cout, R, S, pad, stride, "bf16", x, w, b, 1, cfg=umma(halo=1, tile_m=tile_m, tile_n=256, fit=2))
    assert st == 0 and ok, tdx.tdx_last_error()
    P, Q = oracle.conv_out_dim(H, R, pad, stride), oracle.conv_out_dim(W, S, pad, stride)
    rows = structured_rows(N * P * Q, max_blocks=24)
    err = conv_error(N, H, W, Cin, Cout, R, S, pad, stride, "bf16", x, w, b, 1, y, rows=rows)
    assert err < TIGHT["bf16"], err
    st, y1, ok = run_conv(N, H, W, Cin, Cout, R, S, pad, stride, "bf16", x, w, b, 1, cfg=umma(halo=1, tile_m=tile_m, tile_n=256, fit=1))
    assert st == 0 and ok, tdx.tdx_last_error()
    assert np.array_equal(y, y1)
    assert tdx.tdx_check_device_status() == 0
