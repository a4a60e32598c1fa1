"""The library's launches can be captured into a CUDA graph (after one eager call per shape has filled the
descriptor, plan and workspace caches) and replayed: the replays must reproduce the eager results bit for bit,
and those must agree with the CPU oracle."""
import numpy as np
import pytest
import torch

import paper_2409_03864_b200 as tdx
import seeded_inputs as si
from gpu_util import TIGHT, conv_error, gemm_error, to_dev

pytestmark = pytest.mark.gpu


def umma(**kw):
    return tdx.tdx_config(kernel=tdx.TDX_KERNEL_UMMA, **kw)


def test_graph_replay_reproduces_eager_results():
    stream = torch.cuda.Stream()
    raw = stream.cuda_stream

    # (a) fp32 CUDA-core GEMM
    Ma, Na, Ka = 256, 256, 256
    Aa, Ba = si.gemm_f32_uniform(Ma, Na, Ka, seed=90)
    dAa, dBa = to_dev(Aa), to_dev(Ba)
    Ca = torch.zeros(Ma * Na, dtype=torch.float32, device="cuda")
    # (b) bf16 tensor-core GEMM, C = -(A . B^T), fitted tile table
    Mb, Nb, Kb = 1280, 4096, 256
    Ab, Bb = si.gemm_bf16_normal(Mb, Nb, Kb, seed=91, transB=1)
    dAb, dBb = to_dev(Ab), to_dev(Bb)
    Cb = torch.zeros(Mb * Nb, dtype=torch.int16, device="cuda")
    # (c) split-K GEMM (caller's workspace, GEMM kernel + reduction kernel)
    Mc, Nc, Kc = 128, 256, 2048
    Ac, Bc = si.gemm_bf16_normal(Mc, Nc, Kc, seed=92, transB=0)
    dAc, dBc = to_dev(Ac), to_dev(Bc)
    Cc = torch.zeros(Mc * Nc, dtype=torch.int16, device="cuda")
    ws = torch.zeros(4 * Mc * Nc, dtype=torch.float32, device="cuda")
    # (d) convolution + bias + ReLU (halo kernel)
    Nd, H, W, Cin, Cout = 2, 24, 24, 64, 64
    x, w, b = si.conv_bf16(Nd, H, W, Cin, Cout, 3, 3, seed=93)
    dx, dw, db = to_dev(x), to_dev(w), to_dev(b)
    y = torch.zeros(Nd * H * W * Cout, dtype=torch.int16, device="cuda")

    def launch_all():
        tdx.check(tdx.tdx_gemm(Ma, Na, Ka, 0, 0, 1.0, tdx.TDX_F32, dAa, dBa, Ca, raw))
        tdx.check(tdx.tdx_gemm_ex(Mb, Nb, Kb, 0, 1, -1.0, tdx.TDX_BF16, dAb, dBb, Cb, raw,
                                  umma(tile_m=256, tile_n=256, fit=2), None, 0))
        tdx.check(tdx.tdx_gemm_ex(Mc, Nc, Kc, 0, 0, 1.0, tdx.TDX_BF16, dAc, dBc, Cc, raw,
                                  umma(tile_m=128, tile_n=128, split_k=4, store_mode=1), ws, ws.numel() * 4))
        tdx.check(tdx.tdx_conv2d_bias_relu(Nd, H, W, Cin, Cout, 3, 3, 1, 1, tdx.TDX_BF16, dx, dw, db, 1, y, raw))

    outs = (Ca, Cb, Cc, y)
    with torch.cuda.stream(stream):
        launch_all()                      # eager: fills the caches, gives the expected bits
    stream.synchronize()
    eager = [o.clone() for o in outs]
    n0 = tdx.tdx_kernel_launch_count()

    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        launch_all()
    captured = tdx.tdx_kernel_launch_count() - n0
    assert captured >= 5                  # four calls, one of them two kernels
    for rep in range(3):
        for o in outs:
            o.zero_()
        with torch.cuda.stream(stream):
            g.replay()
        stream.synchronize()
        for o, e in zip(outs, eager):
            assert torch.equal(o, e), f"replay {rep} differs from the eager result"
    tdx.check(tdx.tdx_check_device_status(raw))

    assert gemm_error(Ma, Na, Ka, 0, 0, 1.0, "f32", Aa, Ba, Ca.cpu().numpy().reshape(Ma, Na)) < TIGHT["f32"]
    assert gemm_error(Mb, Nb, Kb, 0, 1, -1.0, "bf16", Ab, Bb, Cb.cpu().numpy().view(np.uint16).reshape(Mb, Nb)) < TIGHT["bf16"]
    assert gemm_error(Mc, Nc, Kc, 0, 0, 1.0, "bf16", Ac, Bc, Cc.cpu().numpy().view(np.uint16).reshape(Mc, Nc)) < TIGHT["bf16"]
    assert conv_error(Nd, H, W, Cin, Cout, 3, 3, 1, 1, "bf16", x, w, b, 1,
                      y.cpu().numpy().view(np.uint16).reshape(-1, Cout)) < TIGHT["bf16"]
