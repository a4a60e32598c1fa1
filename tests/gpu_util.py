"""Helpers shared by the GPU parity tests: device buffers via torch (memory and streams only),
canary guard bands around outputs, and comparison with the CPU oracle."""
import numpy as np
import torch

import oracle
import paper_2409_03864_b200 as tdx

DT = {"f32": tdx.TDX_F32, "bf16": tdx.TDX_BF16}
# tolerances of the normalised error metric (oracle.metric): fp32 CUDA-core paths, bf16 tensor-core paths
TOL = {"f32": 1e-5, "bf16": 2e-2}
# tighter internal bounds: bf16 output rounding alone is 2^-9 of |C| <= scale; fp32 FMA chains ~ sqrt(K) 2^-24
TIGHT = {"f32": 2e-6, "bf16": 4.5e-3}

GUARD = 1024          # canary elements before and after every output
CANARY_F32 = np.float32(-12345.678)
CANARY_BF16 = np.uint16(0xC2F7)


def to_dev(arr: np.ndarray) -> torch.Tensor:
    """numpy (float32, or uint16 bf16 bit patterns) -> device tensor with the same bytes."""
    a = np.ascontiguousarray(arr)
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda()
    return torch.from_numpy(a).cuda()


class GuardedOut:
    """Device output buffer with canary guard bands; `.ptr` is the address of the payload."""

    def __init__(self, n_elems: int, dtype: str):
        self.dtype, self.n = dtype, int(n_elems)
        if dtype == "f32":
            self.buf = torch.full((self.n + 2 * GUARD,), float(CANARY_F32), dtype=torch.float32, device="cuda")
        else:
            self.buf = torch.full((self.n + 2 * GUARD,), int(CANARY_BF16.view(np.int16)), dtype=torch.int16,
                                  device="cuda")
        self.ptr = self.buf.data_ptr() + GUARD * self.buf.element_size()

    def host(self) -> np.ndarray:
        h = self.buf.cpu().numpy()
        return h.view(np.uint16) if self.dtype == "bf16" else h

    def payload(self) -> np.ndarray:
        return self.host()[GUARD:GUARD + self.n]

    def guards_intact(self) -> bool:
        h = self.host()
        c = CANARY_BF16 if self.dtype == "bf16" else CANARY_F32
        return bool((h[:GUARD] == c).all() and (h[GUARD + self.n:] == c).all())

    def untouched(self) -> bool:
        c = CANARY_BF16 if self.dtype == "bf16" else CANARY_F32
        return bool((self.host() == c).all())


def run_gemm(M, N, K, transA, transB, alpha, dtype, A, B, cfg=None, workspace=None):
    """Runs tdx_gemm(_ex) on device copies of A and B; returns (status, payload array, guards ok)."""
    dA, dB = to_dev(A), to_dev(B)
    out = GuardedOut(M * N, dtype)
    ws_ptr, ws_bytes = None, 0
    if workspace is not None:
        ws_ptr, ws_bytes = workspace.data_ptr(), workspace.numel() * workspace.element_size()
    if cfg is None and workspace is None:
        st = tdx.tdx_gemm(M, N, K, transA, transB, alpha, DT[dtype], dA, dB, out.ptr)
    else:
        st = tdx.tdx_gemm_ex(M, N, K, transA, transB, alpha, DT[dtype], dA, dB, out.ptr, None, cfg, ws_ptr, ws_bytes)
    torch.cuda.synchronize()
    return st, out.payload().reshape(M, N), out.guards_intact() if st == 0 else out.untouched()


def gemm_error(M, N, K, transA, transB, alpha, dtype, A, B, got, rows=None):
    ref = oracle.gemm(M, N, K, transA, transB, alpha, dtype, A, B, rows=rows)
    sc = oracle.gemm_row_scales(M, N, K, transA, transB, alpha, dtype, A, B, rows=rows)
    vals = oracle.decode(got, dtype).reshape(M, N)
    if rows is not None:
        vals = vals[np.asarray(rows)]
    return oracle.max_normalised_error(vals, ref, sc)


def run_conv(N, H, W, Cin, Cout, R, S, pad, stride, dtype, x, w, bias, relu, cfg=None):
    P, Q = oracle.conv_out_dim(H, R, pad, stride), oracle.conv_out_dim(W, S, pad, stride)
    dx, dw = to_dev(x), to_dev(w)
    db = None if bias is None else to_dev(bias)
    out = GuardedOut(N * P * Q * Cout, dtype)
    if cfg is None:
        st = tdx.tdx_conv2d_bias_relu(N, H, W, Cin, Cout, R, S, pad, stride, DT[dtype], dx, dw, db, relu, out.ptr)
    else:
        st = tdx.tdx_conv2d_bias_relu_ex(N, H, W, Cin, Cout, R, S, pad, stride, DT[dtype], dx, dw, db, relu, out.ptr,
                                         None, cfg)
    torch.cuda.synchronize()
    return st, out.payload().reshape(N * P * Q, Cout), out.guards_intact() if st == 0 else out.untouched()


def conv_error(N, H, W, Cin, Cout, R, S, pad, stride, dtype, x, w, bias, relu, got, rows=None):
    ref = oracle.conv2d(N, H, W, Cin, Cout, R, S, pad, stride, dtype, x, w, bias, relu, rows=rows)
    sc = oracle.conv_row_scales(N, H, W, Cin, Cout, R, S, pad, stride, dtype, x, w, bias, rows=rows)
    vals = oracle.decode(got, dtype).reshape(-1, Cout)
    if rows is not None:
        vals = vals[np.asarray(rows)]
    return oracle.max_normalised_error(vals, ref, sc)


def structured_rows(M, per_block=(0, 1, 63, 64, 126, 127), block=128, extra=2, seed=0, max_blocks=None):
    """Rows {0,1,63,64,126,127} (+ `extra` seeded ones) of 128-row blocks; all blocks, or an even subset."""
    nblk = -(-M // block)
    blocks = np.arange(nblk)
    if max_blocks is not None and nblk > max_blocks:
        blocks = np.unique(np.linspace(0, nblk - 1, max_blocks).astype(np.int64))
    rng = np.random.default_rng(seed)
    rows = []
    for b in blocks:
        cand = [b * block + r for r in per_block] + list(b * block + rng.integers(0, block, size=extra))
        rows.extend(int(r) for r in cand if r < M)
    return np.array(sorted(set(rows)), dtype=np.int64)
