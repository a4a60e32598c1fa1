"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, validates arguments before touching a device, and lists a search space that
obeys the static constraints."""
import ctypes
import os
import re

import pytest

import paper_2409_03864_b200 as tdx
from paper_2409_03864_b200 import build as tdx_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    tdx_build.build()


@pytest.fixture(autouse=True)
def heuristics_only():
    """These tests look at the heuristic defaults: run them without the shipped tuning cache, restore it after."""
    tdx.tdx_tune_clear()
    yield
    tdx.tdx_tune_clear()
    shipped = os.path.join(ROOT, "paper_2409_03864_b200", "tuned_b200.json")
    if os.path.exists(shipped):
        tdx.tdx_tune_load(shipped)


def test_shipped_tuning_cache_loads_and_is_feasible():
    shipped = os.path.join(ROOT, "paper_2409_03864_b200", "tuned_b200.json")
    assert os.path.exists(shipped)
    assert tdx.tdx_tune_load(shipped) == tdx.TDX_OK
    st, c = tdx.tdx_default_gemm_config(4096, 4096, 4096, 0, 1, tdx.TDX_BF16)
    assert st == tdx.TDX_OK and c.kernel == tdx.TDX_KERNEL_UMMA and c.tile_m in (128, 256)
    st, c = tdx.tdx_default_conv2d_config(32, 56, 56, 256, 256, 3, 3, 1, 1, tdx.TDX_BF16)
    assert st == tdx.TDX_OK and c.patch_w * c.patch_h >= 8


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "tdx.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tdx_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_symbols()
    assert len(names) >= 18
    L = ctypes.CDLL(str(tdx_build.LIB))
    for n in names:
        assert hasattr(L, n), f"{n} declared in tdx.h but not exported"
    assert set(names) == set(tdx.binding.EXPORTS)
    assert tdx.tdx_version().startswith("tdx ")


def test_gemm_argument_validation_is_silenceable_and_precedes_cuda():
    bad = [
        dict(M=-1), dict(N=-3), dict(K=-1), dict(transA=2), dict(transB=-1), dict(dtype=7),
        dict(A=None), dict(B=None), dict(C=None),
    ]
    base = dict(M=8, N=8, K=8, transA=0, transB=0, alpha=1.0, dtype=tdx.TDX_BF16, A=256, B=512, C=1024)
    for b in bad:
        a = dict(base, **b)
        st = tdx.tdx_gemm(**a)
        assert st == tdx.TDX_ERR_INVALID_ARG, (b, st)
        assert tdx.tdx_last_error()
    # misaligned element pointer
    assert tdx.tdx_gemm(**dict(base, A=257)) == tdx.TDX_ERR_ALIGNMENT
    # empty problems are a no-op even without a device
    assert tdx.tdx_gemm(**dict(base, M=0, A=None, B=None, C=None)) == tdx.TDX_OK
    assert tdx.tdx_gemm(**dict(base, N=0)) == tdx.TDX_OK


def test_batched_gemm_argument_validation():
    base = dict(batch=2, M=8, N=8, K=8, transA=0, transB=0, alpha=1.0, beta=1.0, dtype=tdx.TDX_F32, A=256, B=512, C=1024)
    for b in [dict(batch=-1), dict(M=-1), dict(K=-2), dict(transB=3), dict(dtype=9), dict(A=None), dict(C=None),
              dict(strideA=-8), dict(strideC=63), dict(alpha=float("nan")), dict(beta=float("nan"))]:
        st = tdx.tdx_gemm_batched(**dict(base, **b))
        assert st == tdx.TDX_ERR_INVALID_ARG, (b, st)
    assert tdx.tdx_gemm_batched(**dict(base, C=1026)) == tdx.TDX_ERR_ALIGNMENT
    assert tdx.tdx_gemm_batched(**dict(base, batch=0)) == tdx.TDX_OK
    assert tdx.tdx_gemm_batched(**dict(base, N=0)) == tdx.TDX_OK


def test_conv_argument_validation():
    base = dict(N=1, H=8, W=8, Cin=8, Cout=8, R=3, S=3, pad=1, stride=1, dtype=tdx.TDX_BF16, x=256, w=512, bias=None,
                relu=1, y=1024)
    for b in [dict(N=-1), dict(Cin=0), dict(R=0), dict(S=-1), dict(pad=-1), dict(stride=0), dict(dtype=5),
              dict(relu=2), dict(x=None), dict(w=None), dict(y=None)]:
        st = tdx.tdx_conv2d_bias_relu(**dict(base, **b))
        assert st == tdx.TDX_ERR_INVALID_ARG, (b, st)
    # filter larger than the padded image: empty output, no-op
    assert tdx.tdx_conv2d_bias_relu(**dict(base, H=1, W=1, pad=0)) == tdx.TDX_OK
    assert tdx.tdx_conv2d_bias_relu(**dict(base, Cout=0)) == tdx.TDX_OK


def test_infeasible_explicit_config_is_reported_before_any_device_work():
    base = dict(M=256, N=256, K=256, transA=0, transB=1, alpha=1.0, dtype=tdx.TDX_BF16, A=256, B=512, C=1024)
    for kw in [dict(tile_n=48), dict(tile_n=512), dict(stages=9), dict(tile_m=64), dict(tile_m=384), dict(tile_m=256, tile_n=256, stages=4),
               dict(split_k=7),
               dict(tile_k=32), dict(cta_pair=3), dict(store_mode=3),
               dict(store_mode=2, split_k=2), dict(store_mode=2, tile_m=256, tile_n=256, stages=4), dict(kernel=9), dict(kernel=tdx.TDX_KERNEL_SIMT)]:
        cfg = tdx.tdx_config(kernel=kw.pop("kernel", tdx.TDX_KERNEL_UMMA), **kw)
        assert tdx.tdx_gemm_ex(**base, cfg=cfg) == tdx.TDX_ERR_CONFIG, kw
    # N-major B (transB=0) needs tile_n % 64 == 0
    cfg = tdx.tdx_config(kernel=tdx.TDX_KERNEL_UMMA, tile_n=32)
    assert tdx.tdx_gemm_ex(**dict(base, transB=0), cfg=cfg) == tdx.TDX_ERR_CONFIG
    # forcing the tensor-core kernel on a pitch that is not a multiple of 16 bytes
    cfg = tdx.tdx_config(kernel=tdx.TDX_KERNEL_UMMA)
    assert tdx.tdx_gemm_ex(**dict(base, K=100), cfg=cfg) == tdx.TDX_ERR_ALIGNMENT
    # conv: split-K and bad patches
    cbase = dict(N=1, H=16, W=16, Cin=64, Cout=64, R=3, S=3, pad=1, stride=1, dtype=tdx.TDX_BF16, x=256, w=512,
                 bias=None, relu=1, y=1024)
    for kw in [dict(split_k=2), dict(patch_w=4, patch_h=4), dict(patch_w=24, patch_h=2), dict(patch_w=64, patch_h=4)]:
        cfg = tdx.tdx_config(kernel=tdx.TDX_KERNEL_UMMA, **kw)
        assert tdx.tdx_conv2d_bias_relu_ex(**cbase, cfg=cfg) == tdx.TDX_ERR_CONFIG, kw


def test_workspace_size():
    st, b = tdx.tdx_gemm_workspace_size(128, 8192, 8192, tdx.TDX_BF16, tdx.tdx_config(split_k=4))
    assert st == tdx.TDX_OK and b == 4 * 128 * 8192 * 4
    st, b = tdx.tdx_gemm_workspace_size(128, 8192, 8192, tdx.TDX_BF16, tdx.tdx_config(split_k=1))
    assert st == tdx.TDX_OK and b == 0
    assert tdx.tdx_gemm_workspace_size(-1, 1, 1, tdx.TDX_BF16, None)[0] == tdx.TDX_ERR_INVALID_ARG


SMEM_LIMIT = 232448


@pytest.mark.parametrize("shape", [(1024, 1024, 1024), (8192, 8192, 8192), (128, 8192, 8192), (8192, 128, 8192),
                                   (4096, 4096, 512)])
def test_gemm_search_space_obeys_constraints(shape):
    M, N, K = shape
    st, cfgs = tdx.tdx_enum_gemm_configs(M, N, K, 0, 0, tdx.TDX_BF16)
    assert st == tdx.TDX_OK and len(cfgs) >= 4
    num_kb = -(-K // 64)
    seen = set()
    for c in cfgs:
        key = tuple(c.values())
        assert key not in seen
        seen.add(key)
        assert c["kernel"] == tdx.TDX_KERNEL_UMMA and c["tile_m"] in (128, 256) and c["tile_k"] == 64
        assert c["tile_n"] % 64 == 0                          # B is read N-major here
        assert 2 <= c["stages"] <= 8
        assert c["store_mode"] in (1, 2, 3)
        staging = {1: 0, 2: 16 * 2048, 3: (c["tile_m"] // 128) * 8 * 2048}[c["store_mode"]]
        rows_per_cta = 128 + c["tile_n"] // 2 if c["cta_pair"] == 2 else c["tile_m"] + c["tile_n"]
        assert c["stages"] * rows_per_cta * 128 + 1024 + 512 + staging <= SMEM_LIMIT
        if c["cta_pair"] == 2:
            assert c["tile_m"] == 256 and c["split_k"] == 1 and c["tile_n"] % 128 == 0
        if c["store_mode"] == 2:
            assert c["split_k"] == 1
        if c["store_mode"] == 3:
            # split-K summed inside a cluster: cluster size = split_k, slices of whole 32-column steps, and the receive
            # slots for the other ranks' slices fit the pipeline stages
            assert 2 <= c["split_k"] <= 8 and c["cta_pair"] == 1 and c["fit"] == 1
            assert c["tile_n"] % (32 * c["split_k"]) == 0
            assert (c["split_k"] - 1) * c["tile_m"] * (c["tile_n"] // c["split_k"]) * 4 <= c["stages"] * rows_per_cta * 128
        halves = 1 if c["cta_pair"] == 2 else c["tile_m"] // 128
        assert halves * c["tile_n"] <= 512                     # one tile's accumulators fit in a CTA's TMEM
        per = -(-num_kb // c["split_k"])
        assert (c["split_k"] - 1) * per < num_kb               # no empty K slice
    if M * N <= 128 * 8192:
        assert any(c["split_k"] > 1 for c in cfgs)             # skinny shapes get split-K candidates
        assert any(c["store_mode"] == 3 for c in cfgs)         # ... with the sum in a workspace and inside clusters
    if shape == (8192, 8192, 8192):
        assert all(c["split_k"] == 1 for c in cfgs)


def test_search_space_for_other_kernels():
    st, cfgs = tdx.tdx_enum_gemm_configs(256, 256, 256, 0, 0, tdx.TDX_F32)
    assert st == tdx.TDX_OK and [c["kernel"] for c in cfgs] == [tdx.TDX_KERNEL_SIMT]
    st, cfgs = tdx.tdx_enum_gemm_configs(196, 256, 2305, 0, 0, tdx.TDX_BF16)   # K pitch not 16-byte aligned
    assert st == tdx.TDX_OK and [c["kernel"] for c in cfgs] == [tdx.TDX_KERNEL_GENERIC]
    st, cfgs = tdx.tdx_enum_conv2d_configs(32, 56, 56, 256, 256, 3, 3, 1, 1, tdx.TDX_BF16)
    assert st == tdx.TDX_OK and cfgs
    for c in cfgs:
        a = c["patch_w"] * c["patch_h"]
        assert c["patch_w"] >= 8 and a <= 128 and a & (a - 1) == 0 and c["split_k"] == 1
    st, cfgs = tdx.tdx_enum_conv2d_configs(8, 56, 56, 64, 128, 3, 3, 1, 2, tdx.TDX_BF16)  # stride 2: per-tap loads only
    assert st == tdx.TDX_OK and cfgs and all(c["kernel"] == tdx.TDX_KERNEL_UMMA and c["halo"] == 1 for c in cfgs)
    assert all(c["patch_w"] * 2 <= 256 and c["patch_h"] * 2 <= 256 for c in cfgs)
    st, cfgs = tdx.tdx_enum_conv2d_configs(1, 8, 8, 8, 8, 3, 3, 1, 9, tdx.TDX_BF16)   # stride 9: beyond the copy's reach
    assert [c["kernel"] for c in cfgs] == [tdx.TDX_KERNEL_GENERIC]
    st, cfgs = tdx.tdx_enum_conv2d_configs(1, 8, 8, 7, 8, 3, 3, 1, 1, tdx.TDX_BF16)   # Cin pitch not 16-byte aligned
    assert [c["kernel"] for c in cfgs] == [tdx.TDX_KERNEL_GENERIC]


def test_default_configs():
    st, c = tdx.tdx_default_gemm_config(4096, 4096, 4096, 0, 1, tdx.TDX_BF16)
    assert st == tdx.TDX_OK and c.kernel == tdx.TDX_KERNEL_UMMA and c.tile_n == 256 and c.split_k == 1
    assert c.tile_m == 256 and c.stages == 3                 # 3 x 64 KiB stages fit in shared memory
    st, c = tdx.tdx_default_gemm_config(128, 8192, 8192, 0, 0, tdx.TDX_BF16)
    assert st == tdx.TDX_OK and c.split_k > 1
    st, c = tdx.tdx_default_gemm_config(256, 256, 256, 0, 0, tdx.TDX_F32)
    assert st == tdx.TDX_OK and c.kernel == tdx.TDX_KERNEL_SIMT
    st, c = tdx.tdx_default_conv2d_config(32, 56, 56, 256, 256, 3, 3, 1, 1, tdx.TDX_BF16)
    # halo reuse; 56 rows are 3.5 patches, so the patches are cut from the stacked column of images (32 * 57 = 114 * 16)
    assert st == tdx.TDX_OK and (c.patch_w, c.patch_h, c.halo) == (8, 16, 3) and c.tile_n == 256
    st, c = tdx.tdx_default_conv2d_config(4, 128, 128, 64, 64, 3, 3, 1, 1, tdx.TDX_BF16)
    assert st == tdx.TDX_OK and (c.patch_w, c.patch_h, c.halo) == (8, 16, 2) and c.tile_n == 64
    st, c = tdx.tdx_default_conv2d_config(4, 128, 128, 64, 64, 1, 1, 0, 1, tdx.TDX_BF16)          # 1 x 1: nothing to reuse
    assert st == tdx.TDX_OK and c.halo == 1 and c.patch_w * c.patch_h in (32, 64, 128)
    st, c = tdx.tdx_default_conv2d_config(4, 64, 64, 64, 256, 9, 9, 4, 1, tdx.TDX_BF16)           # halo tile too large
    assert st == tdx.TDX_OK and c.halo in (1, 2, 3) and c.stages >= 2


@pytest.mark.parametrize("shape", [(4096, 4096, 4096), (4096, 4096, 512), (2048, 3072, 1024), (1000, 2000, 512),
                                   (5000, 3000, 256), (256, 640, 64), (8192, 8192, 8192)])
@pytest.mark.parametrize("tile", [(256, 256), (128, 256), (256, 192)])
def test_fitted_tile_plan_covers_the_output_once_and_balances_the_ctas(shape, tile):
    # host logic of fit = 2: every row block's columns are covered exactly once by tiles whose widths are multiples
    # of 64 and at most tile_n; each CTA's list is dense; the model's longest CTA is never worse than the uniform grid
    M, N, K = shape
    tm, tn = tile
    ctas = 148
    st, rounds, used, tiles, fit, uni = tdx.tdx_gemm_tile_plan(M, N, K, tm, tn, 2, ctas)
    assert st == tdx.TDX_OK
    assert fit <= uni * (1 + 1e-12)
    if rounds == 0:
        assert fit == uni                       # uniform grid kept
        return
    assert 1 <= used <= ctas
    cover = {}
    for cta in range(used):
        ended = False
        for r in range(rounds):
            m, n0, w = tiles[r][cta]
            if w == 0:
                ended = True
                continue
            assert not ended, "a CTA's tile list must not have holes"
            assert w % 64 == 0 and 128 <= w <= tn and n0 % 64 == 0 and 0 <= m < -(-M // tm)
            cover.setdefault(m, []).append((n0, w))
    assert sorted(cover) == list(range(-(-M // tm)))
    for m, segs in cover.items():
        segs.sort()
        pos = 0
        for n0, w in segs:
            assert n0 == pos, (m, segs)
            pos += w
        assert N <= pos < N + tn
    per_cta = [sum(tiles[r][c][2] for r in range(rounds)) for c in range(used)]
    assert max(per_cta) - min(per_cta) <= tn     # column-weighted load differs by at most one wide tile
    if shape == (4096, 4096, 4096) and tile == (256, 256):
        # 256 uniform tiles on 148 CTAs take two tile times; 148 wide + 144 tiles of 192 columns take 1.75
        widths = sorted(t[2] for row in tiles for t in row if t[2])
        assert widths.count(256) == 148 and widths.count(192) == 144 and fit < 0.92 * uni


def test_tuning_cache_round_trip(tmp_path):
    path = tmp_path / "cache.json"
    path.write_text('{"version": 1, "entries": [\n  {"key": "gemm:640:640:640:0:1:1", '
                    '"cfg": [1, 128, 64, 64, 3, 1, 2, 1, 2, 0, 0], "us": 12.500}\n]}\n')
    assert tdx.tdx_tune_clear() == tdx.TDX_OK
    assert tdx.tdx_tune_load(str(path)) == tdx.TDX_OK
    st, c = tdx.tdx_default_gemm_config(640, 640, 640, 0, 1, tdx.TDX_BF16)
    assert st == tdx.TDX_OK and (c.tile_n, c.stages, c.split_k, c.raster) == (64, 3, 2, 2)
    out = tmp_path / "out.json"
    assert tdx.tdx_tune_save(str(out)) == tdx.TDX_OK
    assert "gemm:640:640:640:0:1:1" in out.read_text() and "[1, 128, 64, 64, 3, 1, 2, 1, 2, 0, 0, 0, 0, 0]" in out.read_text()
    assert tdx.tdx_tune_clear() == tdx.TDX_OK
    st, c = tdx.tdx_default_gemm_config(640, 640, 640, 0, 1, tdx.TDX_BF16)
    assert c.tile_n != 64 or c.split_k != 2
    assert tdx.tdx_tune_load(str(tmp_path / "missing.json")) == tdx.TDX_ERR_INVALID_ARG
    bad = tmp_path / "bad.json"
    bad.write_text('{"entries": [{"key": "gemm:1:1:1:0:0:1", "cfg": [1, 2, 3]}]}')
    assert tdx.tdx_tune_load(str(bad)) == tdx.TDX_ERR_INVALID_ARG


@pytest.mark.parametrize("shape", [(128, 8192, 8192, 128, 192), (8192, 128, 8192, 128, 128), (128, 8192, 8192, 128, 256),
                                   (300, 1000, 4100, 128, 128), (128, 128, 64 * 9, 128, 128), (512, 512, 64 * 3, 256, 256)])
@pytest.mark.parametrize("ctas", [148, 132, 7])
def test_k_balanced_plan_covers_every_unit_once_and_evenly(shape, ctas):
    # host only: the tiles x K blocks units are dealt to the CTAs in nearly equal runs; every unit exactly once;
    # a tile's pieces carry slots in ascending K order; no piece shorter than the snapping length unless it is a whole tile
    M, N, K, tm, tn = shape
    st, rounds, used, ent, slots = tdx.tdx_gemm_k_balanced_plan(M, N, K, tm, tn, ctas)
    assert st == tdx.TDX_OK, tdx.tdx_last_error()
    num_kb = -(-K // 64)
    tiles_m, tiles_n = -(-M // tm), -(-N // tn)
    units = tiles_m * tiles_n * num_kb
    assert 1 <= used <= min(ctas, max(1, units // 4)) and rounds >= 1
    seen = {}
    loads = []
    for c in range(used):
        load = 0
        for r in range(rounds):
            m, n0, w, kb0, kb1, slot = ent[r][c]
            if w == 0:
                continue
            assert 0 <= m < tiles_m and n0 % tn == 0 and n0 < N and w % 64 == 0 and 0 < w <= tn and n0 + w >= min(N, n0 + tn)
            assert 0 <= kb0 < kb1 <= num_kb
            assert (kb1 - kb0 >= 4) or (kb0 == 0 and kb1 == num_kb) or num_kb < 8, (kb0, kb1)
            seen.setdefault((m, n0), []).append((slot, kb0, kb1))
            load += kb1 - kb0
        loads.append(load)
    assert len(seen) == tiles_m * tiles_n
    for pieces in seen.values():
        pieces.sort()
        assert [s for s, _, _ in pieces] == list(range(len(pieces)))          # slots 0, 1, 2, ...
        assert pieces[0][1] == 0 and pieces[-1][2] == num_kb
        assert all(a[2] == b[1] for a, b in zip(pieces, pieces[1:]))          # contiguous, ascending K
        assert len(pieces) <= slots
    assert sum(loads) == units
    share = units / used
    assert max(loads) <= share + 5 and min(loads) >= share - 5                # even up to the snapping length


def test_cluster_reduction_config_constraints_and_workspace_size():
    # store_mode 3 (split-K summed inside a cluster of split_k CTAs): no workspace; constraints checked before any launch
    M, N, K = 128, 8192, 8192
    ok = tdx.tdx_config(kernel=tdx.TDX_KERNEL_UMMA, tile_m=128, tile_n=192, split_k=3, store_mode=3)
    st, need = tdx.tdx_gemm_workspace_size(M, N, K, tdx.TDX_BF16, ok)
    assert st == 0 and need == 0
    base = dict(M=M, N=N, K=K, transA=0, transB=0, alpha=1.0, dtype=tdx.TDX_BF16, A=256, B=512, C=1024)
    for kw in [dict(tile_m=128, tile_n=192, split_k=1),              # nothing to sum
               dict(tile_m=128, tile_n=192, split_k=4),              # 192 columns do not cut into four slices of 32-column steps
               dict(tile_m=128, tile_n=128, split_k=16),             # larger than a cluster
               dict(tile_m=128, tile_n=256, split_k=2, fit=2),       # uniform grid only
               dict(tile_m=256, tile_n=256, split_k=2, cta_pair=2)]:
        cfg = tdx.tdx_config(kernel=tdx.TDX_KERNEL_UMMA, store_mode=3, **kw)
        assert tdx.tdx_gemm_ex(**base, cfg=cfg) == tdx.TDX_ERR_CONFIG, kw
    # the convolution has no split-K, hence no cluster reduction
    cfg = tdx.tdx_config(kernel=tdx.TDX_KERNEL_UMMA, store_mode=3, split_k=2, tile_m=128, tile_n=64)
    assert tdx.tdx_conv2d_bias_relu_ex(1, 16, 16, 64, 64, 3, 3, 1, 1, tdx.TDX_BF16, 256, 512, 1024, 1, 2048, None, cfg) == tdx.TDX_ERR_CONFIG


def test_k_balanced_config_constraints_and_workspace_size():
    M, N, K = 128, 8192, 8192
    ok = tdx.tdx_config(kernel=tdx.TDX_KERNEL_UMMA, tile_m=128, tile_n=192, fit=3, split_k=1, store_mode=1)
    st, need = tdx.tdx_gemm_workspace_size(M, N, K, tdx.TDX_BF16, ok)
    _, _, _, _, slots = tdx.tdx_gemm_k_balanced_plan(M, N, K, 128, 192, 148)
    assert st == 0 and need == slots * M * N * 4 and 2 <= slots <= 6
    base = dict(M=M, N=N, K=K, transA=0, transB=0, alpha=1.0, dtype=tdx.TDX_BF16, A=256, B=512, C=1024)
    for kw in [dict(split_k=2), dict(store_mode=2), dict(tile_n=96), dict(cta_pair=2, tile_m=256, tile_n=256)]:
        cfg = tdx.tdx_config(kernel=tdx.TDX_KERNEL_UMMA, fit=3, **kw)
        assert tdx.tdx_gemm_ex(**base, cfg=cfg) == tdx.TDX_ERR_CONFIG, kw
    st, cfgs = tdx.tdx_enum_gemm_configs(M, N, K, 0, 0, tdx.TDX_BF16)
    assert st == 0 and any(c["fit"] == 3 for c in cfgs)
    st, cfgs = tdx.tdx_enum_gemm_configs(8192, 8192, 8192, 0, 0, tdx.TDX_BF16)
    assert st == 0 and not any(c["fit"] == 3 for c in cfgs)                   # many tiles: nothing to balance


def test_force_config_environment_variable():
    # read once per process, so each case runs in a child process; host only (the default-config query shows nothing of
    # it -- the override applies to calls -- so an infeasible forced configuration is the observable: CONFIG before any
    # device work, with the variable's fields in the message)
    import subprocess
    import sys
    code = ("import paper_2409_03864_b200 as tdx; "
            "st = tdx.tdx_gemm(512, 512, 512, 0, 1, 1.0, tdx.TDX_BF16, 256, 512, 1024); "
            "print(st, tdx.tdx_last_error())")
    env = dict(os.environ, TDX_FORCE_CONFIG="tile_m=128,tile_n=48")
    r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, cwd=ROOT, timeout=120)
    assert r.returncode == 0 and r.stdout.split()[0] == str(tdx.TDX_ERR_CONFIG) and "tile_n" in r.stdout, r.stdout + r.stderr
    env = dict(os.environ, TDX_FORCE_CONFIG="tile_q=3")
    r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, cwd=ROOT, timeout=120)
    assert "ignored" in r.stderr and r.stdout.split()[0] != str(tdx.TDX_ERR_CONFIG)      # void: the call proceeds (and finds no device here)
