"""The model-guided tile-configuration search against the exhaustive one (GPU), and the cost model's ordering (host)."""
import pytest

import paper_2409_03864_b200 as tdx


def umma(**kw):
    return tdx.tdx_config(kernel=tdx.TDX_KERNEL_UMMA, **kw)


def test_cost_model_orders_known_cases():
    # host only: orderings that the measurements behind the model established
    def us(M, N, K, tB, **kw):
        st, v = tdx.tdx_model_gemm_us(M, N, K, 0, tB, tdx.TDX_BF16, umma(**kw))
        assert st == tdx.TDX_OK, tdx.tdx_last_error()
        return v
    big = (4096, 4096, 4096, 1)
    assert us(*big, tile_m=256, tile_n=256, fit=2) < us(*big, tile_m=256, tile_n=256, fit=1)     # the fitted plan fills the last wave
    assert us(*big, tile_m=256, tile_n=256, fit=1) < us(*big, tile_m=128, tile_n=256, fit=1)     # L2 ingest bounds 128-row tiles
    assert us(*big, tile_m=128, tile_n=256, fit=1) < us(*big, tile_m=128, tile_n=64)             # narrow MMAs run at half rate
    skinny = (128, 8192, 8192, 0)
    assert us(*skinny, tile_m=128, tile_n=128, split_k=2, store_mode=1) < us(*skinny, tile_m=128, tile_n=128, split_k=1)
    assert us(*skinny, tile_m=128, tile_n=128, split_k=2, store_mode=1) < us(*skinny, tile_m=128, tile_n=128, split_k=16, store_mode=1)
    # never below the time to stream the operands once
    assert us(*skinny, tile_m=128, tile_n=128, split_k=2, store_mode=1) >= (128 * 8192 + 8192 * 8192 + 128 * 8192) * 2 / 5.0e6
    st, _ = tdx.tdx_model_gemm_us(256, 256, 256, 0, 0, tdx.TDX_F32, umma())
    assert st == tdx.TDX_ERR_UNSUPPORTED


@pytest.mark.gpu
@pytest.mark.parametrize("shape", [(1024, 1024, 1024, 0), (2048, 2048, 1024, 1), (128, 4096, 4096, 0)])
def test_guided_search_finds_a_configuration_close_to_the_exhaustive_best(shape):
    M, N, K, tB = shape
    budget = 16
    st, best_all, us_all, tried_all = tdx.tdx_tune_gemm(M, N, K, 0, tB, tdx.TDX_BF16, iters=10, cap=8192)
    assert st == 0, tdx.tdx_last_error()
    st, best, us, tried, n_space = tdx.tdx_tune_gemm_guided(M, N, K, 0, tB, tdx.TDX_BF16, budget, iters=10, cap=8192)
    assert st == 0, tdx.tdx_last_error()
    assert n_space == len(tried_all) and n_space > 4 * budget         # the model really pruned something
    assert 1 <= len(tried) <= budget + 5                              # the budget, the automatic choice, up to four cached winners of other shapes
    # within 15 % of the exhaustive winner (timing noise between the two searches is a few per cent)
    assert us <= 1.15 * us_all, (best.as_dict(), us, best_all.as_dict(), us_all)
    # the winner is stored like the exhaustive one and is what the next call uses
    st, c = tdx.tdx_default_gemm_config(M, N, K, 0, tB, tdx.TDX_BF16)
    assert st == 0 and c.as_dict() == best.as_dict()
    assert tdx.tdx_tune_clear() == 0


@pytest.mark.gpu
def test_search_on_first_use_caches_the_winner_and_keeps_parity(tmp_path):
    # tdx_set_autotune(budget): the first automatic call on an unknown bf16 shape runs the guided search and caches its
    # winner; the result of that call and of the next one (served from the cache) match the oracle
    import json
    import numpy as np
    import seeded_inputs as si
    from gpu_util import TIGHT, gemm_error, run_gemm
    M, N, K = 1152, 896, 640
    key = f"gemm:{M}:{N}:{K}:0:1:{tdx.TDX_BF16}"
    path = tmp_path / "cache.json"
    assert tdx.tdx_tune_save(str(path)) == 0
    assert key not in path.read_text()
    A, B = si.gemm_bf16_normal(M, N, K, seed=95, transB=1)
    assert tdx.tdx_set_autotune(6) == 0
    try:
        for _ in range(2):
            st, C, ok = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B)
            assert st == 0 and ok, tdx.tdx_last_error()
            assert gemm_error(M, N, K, 0, 1, 1.0, "bf16", A, B, C) < TIGHT["bf16"]
    finally:
        assert tdx.tdx_set_autotune(0) == 0
    assert tdx.tdx_tune_save(str(path)) == 0
    assert key in path.read_text()


@pytest.mark.gpu
def test_exhaustive_gemm_search_winner_matches_the_oracle():
    # whatever the search caches is what plain calls are then served with: run it and compare with the oracle
    import seeded_inputs as si
    from gpu_util import TIGHT, gemm_error, run_gemm
    M, N, K = 640, 1152, 768
    st, best, us, tried = tdx.tdx_tune_gemm(M, N, K, 0, 1, tdx.TDX_BF16, iters=5, cap=8192)
    assert st == 0 and us > 0 and len(tried) > 8, tdx.tdx_last_error()
    assert us <= min(t for _, t in tried) * 1.0001              # the fastest candidate passed the search's own output check
    try:
        st, c = tdx.tdx_default_gemm_config(M, N, K, 0, 1, tdx.TDX_BF16)
        assert st == 0 and c.as_dict() == best.as_dict()
        A, B = si.gemm_bf16_normal(M, N, K, seed=96, transB=1)
        st, C, ok = run_gemm(M, N, K, 0, 1, -1.0, "bf16", A, B)             # served from the cache
        assert st == 0 and ok, tdx.tdx_last_error()
        assert gemm_error(M, N, K, 0, 1, -1.0, "bf16", A, B, C) < TIGHT["bf16"]
        assert tdx.tdx_check_device_status() == 0
    finally:
        assert tdx.tdx_tune_clear() == 0
        tdx.tdx_tune_load(str(__import__("pathlib").Path(tdx.__file__).parent / "tuned_b200.json"))


@pytest.mark.gpu
@pytest.mark.parametrize("case", [(2, 28, 28, 64, 128, 3, 3, 1, 1), (2, 30, 30, 64, 64, 3, 3, 1, 2), (3, 14, 14, 128, 64, 1, 1, 0, 1)])
def test_conv_search_winner_matches_the_oracle(case):
    # tdx_tune_conv2d: every candidate of the convolution's search space is timed, the winner's output is checked
    # against the generic kernel inside the search, cached, and then serves tdx_conv2d_bias_relu: compare with the oracle
    import seeded_inputs as si
    from gpu_util import TIGHT, conv_error, run_conv
    N, H, W, Cin, Cout, R, S, pad, stride = case
    st, space = tdx.tdx_enum_conv2d_configs(N, H, W, Cin, Cout, R, S, pad, stride, tdx.TDX_BF16)
    assert st == 0 and len(space) > 1
    st, best, us, tried = tdx.tdx_tune_conv2d(N, H, W, Cin, Cout, R, S, pad, stride, tdx.TDX_BF16, iters=5, cap=4096)
    assert st == 0 and us > 0, tdx.tdx_last_error()
    assert 1 < len(tried) <= len(space)
    assert best.as_dict() in space
    try:
        st, c = tdx.tdx_default_conv2d_config(N, H, W, Cin, Cout, R, S, pad, stride, tdx.TDX_BF16)
        assert st == 0 and c.as_dict() == best.as_dict()
        x, w, b = si.conv_bf16(N, H, W, Cin, Cout, R, S, seed=97)
        st, y, ok = run_conv(N, H, W, Cin, Cout, R, S, pad, stride, "bf16", x, w, b, 1)
        assert st == 0 and ok, tdx.tdx_last_error()
        assert conv_error(N, H, W, Cin, Cout, R, S, pad, stride, "bf16", x, w, b, 1, y) < TIGHT["bf16"]
        assert tdx.tdx_check_device_status() == 0
    finally:
        assert tdx.tdx_tune_clear() == 0
        tdx.tdx_tune_load(str(__import__("pathlib").Path(tdx.__file__).parent / "tuned_b200.json"))


def test_conv_cost_model_orders_known_cases():
    # host only: orderings the measurements established for the two convolution kernels
    def us(case, **kw):
        st, v = tdx.tdx_model_conv2d_us(*case, tdx.TDX_BF16, umma(**kw))
        assert st == tdx.TDX_OK, tdx.tdx_last_error()
        return v
    c4 = (32, 56, 56, 256, 256, 3, 3, 1, 1)
    assert us(c4, halo=3, tile_m=128, tile_n=256) < us(c4, halo=2, tile_m=128, tile_n=256)      # stacking wastes fewer rows
    assert us(c4, halo=2, tile_m=128, tile_n=256) < us(c4, halo=1, tile_m=128, tile_n=256)      # the window is fetched once, not nine times
    assert us(c4, halo=3, tile_m=128, tile_n=256) < us(c4, halo=3, tile_m=128, tile_n=64)       # narrow MMAs run at half rate
    s2 = (32, 56, 56, 256, 512, 3, 3, 1, 2)
    assert us(s2, halo=1, tile_m=128, tile_n=256) > 0
    st, _ = tdx.tdx_model_conv2d_us(1, 9, 11, 5, 7, 3, 3, 1, 1, tdx.TDX_BF16, tdx.tdx_config())    # generic kernel: no model
    assert st == tdx.TDX_ERR_UNSUPPORTED


@pytest.mark.gpu
@pytest.mark.parametrize("case", [(2, 64, 64, 64, 64, 3, 3, 1, 1), (8, 56, 56, 128, 256, 3, 3, 1, 1), (8, 28, 28, 256, 512, 3, 3, 1, 2)])
def test_guided_conv_search_finds_a_configuration_close_to_the_exhaustive_best(case):
    # scaled-down relatives of the two convolution workloads and a strided layer: a budget of 16 candidates, chosen by
    # the cost model, lands within 15 % of the winner of the exhaustive search
    budget = 16
    st, best_all, us_all, tried_all = tdx.tdx_tune_conv2d(*case, tdx.TDX_BF16, iters=8, cap=8192)
    assert st == 0, tdx.tdx_last_error()
    st, best, us, tried, n_space = tdx.tdx_tune_conv2d_guided(*case, tdx.TDX_BF16, budget, iters=8, cap=8192)
    assert st == 0, tdx.tdx_last_error()
    assert n_space == len(tried_all) and n_space > 4 * budget
    assert 1 <= len(tried) <= budget + 1
    assert us <= 1.15 * us_all, (best.as_dict(), us, best_all.as_dict(), us_all)
    st, c = tdx.tdx_default_conv2d_config(*case, tdx.TDX_BF16)
    assert st == 0 and c.as_dict() == best.as_dict()
    assert tdx.tdx_tune_clear() == 0
    tdx.tdx_tune_load(str(__import__("pathlib").Path(tdx.__file__).parent / "tuned_b200.json"))


@pytest.mark.gpu
def test_search_over_a_stated_space():
    # Case Study 5's form: ranges + "divides" + a conditional; the winner comes from that space only, is checked and cached
    M, N, K = 1536, 1280, 1024
    space = ("tile_m in {128, 256}; tile_n in 64..256 step 64; split_k in {1, 2}; "
             "require M % tile_m == 0; require N % tile_n == 0; store_mode == 2 only if split_k == 1")
    st, cfgs, prod, kept = tdx.tdx_enum_gemm_space(M, N, K, 0, 1, tdx.TDX_BF16, space)
    assert st == 0 and prod == 16 and kept == 12          # tile_n 192 does not divide 1280: four candidates gone
    st, best, us, tried, n_cand = tdx.tdx_tune_gemm_space(M, N, K, 0, 1, tdx.TDX_BF16, space, iters=8, cap=512)
    assert st == 0 and us > 0, tdx.tdx_last_error()
    assert n_cand == len(cfgs) == len(tried)
    assert best.as_dict() in cfgs and best.tile_n != 192
    st, best2, us2, tried2, _ = tdx.tdx_tune_gemm_space(M, N, K, 0, 1, tdx.TDX_BF16, space, budget=4, iters=8, cap=512)
    assert st == 0 and len(tried2) <= 4 and best2.as_dict() in cfgs and us2 <= 1.2 * us
    try:
        import seeded_inputs as si
        from gpu_util import TIGHT, gemm_error, run_gemm
        A, B = si.gemm_bf16_normal(M, N, K, seed=99, transB=1)
        st, C, ok = run_gemm(M, N, K, 0, 1, 1.0, "bf16", A, B)             # served with the cached winner
        assert st == 0 and ok and gemm_error(M, N, K, 0, 1, 1.0, "bf16", A, B, C) < TIGHT["bf16"]
    finally:
        assert tdx.tdx_tune_clear() == 0
        tdx.tdx_tune_load(str(__import__("pathlib").Path(tdx.__file__).parent / "tuned_b200.json"))
    # constraints nothing satisfies
    st, *_ = tdx.tdx_tune_gemm_space(M, N, K, 0, 1, tdx.TDX_BF16, "tile_n in {192}; require N % tile_n == 0", iters=2)
    assert st == tdx.TDX_ERR_UNSUPPORTED
