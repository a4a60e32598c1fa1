"""The caller-stated search space (tdx_enum_gemm_space): ranges, the two constraint kinds of the paper's Case Study 5
-- a tile size must divide its dimension; vectorise only if a divisibility condition holds -- and the hardware's own
constraints applied afterwards.  Host only."""
import pytest

import paper_2409_03864_b200 as tdx

BF16 = tdx.TDX_BF16


def enum(M, N, K, space, tA=0, tB=1):
    st, cfgs, prod, kept = tdx.tdx_enum_gemm_space(M, N, K, tA, tB, BF16, space)
    assert st == tdx.TDX_OK, tdx.tdx_last_error()
    return cfgs, prod, kept


def test_ranges_form_a_cross_product():
    cfgs, prod, kept = enum(1024, 1024, 1024, "tile_m in {128, 256}; tile_n in 64..256 step 64; split_k in {1, 2}")
    assert prod == 2 * 4 * 2 and kept == prod
    seen = {(c["tile_m"], c["tile_n"], c["split_k"]) for c in cfgs}
    assert seen <= {(m, n, s) for m in (128, 256) for n in (64, 128, 192, 256) for s in (1, 2)}
    assert len(seen) == len(cfgs)                         # no duplicates
    assert all(c["kernel"] == tdx.TDX_KERNEL_UMMA and c["stages"] >= 2 and c["store_mode"] in (1, 2) for c in cfgs)
    # parameters that were not mentioned were filled in by the library's rules
    assert all(c["tile_k"] == 64 and c["cta_pair"] == 1 for c in cfgs)


def test_tile_sizes_must_divide_their_dimension():
    # the first constraint kind: `require M % tile_m == 0` / `require N % tile_n == 0`
    space = "tile_m in {128, 256}; tile_n in 32..256 step 32; require M % tile_m == 0; require N % tile_n == 0"
    cfgs, prod, kept = enum(384, 480, 512, space)
    assert prod == 16
    # 384 = 3 * 128 (256 does not divide it); of 32..256 step 32 only 32, 96, 160, 240(no: not in the list), 480's divisors
    divisors_n = [n for n in range(32, 257, 32) if 480 % n == 0]
    assert divisors_n == [32, 96, 160]
    assert kept == 1 * len(divisors_n)
    assert {(c["tile_m"], c["tile_n"]) for c in cfgs} == {(128, n) for n in divisors_n}
    # a shape everything divides keeps the whole cross product
    _, prod, kept = enum(512, 512, 512, "tile_m in {128, 256}; tile_n in {64, 128, 256}; require M % tile_m == 0; require N % tile_n == 0")
    assert kept == prod == 6


def test_vectorised_stores_only_if_the_row_length_divides():
    # the second kind, the paper's conditional `vect`: a value of one parameter is allowed only under a condition
    space = "store_mode in {1, 2}; tile_n in {64, 128}; store_mode == 2 only if N % 64 == 0 && split_k == 1; split_k in {1, 2}"
    cfgs, prod, kept = enum(512, 520, 512, space)          # 520 % 64 != 0: no staged (whole-line) stores
    assert prod == 8 and kept == 4
    assert cfgs and all(c["store_mode"] == 1 for c in cfgs)
    cfgs, prod, kept = enum(512, 512, 512, space)          # 512 % 64 == 0: staged stores where K is not split
    assert kept == 6
    assert {(c["store_mode"], c["split_k"]) for c in cfgs} == {(1, 1), (1, 2), (2, 1)}


def test_the_hardware_constraints_still_apply():
    # 8 stages of a 256 x 256 tile do not fit shared memory; tile_n = 96 is no multiple of 64 for an N-major B
    cfgs, prod, kept = enum(2048, 2048, 2048, "tile_m in {256}; tile_n in {256}; stages in 2..8")
    assert prod == kept == 7 and sorted(c["stages"] for c in cfgs) == [2, 3]
    cfgs, prod, kept = enum(2048, 2048, 2048, "tile_n in {64, 96, 128}", tA=0, tB=0)
    assert kept == 3 and sorted(c["tile_n"] for c in cfgs) == [64, 128]
    # an empty K slice is infeasible whatever the stated rules say
    cfgs, _, _ = enum(256, 256, 192, "split_k in {1, 2, 3, 4}; store_mode in {1}")
    assert sorted(c["split_k"] for c in cfgs) == [1, 2, 3]


def test_expressions():
    space = ("tile_m in {128, 256}; tile_n in {64, 128, 192, 256}; "
             "require (tile_m * tile_n >= 32768 || K < 1024) && !(tile_m == 256 && tile_n == 64); "
             "require num_kb / 4 >= 2; require transB == 1")
    cfgs, prod, kept = enum(1024, 1024, 2048, space)
    want = {(m, n) for m in (128, 256) for n in (64, 128, 192, 256) if m * n >= 32768 and not (m == 256 and n == 64)}
    assert kept == len(want) and {(c["tile_m"], c["tile_n"]) for c in cfgs} == want
    _, _, kept = enum(1024, 1024, 2048, space, tB=0)
    assert kept == 0


@pytest.mark.parametrize("space,fragment", [
    ("tile_q in {1, 2}", "unknown parameter"),
    ("tile_m in {128}; tile_m in {256}", "given twice"),
    ("tile_m in 128", "expected"),
    ("tile_m in {128}; require M % tile_z == 0", "unknown name"),
    ("tile_m in {128}; require M % 0 == 0", "division by zero"),
    ("tile_m in {128}; require (M > 1", "missing ')'"),
    ("tile_m in {}", "empty range"), ("tile_m in {128, x}", "expected an integer"),
    ("garbage", "cannot read"),
    ("tile_m in 1..10000000", "bad range"),
])
def test_syntax_errors_are_reported(space, fragment):
    st, cfgs, _, _ = tdx.tdx_enum_gemm_space(512, 512, 512, 0, 1, BF16, space)
    assert st == tdx.TDX_ERR_INVALID_ARG and cfgs == []
    assert fragment in tdx.tdx_last_error()


def test_other_problems_are_refused():
    assert tdx.tdx_enum_gemm_space(256, 256, 256, 0, 0, tdx.TDX_F32, "tile_m in {128}")[0] == tdx.TDX_ERR_UNSUPPORTED
    assert tdx.tdx_enum_gemm_space(196, 256, 2305, 0, 0, BF16, "tile_m in {128}")[0] == tdx.TDX_ERR_UNSUPPORTED
