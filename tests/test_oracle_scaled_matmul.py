"""Pins for the fp64 oracle of the block-scaled minifloat matmul (Section 3.2 numeric precision;
Section 6 ScaledMatMul): published value grids, library decoders, closed forms, brute force.  No GPU."""
import numpy as np
import pytest
import torch

from oracle import scaled_matmul as sm


def test_fp4_e2m1_grid_is_the_published_one():
    t = sm.decode_table(sm.E2M1)
    assert list(t[:8]) == [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]
    assert list(t[8:]) == [-0.0, -0.5, -1.0, -1.5, -2.0, -3.0, -4.0, -6.0]
    assert np.signbit(t[8])


def test_fp6_and_fp8_extremes():
    # largest normal / smallest subnormal of each grid, from the format parameters
    assert np.nanmax(sm.decode_table(sm.E2M3)) == 7.5 and sm.decode_table(sm.E2M3)[1] == 0.125
    assert np.nanmax(sm.decode_table(sm.E3M2)) == 28.0 and sm.decode_table(sm.E3M2)[1] == 0.0625
    e4 = sm.decode_table(sm.E4M3)
    assert np.nanmax(e4) == 448.0 and e4[1] == 2.0 ** -9 and np.isnan(e4[0x7F]) and np.isnan(e4[0xFF])
    assert not np.isinf(e4).any()
    e5 = sm.decode_table(sm.E5M2)
    assert np.nanmax(e5[np.isfinite(e5)]) == 57344.0 and e5[1] == 2.0 ** -16
    assert e5[0x7C] == np.inf and e5[0xFC] == -np.inf and np.isnan(e5[0x7D:0x80]).all()


def test_fp8_tables_match_library_decoders():
    codes = torch.arange(256, dtype=torch.uint8)
    for fmt, dt in ((sm.E4M3, torch.float8_e4m3fn), (sm.E5M2, torch.float8_e5m2)):
        lib = codes.view(dt).double().numpy()
        ours = sm.decode_table(fmt)
        assert np.array_equal(np.isnan(lib), np.isnan(ours))
        ok = ~np.isnan(lib)
        assert np.array_equal(lib[ok], ours[ok]) and np.array_equal(np.signbit(lib[ok]), np.signbit(ours[ok]))
    # E5M2 is the high byte of IEEE half precision
    half = (np.arange(256, dtype=np.uint16) << 8).view(np.float16).astype(np.float64)
    ok = ~np.isnan(half)
    assert np.array_equal(half[ok], sm.decode_table(sm.E5M2)[ok])


def test_e8m0_scales_match_library_and_closed_form():
    e = np.arange(256)
    ours = sm.scale_value(e)
    assert ours[127] == 1.0 and ours[0] == 2.0 ** -127 and ours[254] == 2.0 ** 127 and np.isnan(ours[255])
    lib = torch.arange(256, dtype=torch.uint8).view(torch.float8_e8m0fnu).double().numpy()
    assert np.array_equal(lib[:255], ours[:255]) and np.isnan(lib[255])


def test_generic_format_reduces_to_known_ones_and_to_integers():
    # fNe5m10 without specials below the top exponent is IEEE half on all finite codes
    f16 = sm.decode_table(sm.MiniFloat(5, 10, "ieee"))
    ref = np.arange(65536, dtype=np.uint16).view(np.float16).astype(np.float64)
    ok = np.isfinite(ref)
    assert np.array_equal(f16[ok], ref[ok])
    # one exponent bit (bias 0): subnormals 0.m * 2^1 then the binade [2, 4): a fixed-point grid of step 0.5
    t = sm.decode_table(sm.MiniFloat(1, 2, "none"))
    assert list(t[:8]) == [0.0, 0.5, 1.0, 1.5, 2.0, 2.5, 3.0, 3.5]
    # grids are symmetric and monotone in the magnitude code
    for fmt in (sm.E2M1, sm.E2M3, sm.E3M2, sm.MiniFloat(3, 4, "none")):
        t = sm.decode_table(fmt)
        half = t.size // 2
        assert np.array_equal(t[half:], -t[:half]) and (np.diff(t[:half]) > 0).all()


def test_nibble_unpacking_order():
    packed = np.array([[0x21, 0xF0]], np.uint8)
    assert sm.unpack_nibbles(packed).tolist() == [[1, 2, 0, 15]]


def test_dequantise_blocks_and_matmul_brute_force():
    rng = np.random.default_rng(0)
    N, K, M = 3, 64, 2
    codes = rng.integers(0, 16, size=(N, K)).astype(np.uint8)
    scales = rng.integers(120, 135, size=(N, K // 32)).astype(np.uint8)
    W = sm.dequantise(codes, scales, sm.E2M1)
    grid = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]
    x = rng.standard_normal((M, K))
    bias = rng.standard_normal(N)
    y = sm.scaled_matmul(x, codes, scales, sm.E2M1, bias)
    for n in range(N):
        for k in range(K):
            c = int(codes[n, k])
            v = (-1.0 if c & 8 else 1.0) * grid[c & 7] * 2.0 ** (int(scales[n, k // 32]) - 127)
            assert W[n, k] == v
    for m in range(M):
        for n in range(N):
            acc = bias[n]
            for k in range(K):
                acc += x[m, k] * W[n, k]
            assert abs(acc - y[m, n]) <= 1e-12 * (1 + abs(acc))
    # scale 127 everywhere and codes of 1.0 -> plain row sums of x
    ones = np.full((N, K), 2, np.uint8)                      # code 2 = 1.0 in E2M1
    y1 = sm.scaled_matmul(x, ones, np.full((N, K // 32), 127, np.uint8), sm.E2M1)
    np.testing.assert_allclose(y1, np.repeat(x.sum(1, keepdims=True), N, 1), rtol=1e-14)
    # raising one block's scale byte by 1 doubles exactly that block's contribution
    s2 = np.full((N, K // 32), 127, np.uint8)
    s2[1, 1] = 128
    y2 = sm.scaled_matmul(x, ones, s2, sm.E2M1)
    np.testing.assert_allclose(y2[:, 1] - y1[:, 1], x[:, 32:].sum(1), rtol=1e-13)
    assert np.array_equal(y2[:, [0, 2]], y1[:, [0, 2]])


def test_shape_checks():
    with pytest.raises(AssertionError):
        sm.dequantise(np.zeros((2, 48), np.uint8), np.zeros((2, 1), np.uint8), sm.E4M3)


# ---------------------------------------------------------------- quantised activations (MX rule)
def test_element_maxima_give_the_shared_exponent_offsets():
    assert sm.emax(sm.E4M3) == 8 and sm.emax(sm.E5M2) == 15 and sm.emax(sm.E2M1) == 2


def test_quantise_elements_is_the_identity_on_the_grid_and_rounds_to_even_between():
    for fmt in (sm.E4M3, sm.E5M2, sm.E2M1):
        t = sm.decode_table(fmt)
        finite = np.array([c for c in range(t.size) if np.isfinite(t[c])])
        assert np.array_equal(sm.quantise_elements(t[finite], fmt), finite)          # signed zero included
    # E4M3 around 1: grid step 1/8; midpoints go to the even mantissa
    assert sm.quantise_elements(np.array([1.0625, 1.1875, 1.06, 1.07]), sm.E4M3).tolist() == [0x38, 0x3A, 0x38, 0x39]
    # saturation keeps the sign and never produces the NaN code
    assert sm.quantise_elements(np.array([1e9, -1e9, 449.0, 464.0]), sm.E4M3).tolist() == [0x7E, 0xFE, 0x7E, 0x7E]
    # subnormal range of E4M3: step 2^-9, half a step rounds to even (zero), just above goes up
    assert sm.quantise_elements(np.array([2.0 ** -10, 2.0 ** -10 * 1.01, 3 * 2.0 ** -10]), sm.E4M3).tolist() == [0, 1, 2]


def test_quantise_elements_agrees_with_the_library_cast_in_range():
    rng = np.random.default_rng(1)
    v = np.concatenate([rng.standard_normal(4000) * 50, rng.standard_normal(4000) * 0.01, rng.uniform(-448, 448, 4000)])
    v = v.astype(np.float32).astype(np.float64)
    for fmt, dt, top in ((sm.E4M3, torch.float8_e4m3fn, 448.0), (sm.E5M2, torch.float8_e5m2, 57344.0)):
        inside = v[np.abs(v) <= top]
        lib = torch.from_numpy(inside).to(torch.float32).to(dt).view(torch.uint8).numpy()
        assert np.array_equal(sm.quantise_elements(inside, fmt), lib)


def test_quantise_mx_scales_bounds_and_idempotence():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((7, 128)) * np.exp2(rng.integers(-20, 20, size=(7, 1)))
    x[3, 32:64] = 0.0                                   # an all-zero block
    x[5, 0] = 3.0e38                                     # the top of the range
    codes, scales = sm.quantise_mx(x, sm.E4M3)
    assert codes.shape == (7, 128) and scales.shape == (7, 4) and scales[3, 1] == 127
    xq = sm.dequantise(codes, scales, sm.E4M3)
    assert np.isfinite(xq).all() and np.all(xq[3, 32:64] == 0)
    blocks = np.abs(x.reshape(7, 4, 32)).max(axis=2)
    s = scales.astype(np.int64) - 127
    nz = blocks > 0
    # the block maximum lands in the top binade of the element grid: 2^8 <= amax / 2^s < 2^9
    ratio = blocks[nz] / np.exp2(s[nz])
    assert np.all(ratio >= 256) and np.all(ratio < 512)
    # error: half an element step (2^(e-3) for a value in binade e, never below the subnormal step) or saturation
    scaled = x.reshape(7, 4, 32) / np.exp2(s)[:, :, None]
    err = np.abs(xq.reshape(7, 4, 32) / np.exp2(s)[:, :, None] - scaled)
    step = np.exp2(np.maximum(np.floor(np.log2(np.maximum(np.abs(scaled), 1e-300))), -6) - 3)
    assert np.all((err <= step / 2) | (np.abs(scaled) > 448))
    assert np.all(np.abs(scaled) < 512)
    # quantising what is already on the grid changes nothing when the block maximum is in the top binade
    c2, s2 = sm.quantise_mx(xq, sm.E4M3)
    assert np.array_equal(sm.dequantise(c2, s2, sm.E4M3), xq)


def test_mx_matmul_is_the_plain_product_of_the_two_dequantised_operands():
    rng = np.random.default_rng(3)
    a_codes, a_scales = sm.quantise_mx(rng.standard_normal((5, 64)), sm.E4M3)
    w_codes, w_scales = sm.quantise_mx(rng.standard_normal((3, 64)) * 0.05, sm.E5M2)
    y = sm.mx_matmul(a_codes, a_scales, sm.E4M3, w_codes, w_scales, sm.E5M2, bias=np.array([1.0, 0.0, -1.0]))
    A, W = sm.dequantise(a_codes, a_scales, sm.E4M3), sm.dequantise(w_codes, w_scales, sm.E5M2)
    brute = np.array([[sum(A[m, k] * W[n, k] for k in range(64)) for n in range(3)] for m in range(5)])
    assert np.abs(y - (brute + np.array([1.0, 0.0, -1.0]))).max() <= 1e-12
    # with unit scales and integer-valued elements the product is exact integer arithmetic
    ai = rng.integers(-8, 9, size=(4, 32)).astype(np.float64)
    wi = rng.integers(-8, 9, size=(2, 32)).astype(np.float64)
    ac, asc = sm.quantise_mx(ai * 32, sm.E4M3)          # block maximum 256 -> shared exponent 0
    wc, wsc = sm.quantise_mx(wi * 32, sm.E4M3)
    if np.abs(ai).max() == 8 and np.abs(wi).max() == 8:
        assert np.all(asc == 127) and np.all(wsc == 127)
        assert np.array_equal(sm.mx_matmul(ac, asc, sm.E4M3, wc, wsc, sm.E4M3), (ai * 32) @ (wi * 32).T)
