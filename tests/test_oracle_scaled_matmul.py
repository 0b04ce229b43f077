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
