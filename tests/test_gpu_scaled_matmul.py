"""Block-scaled minifloat dequantisation and ScaledMatMul through the C ABI against the fp64 oracle.

Dequantisation is byte-level work: the bf16 result must equal, bit for bit, the exact weight rounded
the way the kernel's precision fixes it (fp32 round-to-nearest-even of the exact product, which is
exact down to 2^-149, then bf16 round-to-nearest-even, which is exact wherever the product lies in
bf16's range).  The matmul is compared like the other GEMM tests: bf16 storage of the output (relative
2^-8) plus fp32 accumulation slack, and bit-exactly on inputs whose partial sums are all exact."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import scaled_matmul as osm  # noqa: E402
from synth.inputs import bf16_bits, make_block_scaled_weights, pack_nibbles, round_to_bf16  # noqa: E402
from gpu_common import BF16_U, bf16_dev, f32_dev, rand_bf16, to_np64  # noqa: E402

pytestmark = pytest.mark.gpu

# name -> (oracle format, code bits, largest finite magnitude code, packed4)
FORMATS = {
    "fp8_e4m3": (osm.E4M3, 8, 0x7E, False),
    "fp8_e5m2": (osm.E5M2, 8, 0x7B, False),
    "fp6_e3m2": (osm.E3M2, 6, 0x1F, False),
    "fp6_e2m3": (osm.E2M3, 6, 0x1F, False),
    "fp4_e2m1": (osm.E2M1, 4, 0x7, True),
    "f1e3m4": (osm.MiniFloat(3, 4, "none"), 8, 0x7F, False),
    "f1e6m1": (osm.MiniFloat(6, 1, "none"), 8, 0x7F, False),
    "f1e1m2_packed": (osm.MiniFloat(1, 2, "none"), 4, 0x7, True),
}
SPECIAL = {"none": 0, "nan_only": 1, "ieee": 2}


@pytest.fixture(scope="module")
def rlx():
    import paper_2609_37916_b200 as pkg
    from paper_2609_37916_b200.build import build
    build()
    return pkg


def _fmt_word(rlx, name):
    f, _, _, packed = FORMATS[name]
    return rlx.binding.minifloat(f.ebits, f.mbits, SPECIAL[f.special], packed)


def _dev_codes(codes, packed):
    host = pack_nibbles(codes) if packed else codes
    return torch.from_numpy(np.ascontiguousarray(host)).cuda()


def _expected_bf16(w64):
    """exact weight -> fp32 (RNE) -> bf16 (RNE), as float32 values on the bf16 grid"""
    with np.errstate(over="ignore"):
        return round_to_bf16(w64.astype(np.float32))


def _assert_same_bits(got_t, want32):
    got = got_t.float().cpu().numpy()
    nan = np.isnan(want32)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(bf16_bits(got[~nan]), bf16_bits(want32[~nan]))     # includes the sign of zero


@pytest.mark.parametrize("name", list(FORMATS))
def test_dequant_every_code_every_scale_is_exact(rlx, name):
    f, bits, _, packed = FORMATS[name]
    ncodes = 1 << bits
    N, K = 254, max(ncodes, 32)
    codes = np.tile(np.arange(ncodes, dtype=np.uint8), (N, K // ncodes))      # every code, specials included
    scales = np.repeat(np.arange(1, 255, dtype=np.uint8)[:, None], K // 32, 1)  # row n: scale byte n + 1
    scales[7, 0] = 255                                                         # one NaN scale
    got = rlx.dequant_block_scaled_bf16(_dev_codes(codes, packed), torch.from_numpy(scales).cuda(), N, K,
                                        _fmt_word(rlx, name))
    want = osm.dequantise(codes, scales, f)
    # in-range weights are exactly representable: no rounding at all
    inr = np.isfinite(want) & (np.abs(want) < 2.0 ** 127) & ((np.abs(want) >= 2.0 ** -126) | (want == 0))
    assert np.array_equal(to_np64(got)[inr], want[inr])
    _assert_same_bits(got, _expected_bf16(want))


@pytest.mark.parametrize("name", list(FORMATS))
def test_dequant_random_weights_ragged_sizes(rlx, name):
    f, bits, maxmag, packed = FORMATS[name]
    for N, K in [(1, 32), (77, 96), (384, 1536)]:
        codes, scales = make_block_scaled_weights(N + K, N, K, bits, maxmag)
        got = rlx.dequant_block_scaled_bf16(_dev_codes(codes, packed), torch.from_numpy(scales).cuda(), N, K,
                                            _fmt_word(rlx, name))
        assert np.array_equal(to_np64(got), osm.dequantise(codes, scales, f))


@pytest.mark.parametrize("name", ["fp8_e4m3", "fp6_e2m3", "fp4_e2m1"])
@pytest.mark.parametrize("M,N,K", [(300, 384, 768), (129, 1536, 384), (5, 64, 32)])
def test_scaled_matmul_matches_oracle(rlx, name, M, N, K):
    f, bits, maxmag, packed = FORMATS[name]
    rng = np.random.default_rng(M + N + K)
    codes, scales = make_block_scaled_weights(M * 7 + N, N, K, bits, maxmag, 122, 128)
    x = rand_bf16(rng, (M, K))
    bias = rng.standard_normal(N).astype(np.float32)
    res = rand_bf16(rng, (M, N))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = to_np64(rlx.scaled_matmul_bf16(bf16_dev(x), _dev_codes(codes, packed), torch.from_numpy(scales).cuda(),
                                         _fmt_word(rlx, name), f32_dev(bias), bf16_dev(res),
                                         rlx.binding.EPI_BIAS_RESIDUAL, status=status))
    assert int(status.item()) == 0
    ref = osm.scaled_matmul(x.astype(np.float64), codes, scales, f, bias.astype(np.float64)) + res.astype(np.float64)
    W = np.abs(osm.dequantise(codes, scales, f))
    # bf16 store: 2u|ref|; fp32 accumulation of K products: K * 2^-24 * sum_k |x||w| at worst
    acc = K * 2.0 ** -24 * (np.abs(x.astype(np.float64)) @ W.T)
    assert (np.abs(got - ref) <= 2 * BF16_U * np.abs(ref) + acc + 1e-6).all(), float(np.abs(got - ref).max())


def test_scaled_matmul_is_bit_exact_when_sums_are_exact(rlx):
    """Activations in {-1, 0, 1}, FP4 weights (multiples of 0.5 up to 6) and scales 1 or 2: every partial
    sum is a small multiple of 0.5, exact in fp32, so only the final bf16 store rounds."""
    f, bits, maxmag, packed = FORMATS["fp4_e2m1"]
    M, N, K = 200, 128, 64
    rng = np.random.default_rng(9)
    codes, scales = make_block_scaled_weights(9, N, K, bits, maxmag, 127, 128)
    x = rng.integers(-1, 2, size=(M, K)).astype(np.float32)
    zero = np.zeros(N, np.float32)
    got = rlx.scaled_matmul_bf16(bf16_dev(x), _dev_codes(codes, packed), torch.from_numpy(scales).cuda(),
                                 _fmt_word(rlx, "fp4_e2m1"), f32_dev(zero))
    ref = osm.scaled_matmul(x.astype(np.float64), codes, scales, f)
    _assert_same_bits(got, round_to_bf16(ref.astype(np.float32)))
