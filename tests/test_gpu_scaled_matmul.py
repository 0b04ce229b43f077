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


# ---------------------------------------------------------------- block-scaled tensor-core path (both operands FP8)
MX_FORMATS = {"fp8_e4m3": osm.E4M3, "fp8_e5m2": osm.E5M2}


def _mx_word(rlx, name):
    f = MX_FORMATS[name]
    return rlx.binding.minifloat(f.ebits, f.mbits, SPECIAL[f.special], False)


def _u8_dev(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint8)).cuda()


@pytest.mark.parametrize("name", sorted(MX_FORMATS))
def test_quantise_mx_is_bit_exact_against_the_definition(rlx, name):
    """Codes and scale bytes are integer decisions: every one must equal the oracle's (the inputs are bf16,
    the scaling is by exact powers of two, and the rounding rule is round-to-nearest-even on both sides)."""
    fmt = MX_FORMATS[name]
    rng = np.random.default_rng(5)
    M, K = 77, 384
    x = rng.standard_normal((M, K)).astype(np.float32) * np.exp2(rng.integers(-30, 30, size=(M, K // 32))).repeat(32, axis=1).astype(np.float32)
    x[3, 64:96] = 0.0                                      # all-zero block
    x[5, 0] = 3.0e38                                       # top of the range: shared exponent clamps at 127
    x[6, :32] = 1e-38                                      # bottom: bf16 subnormal neighbourhood
    x[7, :32] = np.linspace(0.9, 1.1, 32) * 256.0          # block maximum just past a binade edge
    x[8, :32] = 255.0
    x[8, 5] = 256.0
    # every tie of the element grid: midpoints between neighbouring E4M3 / E5M2 values, block maximum 256 or 2^15
    t = osm.decode_table(fmt)
    pos = np.sort(t[: t.size // 2][np.isfinite(t[: t.size // 2])])
    mids = (pos[:-1] + pos[1:]) / 2
    top = 2.0 ** osm.emax(fmt)
    for r, chunk in enumerate(np.array_split(mids, 8)):
        row = np.zeros(K, np.float32)
        row[:32] = top
        row[32:32 + chunk.size] = chunk[:K - 32]
        row[0] = top
        for b in range(1, K // 32):
            row[b * 32] = top                               # shared exponent 0 in every block
        x[10 + r] = row
    x = round_to_bf16(x)
    codes, scales = rlx.quantise_mx(bf16_dev(x), _mx_word(rlx, name))
    want_codes, want_scales = osm.quantise_mx(x.astype(np.float64), fmt)
    assert np.array_equal(scales.cpu().numpy(), want_scales)
    assert np.array_equal(codes.cpu().numpy(), want_codes)


@pytest.mark.parametrize("N", [256, 384], ids=["tiles_128", "tiles_192"])
def test_mx_matmul_places_every_scale_byte_and_operand_where_the_definition_says(rlx, N):
    """Exact cases that fail if a scale byte reaches the wrong row, column or k-group, or an operand tile is
    transposed: all elements 1.0 with a different power-of-two scale per (row, k-group) and per (column,
    k-group); then integer-valued elements with unit scales (integer arithmetic, exact in fp32)."""
    M, K = 300, 1024                  # ragged rows, two column tiles (128- or 192-wide), 8 stages of k: every ring wraps
    rng = np.random.default_rng(6)
    one = 0x38                          # 1.0 in E4M3
    a_codes = np.full((M, K), one, np.uint8)
    w_codes = np.full((N, K), one, np.uint8)
    a_scales = (127 + rng.integers(-3, 4, size=(M, K // 32))).astype(np.uint8)
    w_scales = (127 + rng.integers(-3, 4, size=(N, K // 32))).astype(np.uint8)
    word = _mx_word(rlx, "fp8_e4m3")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = to_np64(rlx.mx_matmul_bf16(_u8_dev(a_codes), _u8_dev(a_scales), word, _u8_dev(w_codes), _u8_dev(w_scales), word,
                                     status=status))
    assert int(status.item()) == 0
    want = osm.mx_matmul(a_codes, a_scales, osm.E4M3, w_codes, w_scales, osm.E4M3)
    assert np.array_equal(got, round_to_bf16(want.astype(np.float32)).astype(np.float64))   # sums of 32 * 2^e: exact
    # integers in [-4, 4] (E4M3 holds them exactly), unit scales: |sum| <= 16 * 1024, exact in fp32; bf16 rounds once
    ai = rng.integers(-4, 5, size=(M, K))
    wi = rng.integers(-4, 5, size=(N, K))
    ac = osm.quantise_elements(ai.astype(np.float64), osm.E4M3)
    wc = osm.quantise_elements(wi.astype(np.float64), osm.E4M3)
    ones = np.full((max(M, N), K // 32), 127, np.uint8)
    bias = rng.integers(-8, 9, size=N).astype(np.float32)
    got = to_np64(rlx.mx_matmul_bf16(_u8_dev(ac), _u8_dev(ones[:M]), word, _u8_dev(wc), _u8_dev(ones[:N]), word,
                                     bias=f32_dev(bias)))
    exact = (ai @ wi.T + bias).astype(np.float32)
    assert np.array_equal(got, round_to_bf16(exact).astype(np.float64))


@pytest.mark.parametrize("a_name,w_name", [("fp8_e4m3", "fp8_e4m3"), ("fp8_e4m3", "fp8_e5m2"), ("fp8_e5m2", "fp8_e4m3")])
@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (517, 384, 384), (2000, 1536, 384), (1000, 384, 1536)])
def test_quantise_then_mx_matmul_matches_oracle(rlx, a_name, w_name, M, N, K):
    """The whole path on encoder-shaped operands: activations quantised on the GPU (bit-exact, previous test),
    weights quantised by the oracle's rule on the host, product on the block-scaled tensor-core path,
    compared with the fp64 product of the two dequantised operands.  Products are exact; the error is fp32
    accumulation (K terms, relative 2^-24 each against the sum of magnitudes) plus the bf16 store."""
    rng = np.random.default_rng(M + N + K)
    x = rand_bf16(rng, (M, K))
    w = (rng.standard_normal((N, K)) * 0.05).astype(np.float32)
    bias = rng.standard_normal(N).astype(np.float32)
    a_codes, a_scales = rlx.quantise_mx(bf16_dev(x), _mx_word(rlx, a_name))
    w_codes, w_scales = osm.quantise_mx(w.astype(np.float64), MX_FORMATS[w_name])
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = to_np64(rlx.mx_matmul_bf16(a_codes, a_scales, _mx_word(rlx, a_name), _u8_dev(w_codes), _u8_dev(w_scales),
                                     _mx_word(rlx, w_name), bias=f32_dev(bias), status=status))
    assert int(status.item()) == 0
    A = osm.dequantise(a_codes.cpu().numpy(), a_scales.cpu().numpy(), MX_FORMATS[a_name])
    W = osm.dequantise(w_codes, w_scales, MX_FORMATS[w_name])
    ref = A @ W.T + bias
    mag = np.abs(A) @ np.abs(W).T + np.abs(bias)
    half_ulp = np.exp2(np.floor(np.log2(np.maximum(np.abs(ref), 1e-300))) - 8)     # bf16: 8 significant bits
    assert np.all(np.abs(got - ref) <= half_ulp + K * 2.0 ** -23 * mag + 1e-30)
    # and the quantised product stays close to the unquantised one: the point of the format
    full = x.astype(np.float64) @ w.astype(np.float64).T + bias
    rel = np.linalg.norm(got - full) / np.linalg.norm(full)
    assert rel < (0.04 if "e5m2" not in (a_name + w_name) else 0.08)
