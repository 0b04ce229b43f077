"""rlx_attention_kind_bf16 (Causal / SlidingWindow mask kinds, rotary q,k) through the C ABI against the
fp64 oracle on the same seeded inputs.

Tolerances.  Without rotation the kernel differs from the oracle by bf16 rounding of the probabilities
(relative 2^-9 = u on each weight) and of the stored output: |err| <= 2u(max|v| + max|ref|), the bound the
encoder's own attention tests use.  With rotation the kernel also rounds the rotated q and k to bf16
before the tensor-core product, which moves a score by at most  ds = 2u * sum_c |q_c||k_c| / sqrt(d)
(each factor off by u relative; rotation preserves pair lengths, so the sum is bounded by the product of
the row norms); a softmax whose logits move by at most ds changes its weights by at most 2*ds in l1, so
the output moves by at most 2*ds*max|v|.  That worst case is loose, so the root-mean-square error is
also held to 2u*max|v|: a wrong angle, sign or pairing gives errors of order max|v| in both."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import attention_kinds as ak  # noqa: E402
from synth.inputs import round_to_bf16  # noqa: E402
from gpu_common import BF16_U, bf16_dev, i32_dev, rand_bf16, to_np64  # noqa: E402

pytestmark = pytest.mark.gpu

NONE, CAUSAL, SLIDING = ak.KIND_NONE, ak.KIND_CAUSAL, ak.KIND_SLIDING


@pytest.fixture(scope="module")
def rlx():
    import paper_2609_37916_b200 as pkg
    from paper_2609_37916_b200.build import build
    build()
    return pkg


def _run_case(rlx, lengths, h, d, kind, window, theta, gain, seed):
    rng = np.random.default_rng(seed)
    H = h * d
    total = sum(lengths)
    rows = total + 5
    qkv = rand_bf16(rng, (rows, 3 * H))
    qkv[:, :H] = round_to_bf16(qkv[:, :H] * np.float32(gain))
    qkv[total:] = np.float32("nan")                    # rows past the last sequence must not leak in
    start = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    max_len = max(lengths)
    rope = None if theta is None else rlx.rope_tables(max_len, d, theta)
    got = to_np64(rlx.attention_kind_bf16(bf16_dev(qkv), i32_dev(start[:-1]), i32_dev(np.array(lengths)), max_len, h,
                                          kind, window, rope))
    torch.cuda.synchronize()
    assert np.array_equal(got[total:], np.zeros((rows - total, H)))
    vmax = float(np.abs(qkv[:total, 2 * H:]).max())
    for b, n in enumerate(lengths):
        seq = qkv[start[b]:start[b] + n].astype(np.float64)
        ref = ak.attention_one(seq, h, kind, window, theta)
        err = np.abs(got[start[b]:start[b] + n] - ref)
        tol = 2 * BF16_U * (vmax + np.abs(ref).max())
        if theta is not None:
            q = np.abs(seq[:, :H]).reshape(n, h, d)
            k = np.abs(seq[:, H:2 * H]).reshape(n, h, d)
            qn = np.sqrt((q ** 2).sum(-1)).max(0)       # per head: largest row norm
            kn = np.sqrt((k ** 2).sum(-1)).max(0)
            ds = 2 * BF16_U * float((qn * kn).max()) / np.sqrt(d)
            tol += 2 * ds * vmax
            assert np.sqrt((err ** 2).mean()) <= 2 * BF16_U * vmax, (b, n, float(np.sqrt((err ** 2).mean())))
        assert np.isfinite(err).all() and err.max() <= tol, (b, n, float(err.max()), tol)


LENGTHS = [1, 17, 64, 65, 128, 129, 200, 300, 512]


@pytest.mark.parametrize("d", [32, 64])
@pytest.mark.parametrize("kind,window", [(NONE, 0), (CAUSAL, 0), (SLIDING, 1), (SLIDING, 5), (SLIDING, 64),
                                         (SLIDING, 100), (SLIDING, 1000)])
@pytest.mark.parametrize("theta", [None, 10000.0], ids=["plain", "rope"])
def test_kinds_match_oracle(rlx, d, kind, window, theta):
    for gain in (1.0, 4.0):
        _run_case(rlx, LENGTHS, 2, d, kind, window, theta, gain, seed=d + 7 * kind + window)


@pytest.mark.parametrize("kind,window,theta", [(CAUSAL, 0, None), (CAUSAL, 0, 10000.0), (SLIDING, 100, 10000.0),
                                               (SLIDING, 700, None), (NONE, 0, 500000.0)])
def test_long_sequences_beyond_the_encoder_limit(rlx, kind, window, theta):
    """Lengths above 512: many query tiles, and windows that let whole leading key blocks be skipped."""
    _run_case(rlx, [1500, 3, 700], 3, 32, kind, window, theta, 2.0, seed=11)
    _run_case(rlx, [1100], 1, 64, kind, window, theta, 2.0, seed=12)


def test_window_edges_are_exact(rlx):
    """Uniform weights (q = 0) make the output the mean of the visible v rows, so a key wrongly let in or
    left out at either edge of the window shifts the result by a whole 1/w share of a sentinel value."""
    h, d, n = 1, 32, 300
    H = h * d
    for w in (1, 2, 63, 64, 65, 128, 129):
        qkv = np.zeros((n, 3 * H), np.float32)
        qkv[:, 2 * H:] = np.where(np.arange(n) % 7 == 0, np.float32(64.0), np.float32(0.0))[:, None]
        got = to_np64(rlx.attention_kind_bf16(bf16_dev(qkv), i32_dev(np.array([0])), i32_dev(np.array([n])), n, h,
                                              SLIDING, w))
        ref = ak.attention_one(qkv.astype(np.float64), h, SLIDING, w)
        # weights are exactly 1 and the sums exact in fp32; the product with 1/w and the bf16 store round:
        # one bf16 ulp at most, against a shift of 64/w (>= 0.49) for a key wrongly let in or left out
        assert (np.abs(got - ref) <= 2 * BF16_U * np.abs(ref) * 1.001 + 1e-4).all(), w
    got = to_np64(rlx.attention_kind_bf16(bf16_dev(qkv), i32_dev(np.array([0])), i32_dev(np.array([n])), n, h, CAUSAL))
    ref = ak.attention_one(qkv.astype(np.float64), h, CAUSAL)
    assert (np.abs(got - ref) <= 2 * BF16_U * np.abs(ref) * 1.001 + 1e-4).all()


def test_kind_none_without_rope_is_the_encoder_kernel(rlx):
    """Same instantiation as the forward's attention: results must agree bit for bit."""
    rng = np.random.default_rng(3)
    lengths, h, d = [40, 128, 77], 4, 32
    H = h * d
    qkv = bf16_dev(rand_bf16(rng, (sum(lengths), 3 * H)))
    start = i32_dev(np.concatenate([[0], np.cumsum(lengths)])[:-1].astype(np.int32))
    slen = i32_dev(np.array(lengths))
    a = rlx.attention_kind_bf16(qkv, start, slen, max(lengths), h, NONE)
    b = rlx.attention_packed_bf16(qkv, start, slen, max(lengths), h, impl=1)
    assert torch.equal(a, b)


def test_causal_never_reads_the_future_bitwise(rlx):
    rng = np.random.default_rng(4)
    n, h, d = 333, 2, 32
    H = h * d
    qkv = rand_bf16(rng, (n, 3 * H))
    cut = 140
    pert = qkv.copy()
    pert[cut + 1:] = rand_bf16(rng, (n - cut - 1, 3 * H))
    rope = rlx.rope_tables(n, d)
    args = (i32_dev(np.array([0])), i32_dev(np.array([n])), n, h, CAUSAL, 0, rope)
    a = rlx.attention_kind_bf16(bf16_dev(qkv), *args)
    b = rlx.attention_kind_bf16(bf16_dev(pert), *args)
    assert torch.equal(a[:cut + 1], b[:cut + 1]) and not torch.equal(a[cut + 1:], b[cut + 1:])


@pytest.mark.parametrize("d,h", [(32, 3), (64, 2), (128, 2)])
def test_qk_rope_in_place_matches_oracle(rlx, d, h):
    rng = np.random.default_rng(20 + d)
    H = h * d
    lengths = [1, 15, 16, 17, 300, 1029]
    total = sum(lengths)
    rows = total + 4
    qkv = rand_bf16(rng, (rows, 3 * H), 2.0)
    start = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    rope = rlx.rope_tables(max(lengths), d, 10000.0)
    dev = bf16_dev(qkv)
    rlx.qk_rope_bf16(dev, i32_dev(start[:-1]), i32_dev(np.array(lengths)), max(lengths), h, rope)
    got = to_np64(dev)
    ref = ak.rope_qk_packed(qkv.astype(np.float64), start[:-1], lengths, h, 10000.0)
    # v and the rows past the last sequence: untouched, bit for bit
    assert np.array_equal(got[:, 2 * H:], qkv[:, 2 * H:].astype(np.float64))
    assert np.array_equal(got[total:], qkv[total:].astype(np.float64))
    # rotated values: fp32 arithmetic on fp32 tables, then one bf16 rounding (half an ulp <= 2^-8 |ref|)
    err = np.abs(got - ref)
    assert (err <= 2 * BF16_U * np.abs(ref) * 1.01 + 1e-6 * np.abs(qkv).max()).all(), float(err.max())


@pytest.mark.parametrize("d", [32, 64])
def test_separate_and_in_attention_rotation_agree_bitwise(rlx, d):
    rng = np.random.default_rng(30 + d)
    h = 2
    H = h * d
    lengths = [77, 400, 129]
    qkv = rand_bf16(rng, (sum(lengths), 3 * H), 1.5)
    start = i32_dev(np.concatenate([[0], np.cumsum(lengths)])[:-1].astype(np.int32))
    slen = i32_dev(np.array(lengths))
    rope = rlx.rope_tables(max(lengths), d)
    fused = rlx.attention_kind_bf16(bf16_dev(qkv), start, slen, max(lengths), h, CAUSAL, 0, rope)
    rot = rlx.qk_rope_bf16(bf16_dev(qkv), start, slen, max(lengths), h, rope)
    split = rlx.attention_kind_bf16(rot, start, slen, max(lengths), h, CAUSAL, 0, None)
    assert torch.equal(fused, split)


@pytest.mark.parametrize("d,hq,hkv", [(64, 8, 2), (32, 6, 3), (64, 4, 1), (128, 4, 2), (128, 2, 2)])
@pytest.mark.parametrize("kind,window,theta", [(CAUSAL, 0, 10000.0), (SLIDING, 70, None), (NONE, 0, None)])
def test_grouped_query_layout_matches_oracle(rlx, d, hq, hkv, kind, window, theta):
    """Fewer k/v heads than q heads: rows are [hq q heads | hkv k heads | hkv v heads]."""
    rng = np.random.default_rng(d + hq + hkv + kind)
    lengths = [130, 1, 257, 64]
    total = sum(lengths)
    W = (hq + 2 * hkv) * d
    qkv = rand_bf16(rng, (total, W))
    qkv[:, :hq * d] = round_to_bf16(qkv[:, :hq * d] * np.float32(3.0))
    start = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    rope = None if theta is None else rlx.rope_tables(max(lengths), d, theta)
    got = to_np64(rlx.attention_kind_bf16(bf16_dev(qkv), i32_dev(start[:-1]), i32_dev(np.array(lengths)), max(lengths), hq,
                                          kind, window, rope, num_kv_heads=hkv))
    ref = ak.attention_packed(qkv.astype(np.float64), start[:-1], lengths, hq, kind, window, theta, num_kv_heads=hkv)
    vmax = float(np.abs(qkv[:, (hq + hkv) * d:]).max())
    tol = 2 * BF16_U * (vmax + np.abs(ref).max())
    if theta is not None:
        q = np.abs(qkv[:, :hq * d].astype(np.float64)).reshape(total, hq, d)
        k = np.abs(qkv[:, hq * d:(hq + hkv) * d].astype(np.float64)).reshape(total, hkv, d)
        ds = 2 * BF16_U * float(np.sqrt((q ** 2).sum(-1)).max() * np.sqrt((k ** 2).sum(-1)).max()) / np.sqrt(d)
        tol += 2 * ds * vmax
    err = np.abs(got - ref)
    assert np.isfinite(err).all() and err.max() <= tol, (float(err.max()), tol)
    if theta is not None:
        # the separate in-place rotation, then attention without tables: the same bits
        rot = rlx.qk_rope_bf16(bf16_dev(qkv), i32_dev(start[:-1]), i32_dev(np.array(lengths)), max(lengths), hq, rope,
                               num_kv_heads=hkv)
        want = ak.rope_qk_packed(qkv.astype(np.float64), start[:-1], lengths, hq, theta, num_kv_heads=hkv)
        assert (np.abs(to_np64(rot) - want) <= 2 * BF16_U * np.abs(want) * 1.01 + 1e-6 * np.abs(qkv).max()).all()
        split = rlx.attention_kind_bf16(rot, i32_dev(start[:-1]), i32_dev(np.array(lengths)), max(lengths), hq, kind,
                                        window, None, num_kv_heads=hkv)
        assert np.array_equal(to_np64(split), got)


@pytest.mark.parametrize("kind,window,theta", [(CAUSAL, 0, 10000.0), (CAUSAL, 0, None), (SLIDING, 33, 10000.0), (NONE, 0, None)])
def test_head_dim_128(rlx, kind, window, theta):
    """The head size of the larger decoder families: same kernel, one CTA per SM."""
    for gain in (1.0, 3.0):
        _run_case(rlx, [1, 17, 64, 65, 129, 300, 700], 2, 128, kind, window, theta, gain, seed=128 + kind + window)


def test_empty_sequences_and_a_long_one(rlx):
    """Zero-length sequences write nothing; an 8,192-row sequence exercises 64 query tiles and, with a
    window, the skipping of leading key blocks far from the diagonal."""
    rng = np.random.default_rng(77)
    h, d = 1, 32
    H = h * d
    lengths = [0, 8192, 0, 5]
    total = sum(lengths)
    qkv = rand_bf16(rng, (total, 3 * H))
    qkv[:, :H] = round_to_bf16(qkv[:, :H] * np.float32(2.0))
    start = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    for kind, w in ((CAUSAL, 0), (SLIDING, 300)):
        got = to_np64(rlx.attention_kind_bf16(bf16_dev(qkv), i32_dev(start[:-1]), i32_dev(np.array(lengths)), max(lengths), h,
                                              kind, w))
        ref = ak.attention_packed(qkv.astype(np.float64), start[:-1], lengths, h, kind, w)
        vmax = float(np.abs(qkv[:, 2 * H:]).max())
        assert np.abs(got - ref).max() <= 2 * BF16_U * (vmax + np.abs(ref).max())
