"""Pins for the fp64 oracle of attention under the Causal / SlidingWindow mask kinds and rotary
position embedding (Section 3.1 mask kinds, Section 3.2 fused QK-RoPE): closed forms, invariants,
brute force on tiny inputs and library routines.  No GPU."""
import math

import numpy as np
import pytest
import torch

from oracle import attention_kinds as ak
from oracle import encoder_np


def _rand_qkv(rng, L, h, d, scale=1.0):
    return rng.standard_normal((L, 3 * h * d)) * scale


# ---------------------------------------------------------------- brute force on tiny inputs
def _brute(qkv, h, kind, w, theta):
    """Scalar loops, no max subtraction, explicit visibility test and per-pair rotation."""
    L, H3 = qkv.shape
    H = H3 // 3
    d = H // h
    half = d // 2

    def rot(vec, pos):
        out = list(vec)
        for j in range(half):
            a = pos * theta ** (-2.0 * j / d)
            out[j] = vec[j] * math.cos(a) - vec[j + half] * math.sin(a)
            out[j + half] = vec[j + half] * math.cos(a) + vec[j] * math.sin(a)
        return out

    ctx = np.zeros((L, H))
    for head in range(h):
        qs = [[qkv[i, head * d + c] for c in range(d)] for i in range(L)]
        ks = [[qkv[i, H + head * d + c] for c in range(d)] for i in range(L)]
        if theta is not None:
            qs = [rot(qs[i], i) for i in range(L)]
            ks = [rot(ks[i], i) for i in range(L)]
        for i in range(L):
            num = [0.0] * d
            den = 0.0
            for k in range(L):
                if kind == ak.KIND_CAUSAL and not k <= i:
                    continue
                if kind == ak.KIND_SLIDING and not (k <= i and k > i - w):
                    continue
                e = math.exp(sum(qs[i][c] * ks[k][c] for c in range(d)) / math.sqrt(d))
                den += e
                for c in range(d):
                    num[c] += e * qkv[k, 2 * H + head * d + c]
            for c in range(d):
                ctx[i, head * d + c] = num[c] / den
    return ctx


@pytest.mark.parametrize("kind,w", [(ak.KIND_NONE, 0), (ak.KIND_CAUSAL, 0), (ak.KIND_SLIDING, 1),
                                    (ak.KIND_SLIDING, 3), (ak.KIND_SLIDING, 50)])
@pytest.mark.parametrize("theta", [None, 10000.0, 100.0])
def test_brute_force_tiny(kind, w, theta):
    rng = np.random.default_rng(5)
    for L, h, d in [(1, 1, 2), (7, 2, 4), (5, 1, 6)]:
        qkv = _rand_qkv(rng, L, h, d)
        got = ak.attention_one(qkv, h, kind, w, theta)
        np.testing.assert_allclose(got, _brute(qkv, h, kind, w, theta), rtol=1e-12, atol=1e-14)


# ---------------------------------------------------------------- mask kinds: closed forms, invariants
def test_kind_none_is_the_encoder_attention_with_a_full_mask():
    rng = np.random.default_rng(0)
    L, h, d = 19, 3, 8
    qkv = _rand_qkv(rng, L, h, d)
    ref = encoder_np.attention(qkv[None], np.ones((1, L), np.int32), h)[0]
    np.testing.assert_allclose(ak.attention_one(qkv, h, ak.KIND_NONE), ref, rtol=1e-13, atol=1e-15)


def test_causal_first_row_and_no_lookahead():
    rng = np.random.default_rng(1)
    L, h, d = 23, 2, 8
    qkv = _rand_qkv(rng, L, h, d, 2.0)
    H = h * d
    out = ak.attention_one(qkv, h, ak.KIND_CAUSAL)
    np.testing.assert_allclose(out[0], qkv[0, 2 * H:], rtol=0, atol=1e-15)   # row 0 sees only itself
    # rows <= i do not depend on anything after i: bitwise
    cut = 11
    pert = qkv.copy()
    pert[cut + 1:] = rng.standard_normal(pert[cut + 1:].shape)
    out2 = ak.attention_one(pert, h, ak.KIND_CAUSAL)
    assert np.array_equal(out[:cut + 1], out2[:cut + 1])
    assert not np.allclose(out[cut + 1:], out2[cut + 1:])


def test_uniform_scores_give_running_and_moving_means():
    rng = np.random.default_rng(2)
    L, h, d = 17, 2, 4
    H = h * d
    qkv = _rand_qkv(rng, L, h, d)
    qkv[:, :H] = 0.0                                  # q = 0: every visible key gets the same weight
    v = qkv[:, 2 * H:]
    causal = ak.attention_one(qkv, h, ak.KIND_CAUSAL)
    np.testing.assert_allclose(causal, np.cumsum(v, 0) / np.arange(1, L + 1)[:, None], rtol=1e-13, atol=1e-15)
    w = 4
    sw = ak.attention_one(qkv, h, ak.KIND_SLIDING, w)
    ref = np.stack([v[max(0, i - w + 1):i + 1].mean(0) for i in range(L)])
    np.testing.assert_allclose(sw, ref, rtol=1e-13, atol=1e-15)


def test_sliding_window_limits_and_locality():
    rng = np.random.default_rng(3)
    L, h, d = 21, 2, 8
    H = h * d
    qkv = _rand_qkv(rng, L, h, d, 2.0)
    # w = 1: only the query's own position -> ctx = v exactly
    np.testing.assert_allclose(ak.attention_one(qkv, h, ak.KIND_SLIDING, 1), qkv[:, 2 * H:], rtol=0, atol=1e-15)
    # w >= L: the window never cuts -> identical to causal
    assert np.array_equal(ak.attention_one(qkv, h, ak.KIND_SLIDING, L), ak.attention_one(qkv, h, ak.KIND_CAUSAL))
    assert np.array_equal(ak.attention_one(qkv, h, ak.KIND_SLIDING, 10 * L), ak.attention_one(qkv, h, ak.KIND_CAUSAL))
    # locality: row i reads keys i-w+1 .. i and nothing else
    w, kpos = 5, 7
    out = ak.attention_one(qkv, h, ak.KIND_SLIDING, w)
    pert = qkv.copy()
    pert[kpos, H:] += 1.0                             # change key and value at position kpos
    out2 = ak.attention_one(pert, h, ak.KIND_SLIDING, w)
    changed = np.any(out != out2, axis=1)
    assert list(np.nonzero(changed)[0]) == list(range(kpos, kpos + w))
    with pytest.raises(ValueError):
        ak.visible(4, ak.KIND_SLIDING, 0)


def test_visibility_counts():
    L, w = 13, 4
    assert ak.visible(L, ak.KIND_NONE).sum() == L * L
    assert ak.visible(L, ak.KIND_CAUSAL).sum() == L * (L + 1) // 2
    assert list(ak.visible(L, ak.KIND_SLIDING, w).sum(1)) == [min(i + 1, w) for i in range(L)]


@pytest.mark.parametrize("kind,w", [(ak.KIND_CAUSAL, 0), (ak.KIND_SLIDING, 6)])
def test_against_library_sdpa(kind, w):
    rng = np.random.default_rng(4)
    L, h, d = 33, 4, 16
    H = h * d
    qkv = _rand_qkv(rng, L, h, d, 1.5)
    t = torch.from_numpy(qkv).view(L, 3, h, d)
    q, k, v = (t[:, i].transpose(0, 1)[None] for i in range(3))          # [1, h, L, d]
    if kind == ak.KIND_CAUSAL:
        ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True)
    else:
        band = torch.ones(L, L, dtype=torch.bool).tril().triu(-(w - 1))  # library-built band matrix
        ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=band)
    ref = ref[0].transpose(0, 1).reshape(L, H).numpy()
    np.testing.assert_allclose(ak.attention_one(qkv, h, kind, w), ref, rtol=1e-12, atol=1e-14)


def test_heads_are_independent_and_packed_sequences_do_not_mix():
    rng = np.random.default_rng(6)
    h, d = 3, 8
    H = h * d
    lens = [5, 1, 12]
    start = np.concatenate([[0], np.cumsum(lens)])[:-1]
    qkv = _rand_qkv(rng, sum(lens) + 2, h, d)           # two trailing rows belong to no sequence
    out = ak.attention_packed(qkv, start, lens, h, ak.KIND_CAUSAL, 0, 10000.0)
    assert np.all(out[sum(lens):] == 0.0)
    for s0, n in zip(start, lens):
        np.testing.assert_array_equal(out[s0:s0 + n], ak.attention_one(qkv[s0:s0 + n], h, ak.KIND_CAUSAL, 0, 10000.0))
    pert = qkv.copy()
    pert[:, 0:d] += 0.5                                  # head 0's q columns only
    out2 = ak.attention_packed(pert, start, lens, h, ak.KIND_CAUSAL, 0, 10000.0)
    assert np.array_equal(out[:, d:], out2[:, d:]) and not np.array_equal(out[:, :d], out2[:, :d])


# ---------------------------------------------------------------- rotary embedding
def test_rope_closed_forms():
    # d = 2: one pair, angle = pos * theta^0 = pos radians
    x = np.zeros((5, 1, 2))
    x[:, 0, 0] = 1.0
    r = ak.rope(x, 10000.0)
    np.testing.assert_allclose(r[:, 0, 0], np.cos(np.arange(5.0)), rtol=0, atol=1e-15)
    np.testing.assert_allclose(r[:, 0, 1], np.sin(np.arange(5.0)), rtol=0, atol=1e-15)
    # d = 4: second pair turns by pos * theta^(-1/2)
    y = np.zeros((3, 1, 4))
    y[:, 0, 1] = 1.0
    r = ak.rope(y, 100.0)
    np.testing.assert_allclose(r[:, 0, 1], np.cos(np.arange(3.0) / 10.0), rtol=0, atol=1e-15)
    np.testing.assert_allclose(r[:, 0, 3], np.sin(np.arange(3.0) / 10.0), rtol=0, atol=1e-15)
    # position 0 is the identity; v-like tensors are never touched by attention_one (checked below)
    z = np.random.default_rng(0).standard_normal((1, 2, 8))
    assert np.array_equal(ak.rope(z), z)


def test_rope_is_a_rotation_and_relative():
    rng = np.random.default_rng(7)
    L, h, d = 12, 2, 16
    q = rng.standard_normal((L, h, d))
    k = rng.standard_normal((L, h, d))
    rq, rk = ak.rope(q), ak.rope(k)
    half = d // 2
    # each (j, j + d/2) pair keeps its length
    np.testing.assert_allclose(rq[..., :half] ** 2 + rq[..., half:] ** 2, q[..., :half] ** 2 + q[..., half:] ** 2,
                               rtol=1e-13)
    # scores depend on the position difference only: shift every position by a constant
    pos = np.arange(L, dtype=np.float64)
    s0 = np.einsum("ihc,khc->hik", rq, rk)
    s1 = np.einsum("ihc,khc->hik", ak.rope(q, positions=pos + 37.0), ak.rope(k, positions=pos + 37.0))
    np.testing.assert_allclose(s0, s1, rtol=0, atol=1e-12)
    # and they do change when only one side moves
    s2 = np.einsum("ihc,khc->hik", ak.rope(q, positions=pos + 1.0), rk)
    assert not np.allclose(s0, s2)


def test_rope_matches_library_rotate_half_convention():
    from transformers import LlamaConfig
    from transformers.models.llama.modeling_llama import LlamaRotaryEmbedding, apply_rotary_pos_emb

    rng = np.random.default_rng(8)
    L, h, d = 9, 2, 16
    q = rng.standard_normal((L, h, d))
    k = rng.standard_normal((L, h, d))
    cfg = LlamaConfig(hidden_size=h * d, num_attention_heads=h, num_hidden_layers=1, intermediate_size=32,
                      vocab_size=8, max_position_embeddings=64)
    emb = LlamaRotaryEmbedding(cfg)
    tq = torch.from_numpy(q).transpose(0, 1)[None]      # [1, h, L, d]
    tk = torch.from_numpy(k).transpose(0, 1)[None]
    cos, sin = emb(tq, torch.arange(L)[None])           # library angles (fp32 inverse frequencies)
    lq, lk = apply_rotary_pos_emb(tq, tk, cos.double(), sin.double())
    theta = float(getattr(cfg, "rope_theta", None) or cfg.rope_parameters["rope_theta"])
    np.testing.assert_allclose(ak.rope(q, theta), lq[0].transpose(0, 1).numpy(), rtol=0, atol=2e-6)
    np.testing.assert_allclose(ak.rope(k, theta), lk[0].transpose(0, 1).numpy(), rtol=0, atol=2e-6)
    # the pairing itself, with exact fp64 angles in the library's [L, d] layout: agreement to rounding
    inv = theta ** (-2.0 * np.arange(d // 2) / d)
    ang = np.arange(L)[:, None] * inv[None, :]
    c64 = torch.from_numpy(np.concatenate([np.cos(ang), np.cos(ang)], 1))[None]
    s64 = torch.from_numpy(np.concatenate([np.sin(ang), np.sin(ang)], 1))[None]
    lq, lk = apply_rotary_pos_emb(tq, tk, c64, s64)
    np.testing.assert_allclose(ak.rope(q, theta), lq[0].transpose(0, 1).numpy(), rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(ak.rope(k, theta), lk[0].transpose(0, 1).numpy(), rtol=1e-13, atol=1e-15)


def test_rope_leaves_values_alone_and_changes_attention():
    rng = np.random.default_rng(9)
    L, h, d = 10, 2, 8
    H = h * d
    qkv = _rand_qkv(rng, L, h, d)
    qkv[:, :H] = 0.0                                     # uniform weights: output is a mean of raw v rows
    out = ak.attention_one(qkv, h, ak.KIND_CAUSAL, 0, 10000.0)
    np.testing.assert_allclose(out, np.cumsum(qkv[:, 2 * H:], 0) / np.arange(1, L + 1)[:, None], rtol=1e-13)
    qkv = _rand_qkv(rng, L, h, d, 2.0)
    assert not np.allclose(ak.attention_one(qkv, h, ak.KIND_CAUSAL, 0, 10000.0),
                           ak.attention_one(qkv, h, ak.KIND_CAUSAL, 0, None))


def test_rope_qk_packed_composes_with_attention():
    """Rotating q,k first and then attending without rotation is the rotary attention; v, and rows that
    belong to no sequence, pass through untouched."""
    rng = np.random.default_rng(10)
    h, d = 2, 8
    H = h * d
    lens = [6, 1, 9]
    start = np.concatenate([[0], np.cumsum(lens)])[:-1]
    qkv = _rand_qkv(rng, sum(lens) + 3, h, d)
    rot = ak.rope_qk_packed(qkv, start, lens, h, 10000.0)
    assert np.array_equal(rot[:, 2 * H:], qkv[:, 2 * H:]) and np.array_equal(rot[sum(lens):], qkv[sum(lens):])
    assert np.array_equal(rot[start], qkv[start])                  # position 0 of every sequence: identity
    a = ak.attention_packed(rot, start, lens, h, ak.KIND_CAUSAL, 0, None)
    b = ak.attention_packed(qkv, start, lens, h, ak.KIND_CAUSAL, 0, 10000.0)
    np.testing.assert_allclose(a, b, rtol=1e-13, atol=1e-15)


# ---------------------------------------------------------------- grouped-query layout
def test_grouped_query_equals_repeated_kv_heads_and_library():
    rng = np.random.default_rng(11)
    L, hq, hkv, d = 21, 6, 2, 8
    qkv = rng.standard_normal((L, (hq + 2 * hkv) * d)) * 1.5
    got = ak.attention_one(qkv, hq, ak.KIND_CAUSAL, 0, 10000.0, num_kv_heads=hkv)
    # the same thing with every k/v head written out once per q head of its group (plain multi-head layout)
    q, k, v = ak.split_qkv(qkv, hq, hkv)
    full = np.concatenate([q.reshape(L, -1), np.repeat(k, hq // hkv, axis=1).reshape(L, -1),
                           np.repeat(v, hq // hkv, axis=1).reshape(L, -1)], axis=1)
    np.testing.assert_allclose(got, ak.attention_one(full, hq, ak.KIND_CAUSAL, 0, 10000.0), rtol=1e-13, atol=1e-15)
    # library routine with its own grouped-query switch (no rotation)
    tq = torch.from_numpy(q).transpose(0, 1)[None]
    tk = torch.from_numpy(k).transpose(0, 1)[None]
    tv = torch.from_numpy(v).transpose(0, 1)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, enable_gqa=True)
    ref = ref[0].transpose(0, 1).reshape(L, hq * d).numpy()
    np.testing.assert_allclose(ak.attention_one(qkv, hq, ak.KIND_CAUSAL, 0, None, num_kv_heads=hkv), ref,
                               rtol=1e-12, atol=1e-14)
    # perturbing one k/v head reaches exactly the q heads of its group
    pert = qkv.copy()
    pert[:, (hq + 1) * d:(hq + 2) * d] += 0.25                      # k head 1
    out2 = ak.attention_one(pert, hq, ak.KIND_CAUSAL, 0, 10000.0, num_kv_heads=hkv)
    changed = [bool(np.any(got[:, j * d:(j + 1) * d] != out2[:, j * d:(j + 1) * d])) for j in range(hq)]
    assert changed == [False, False, False, True, True, True]
    # the packed rotation touches q and k heads only
    rot = ak.rope_qk_packed(qkv, [0], [L], hq, 10000.0, num_kv_heads=hkv)
    assert np.array_equal(rot[:, (hq + hkv) * d:], qkv[:, (hq + hkv) * d:]) and not np.allclose(rot[1:, :hq * d], qkv[1:, :hq * d])
