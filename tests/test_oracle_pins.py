"""Pins for the fp64 oracle: closed forms, brute force, invariants and library
cross-checks chosen so that a dropped term, a wrong sign/index or a transposed
operand in ``oracle/`` fails at least one of them.  CPU only."""
import math
from dataclasses import replace

import numpy as np
import pytest

from oracle import encoder_np, oracle
from synth.inputs import CONFIGS, EncoderConfig, make_inputs

TINY = EncoderConfig("tiny", 2, 64, 4, 128, 3, 12, 1, 12, 7, vocab=97, max_pos=32)


def tiny_inputs(**kw):
    return make_inputs(TINY, **kw)


# ----------------------------------------------------------------- LayerNorm
def test_ln_closed_forms():
    rng = np.random.default_rng(0)
    H = 48
    v = rng.standard_normal((5, H)) * 3 + 2
    eps = 1e-3
    out = oracle.layernorm(v, np.ones(H), np.zeros(H), eps)
    var = v.var(axis=1)  # biased
    assert np.allclose(out.mean(axis=1), 0, atol=1e-14)
    assert np.allclose(out.var(axis=1), var / (var + eps), rtol=1e-12)
    # an unbiased variance (divide by H-1) would fail the line above
    assert not np.allclose(out.var(axis=1), v.var(axis=1, ddof=1) / (v.var(axis=1, ddof=1) + eps), rtol=1e-6)


def test_ln_constant_row_gives_beta_and_eps_inside_sqrt():
    H = 16
    beta = np.linspace(-1, 1, H).astype(np.float32)
    gamma = np.full(H, 3.0, np.float32)
    out = oracle.layernorm(np.full((1, H), 5.0), gamma, beta, 1e-12)
    assert np.array_equal(out[0], beta.astype(np.float64))
    # eps inside the sqrt: a row with variance s2 scales by 1/sqrt(s2+eps), not 1/(sqrt(s2)+eps)
    v = np.array([[1.0, -1.0]])
    o = oracle.layernorm(v, np.ones(2), np.zeros(2), 3.0)
    assert np.allclose(o, [[0.5, -0.5]], rtol=1e-15)


def test_ln_affine_and_invariance():
    rng = np.random.default_rng(1)
    H = 32
    v = rng.standard_normal((4, H))
    g = rng.standard_normal(H).astype(np.float32)
    b = rng.standard_normal(H).astype(np.float32)
    base = oracle.layernorm(v, np.ones(H), np.zeros(H), 1e-12)
    assert np.allclose(oracle.layernorm(v, g, b, 1e-12), base * g + b, rtol=1e-13, atol=1e-13)
    assert np.allclose(oracle.layernorm(7.5 * v + 3.0, np.ones(H), np.zeros(H), 1e-12), base, atol=1e-10)
    assert np.allclose(oracle.layernorm(base, np.ones(H), np.zeros(H), 1e-12), base, atol=1e-10)


# -------------------------------------------------------------------- Linear
def test_linear_matches_library_matmul_and_identity():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((7, 24))
    w = rng.standard_normal((10, 24)).astype(np.float32)
    b = rng.standard_normal(10).astype(np.float32)
    ref = x @ w.astype(np.float64).T + b
    assert np.allclose(oracle.linear(x, w, b), ref, rtol=1e-12, atol=1e-13)
    assert np.allclose(oracle.linear(x, w), ref - b, rtol=1e-12, atol=1e-13)
    # a transposed weight read ([in,out]) cannot pass a non-square case; identity passes through
    assert np.allclose(oracle.linear(x, np.eye(24, dtype=np.float32)), x)
    one = np.zeros((3, 24), np.float32)
    one[2, 5] = 1.0  # output 2 picks input 5
    assert np.allclose(oracle.linear(x, one)[:, 2], x[:, 5])


# ---------------------------------------------------------------------- GELU
def test_gelu_closed_forms():
    assert oracle.gelu(np.array([0.0]))[0] == 0.0
    # gelu(1) = Phi(1), standard normal CDF at 1 (tables: 0.841344746068543)
    assert abs(oracle.gelu(np.array([1.0]))[0] - 0.841344746068543) < 1e-15
    u = np.linspace(-6, 6, 101)
    g = oracle.gelu(u)
    assert np.allclose(g - oracle.gelu(-u), u, atol=1e-14)  # odd part is u/2 - (-u/2)
    assert abs(oracle.gelu(np.array([12.0]))[0] - 12.0) < 1e-12
    assert -1e-12 < oracle.gelu(np.array([-12.0]))[0] <= 0.0
    # the tanh approximation differs by > 1e-4 somewhere: make sure we are not it
    t = 0.5 * u * (1 + np.tanh(math.sqrt(2 / math.pi) * (u + 0.044715 * u ** 3)))
    assert np.abs(g - t).max() > 1e-4
    from scipy.stats import norm
    assert np.allclose(g, u * norm.cdf(u), atol=1e-15)


# ----------------------------------------------------------------- Attention
def _brute_attention(qkv, mask, h):
    """Naive python loops, no max subtraction, straight from the definition."""
    B, S, H3 = qkv.shape
    H = H3 // 3
    d = H // h
    out = np.zeros((B, S, H))
    for b in range(B):
        for j in range(h):
            for i in range(S):
                num = [0.0] * d
                den = 0.0
                for k in range(S):
                    if mask[b, k] == 0:
                        continue
                    s = sum(qkv[b, i, j * d + c] * qkv[b, k, H + j * d + c] for c in range(d)) / math.sqrt(d)
                    e = math.exp(s)
                    den += e
                    for c in range(d):
                        num[c] += e * qkv[b, k, 2 * H + j * d + c]
                for c in range(d):
                    out[b, i, j * d + c] = num[c] / den
    return out


def test_attention_brute_force_tiny():
    rng = np.random.default_rng(3)
    B, S, h, d = 2, 7, 2, 4
    qkv = rng.standard_normal((B, S, 3 * h * d))
    mask = np.array([[1, 1, 1, 0, 1, 0, 0], [1, 1, 1, 1, 1, 1, 1]], np.int32)  # holes too
    ref = _brute_attention(qkv, mask, h)
    got = oracle.attention(qkv, mask, h, compute_all_rows=True)
    assert np.allclose(got, ref, rtol=1e-12, atol=1e-13)
    assert np.allclose(encoder_np.attention(qkv, mask, h), ref, rtol=1e-12, atol=1e-13)
    # rows skipped when their own mask is 0
    skipped = oracle.attention(qkv, mask, h, compute_all_rows=False)
    assert np.array_equal(skipped[0, 3], np.zeros(h * d)) and np.allclose(skipped[0, 4], ref[0, 4])


def test_attention_softmax_rows_sum_to_one_and_masked_probs_zero():
    rng = np.random.default_rng(4)
    B, S, h, d = 3, 19, 3, 8
    qkv = rng.standard_normal((B, S, 3 * h * d)) * 4
    mask = (rng.random((B, S)) < 0.7).astype(np.int32)
    mask[:, 0] = 1
    _, p = oracle.attention(qkv, mask, h, return_probs=True)
    assert np.allclose(p.sum(-1), 1.0, atol=1e-15)
    assert np.all(p[np.broadcast_to((mask == 0)[:, None, None, :], p.shape)] == 0.0)
    assert np.all(p >= 0)


def test_attention_uniform_scores_give_masked_mean_of_v():
    rng = np.random.default_rng(5)
    B, S, h, d = 2, 9, 2, 4
    H = h * d
    qkv = rng.standard_normal((B, S, 3 * H))
    qkv[..., :H] = 0.0  # q = 0 -> all scores equal
    mask = np.array([[1] * 5 + [0] * 4, [1] * 9], np.int32)
    got = oracle.attention(qkv, mask, h)
    for b in range(B):
        mean_v = qkv[b, mask[b] != 0, 2 * H:].mean(axis=0)
        assert np.allclose(got[b], mean_v[None, :], atol=1e-14)


def test_attention_single_valid_key_returns_its_value():
    rng = np.random.default_rng(6)
    S, h, d = 6, 2, 4
    H = h * d
    qkv = rng.standard_normal((1, S, 3 * H)) * 10
    mask = np.zeros((1, S), np.int32)
    mask[0, 2] = 1
    got = oracle.attention(qkv, mask, h)
    assert np.allclose(got[0], qkv[0, 2, 2 * H:][None, :], atol=1e-14)
    # no valid key at all -> zeros
    assert np.array_equal(oracle.attention(qkv, np.zeros((1, S), np.int32), h), np.zeros((1, S, H)))


def test_attention_scale_is_inverse_sqrt_d():
    # two keys, d=4: q.k = 4a vs 0  ->  p0 = sigmoid(4a/sqrt(4)) = sigmoid(2a)
    a = 0.7
    H = 4
    qkv = np.zeros((1, 2, 3 * H))
    qkv[0, :, :H] = 1.0          # q = ones
    qkv[0, 0, H:2 * H] = a       # k0 = a*ones -> q.k0 = 4a ; k1 = 0
    qkv[0, 0, 2 * H:] = 1.0      # v0 = 1, v1 = 0  -> ctx = p0
    got = oracle.attention(qkv, np.ones((1, 2), np.int32), 1)
    assert np.allclose(got[0, 0], 1 / (1 + math.exp(-2 * a)), rtol=1e-14)


def test_attention_large_logits_are_stable_and_shift_invariant():
    rng = np.random.default_rng(7)
    S, h, d = 8, 1, 4
    qkv = rng.standard_normal((1, S, 3 * d))
    qkv[0, :, :d] *= 300.0  # logits of several hundreds: exp would overflow without the max shift
    got = oracle.attention(qkv, np.ones((1, S), np.int32), h)
    assert np.all(np.isfinite(got))
    # adding the same vector to every key shifts each row's scores by a constant: no change
    shifted = qkv.copy()
    shifted[0, :, d:2 * d] += np.array([0.3, -0.2, 0.1, 0.05])
    qkv[0, :, :d] /= 300.0
    shifted[0, :, :d] /= 300.0
    assert np.allclose(oracle.attention(qkv, np.ones((1, S), np.int32), h),
                       oracle.attention(shifted, np.ones((1, S), np.int32), h), atol=1e-13)


def test_attention_heads_are_independent():
    rng = np.random.default_rng(8)
    B, S, h, d = 1, 5, 3, 4
    H = h * d
    qkv = rng.standard_normal((B, S, 3 * H))
    base = oracle.attention(qkv, np.ones((B, S), np.int32), h)
    pert = qkv.copy()
    pert[..., d:2 * d] += 1.0           # head 1's q
    pert[..., H + d:H + 2 * d] -= 0.5   # head 1's k
    got = oracle.attention(pert, np.ones((B, S), np.int32), h)
    assert np.array_equal(got[..., :d], base[..., :d]) and np.array_equal(got[..., 2 * d:], base[..., 2 * d:])
    assert not np.allclose(got[..., d:2 * d], base[..., d:2 * d])


def test_attention_matches_torch_sdpa_fp64():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(9)
    B, S, h, d = 2, 11, 3, 8
    H = h * d
    qkv = rng.standard_normal((B, S, 3 * H))
    mask = np.array([[1] * 6 + [0] * 5, [1] * 11], np.int32)
    t = torch.from_numpy(qkv).view(B, S, 3, h, d).permute(2, 0, 3, 1, 4)  # [3,B,h,S,d]
    keep = torch.from_numpy(mask != 0)[:, None, None, :]
    ref = torch.nn.functional.scaled_dot_product_attention(t[0], t[1], t[2], attn_mask=keep)
    ref = ref.permute(0, 2, 1, 3).reshape(B, S, H).numpy()
    got = oracle.attention(qkv, mask, h)
    assert np.allclose(got, ref, rtol=1e-12, atol=1e-13)


# ------------------------------------------------------------------- Pooling
def test_pool_closed_forms():
    rng = np.random.default_rng(10)
    B, S, H = 3, 6, 10
    x = rng.standard_normal((B, S, H))
    mask = np.array([[1, 1, 1, 0, 0, 0], [0, 0, 1, 0, 0, 0], [0] * 6], np.int32)
    out = oracle.pool_l2(x, mask)
    m0 = x[0, :3].mean(0)
    assert np.allclose(out[0], m0 / np.linalg.norm(m0), rtol=1e-14)
    assert np.allclose(out[1], x[1, 2] / np.linalg.norm(x[1, 2]), rtol=1e-14)   # single token
    assert np.array_equal(out[2], np.zeros(H))                                   # empty sequence -> zeros
    assert np.allclose(np.linalg.norm(out[:2], axis=1), 1.0, atol=1e-15)
    assert np.allclose(oracle.pool_l2(3.7 * x, mask), out, atol=1e-14)           # scale invariance


# ------------------------------------------------------------- Whole encoder
def test_two_independent_oracles_agree():
    for kw in ({}, {"qk_gain": 8.0, "ln_affine_random": True}, {"mask_holes": 0.3}):
        inp = tiny_inputs(**kw)
        a = oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers)
        b = encoder_np.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers)
        keep = inp.lengths > 0
        assert np.abs(a - b)[keep].max() < 1e-12
        assert np.allclose(np.linalg.norm(a[keep], axis=1), 1.0, atol=1e-14)


def test_all_rows_switch_does_not_change_output():
    inp = tiny_inputs(mask_holes=0.2)
    a = oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers, compute_all_rows=False)
    b, dumps = oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers,
                                      compute_all_rows=True, dumps=True)
    assert np.abs(a - b).max() < 1e-14
    assert dumps["qkv"].shape == (TINY.num_layers, TINY.batch, TINY.seq, 3 * TINY.hidden)


def test_padding_invariance_is_bitwise():
    inp = tiny_inputs()
    base = oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers)
    ids2 = inp.ids.copy()
    ids2[inp.mask == 0] = (ids2[inp.mask == 0] + 13) % TINY.vocab
    assert (inp.mask == 0).any()
    again = oracle.encoder_forward(inp.cfg, ids2, inp.mask, inp.params, inp.layers)
    assert np.array_equal(base, again)
    all_rows = oracle.encoder_forward(inp.cfg, ids2, inp.mask, inp.params, inp.layers, compute_all_rows=True)
    assert np.array_equal(base, all_rows) or np.abs(base - all_rows).max() < 1e-15


def test_padding_length_invariance():
    short = make_inputs(TINY, batch=2, seq=8, lengths=[5, 8])
    long_ = make_inputs(TINY, batch=2, seq=24, lengths=[5, 8], weights=False)
    long_.ids[:, :8] = short.ids   # same tokens, more padding, same parameters
    a = oracle.encoder_forward(short.cfg, short.ids, short.mask, short.params, short.layers)
    b = oracle.encoder_forward(long_.cfg, long_.ids, long_.mask, short.params, short.layers)
    assert np.abs(a - b).max() < 1e-14


def test_without_positions_holes_equal_compaction_and_permutation():
    inp = make_inputs(TINY, batch=1, seq=10, lengths=[10])
    inp.params["pos_emb"] = np.zeros_like(inp.params["pos_emb"])
    mask = np.array([[1, 0, 1, 1, 0, 0, 1, 1, 0, 1]], np.int32)
    holed = oracle.encoder_forward(inp.cfg, inp.ids, mask, inp.params, inp.layers)
    valid = inp.ids[0, mask[0] != 0]
    perm = np.random.default_rng(0).permutation(len(valid))
    compact_ids = np.zeros((1, 10), np.int32)
    compact_ids[0, :len(valid)] = valid[perm]
    compact_mask = (np.arange(10)[None, :] < len(valid)).astype(np.int32)
    compact = oracle.encoder_forward(inp.cfg, compact_ids, compact_mask, inp.params, inp.layers)
    assert np.abs(holed - compact).max() < 1e-13
    # with positions switched back on the order matters (positions really are added)
    full = make_inputs(TINY, batch=1, seq=10, lengths=[10])
    moved = oracle.encoder_forward(full.cfg, compact_ids, compact_mask, full.params, full.layers)
    assert np.abs(moved - compact).max() > 1e-6


def test_zero_linear_weights_closed_form():
    inp = tiny_inputs(ln_affine_random=True)
    for lw in inp.layers:
        for k in ("wqkv", "bqkv", "wo", "bo", "w1", "b1", "w2", "b2"):
            lw[k] = np.zeros_like(lw[k])
    out = oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers)
    # every sub-layer reduces to x <- LN(x), written here with numpy only
    p = inp.params
    e = (p["word_emb"].astype(np.float64)[inp.ids] + p["pos_emb"].astype(np.float64)[None, :TINY.seq]
         + p["type_emb"].astype(np.float64)[0])

    def ln(v, g, b):
        return (v - v.mean(-1, keepdims=True)) / np.sqrt(v.var(-1, keepdims=True) + TINY.ln_eps) * g + b

    x = ln(e, p["emb_ln_g"].astype(np.float64), p["emb_ln_b"].astype(np.float64))
    for lw in inp.layers:
        x = ln(x, lw["ln1_g"].astype(np.float64), lw["ln1_b"].astype(np.float64))
        x = ln(x, lw["ln2_g"].astype(np.float64), lw["ln2_b"].astype(np.float64))
    m = (inp.mask != 0)[..., None]
    pool = (x * m).sum(1) / m.sum(1)
    ref = pool / np.linalg.norm(pool, axis=1, keepdims=True)
    assert np.abs(out - ref).max() < 1e-12


def test_batch_independence_and_permutation():
    inp = tiny_inputs()
    out = oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers)
    perm = np.array([2, 0, 1])
    outp = oracle.encoder_forward(inp.cfg, inp.ids[perm], inp.mask[perm], inp.params, inp.layers)
    assert np.array_equal(outp, out[perm])
    solo = oracle.encoder_forward(replace(inp.cfg, batch=1), inp.ids[1:2], inp.mask[1:2], inp.params, inp.layers)
    assert np.array_equal(solo[0], out[1])


def test_type_embedding_and_bias_terms_are_present():
    inp = tiny_inputs()
    base = oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers)
    for name in ("type_emb", "pos_emb", "word_emb"):
        saved = inp.params[name]
        inp.params[name] = np.zeros_like(saved)
        assert np.abs(oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers) - base).max() > 1e-6
        inp.params[name] = saved
    for name in ("bqkv", "bo", "b1", "b2"):
        saved = inp.layers[0][name]
        inp.layers[0][name] = np.zeros_like(saved)
        assert np.abs(oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers) - base).max() > 1e-7
        inp.layers[0][name] = saved
    # row 1 of the type table is never read (the interface has no type ids)
    inp.params["type_emb"] = inp.params["type_emb"].copy()
    inp.params["type_emb"][1] += 1.0
    assert np.array_equal(oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers), base)


def test_whole_encoder_matches_library_bert_fp64():
    """Reduce the encoder to a library routine: a randomly initialised BertModel
    (post-LN, erf-GELU, eps 1e-12, absolute positions) in fp64 with our weights."""
    torch = pytest.importorskip("torch")
    transformers = pytest.importorskip("transformers")
    inp = tiny_inputs(qk_gain=4.0, ln_affine_random=True)
    c = inp.cfg
    bc = transformers.BertConfig(
        vocab_size=c.vocab, hidden_size=c.hidden, num_hidden_layers=c.num_layers,
        num_attention_heads=c.num_heads, intermediate_size=c.ffn, hidden_act="gelu",
        hidden_dropout_prob=0.0, attention_probs_dropout_prob=0.0, max_position_embeddings=c.max_pos,
        type_vocab_size=c.type_vocab, layer_norm_eps=c.ln_eps)
    try:
        bc._attn_implementation = "eager"
    except Exception:
        pass
    model = transformers.BertModel(bc, add_pooling_layer=False).double().eval()
    t = lambda a: torch.from_numpy(np.asarray(a, np.float64))
    sd = model.state_dict()
    H = c.hidden

    def put(name, val):
        assert name in sd and tuple(sd[name].shape) == tuple(val.shape), name
        sd[name].copy_(t(val))

    with torch.no_grad():
        p = inp.params
        put("embeddings.word_embeddings.weight", p["word_emb"])
        put("embeddings.position_embeddings.weight", p["pos_emb"])
        put("embeddings.token_type_embeddings.weight", p["type_emb"])
        put("embeddings.LayerNorm.weight", p["emb_ln_g"])
        put("embeddings.LayerNorm.bias", p["emb_ln_b"])
        for i, lw in enumerate(inp.layers):
            pre = f"encoder.layer.{i}."
            for j, nm in enumerate(("query", "key", "value")):
                put(pre + f"attention.self.{nm}.weight", lw["wqkv"][j * H:(j + 1) * H])
                put(pre + f"attention.self.{nm}.bias", lw["bqkv"][j * H:(j + 1) * H])
            put(pre + "attention.output.dense.weight", lw["wo"])
            put(pre + "attention.output.dense.bias", lw["bo"])
            put(pre + "attention.output.LayerNorm.weight", lw["ln1_g"])
            put(pre + "attention.output.LayerNorm.bias", lw["ln1_b"])
            put(pre + "intermediate.dense.weight", lw["w1"])
            put(pre + "intermediate.dense.bias", lw["b1"])
            put(pre + "output.dense.weight", lw["w2"])
            put(pre + "output.dense.bias", lw["b2"])
            put(pre + "output.LayerNorm.weight", lw["ln2_g"])
            put(pre + "output.LayerNorm.bias", lw["ln2_b"])
        model.load_state_dict(sd)
        hid = model(input_ids=torch.from_numpy(inp.ids).long(),
                    attention_mask=torch.from_numpy(inp.mask).long()).last_hidden_state
        m = torch.from_numpy(inp.mask != 0).double()[..., None]
        pooled = (hid * m).sum(1) / m.sum(1).clamp(min=1e-9)
        ref = torch.nn.functional.normalize(pooled, p=2, dim=1, eps=1e-12).numpy()
    got, dumps = oracle.encoder_forward(c, inp.ids, inp.mask, p, inp.layers, compute_all_rows=True, dumps=True)
    valid = inp.mask != 0
    assert np.abs(dumps["x"][-1][valid] - hid.numpy()[valid]).max() < 1e-10
    assert np.abs(got - ref).max() < 1e-12


def test_oracle_rejects_bad_arguments():
    inp = tiny_inputs()
    bad = inp.ids.copy()
    bad[0, 0] = TINY.vocab
    with pytest.raises(ValueError):
        oracle.encoder_forward(inp.cfg, bad, inp.mask, inp.params, inp.layers)


def test_benchmark_config_c0_unit_norm_and_oracles_agree():
    inp = make_inputs(CONFIGS["c0"])
    assert inp.lengths.tolist() == [11] and inp.mask[0].tolist() == [1] * 11 + [0] * 5
    a = oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers)
    b = encoder_np.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers)
    assert np.abs(a - b).max() < 1e-13 and abs(np.linalg.norm(a[0]) - 1) < 1e-14


@pytest.mark.parametrize("name", ["c0", "c1"])
def test_stored_golden_embeddings_still_reproduce(name):
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", f"{name}_embedding.txt")
    want = np.loadtxt(path, comments="#")
    inp = make_inputs(CONFIGS[name])
    got = oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers).reshape(-1)
    assert np.abs(got - want).max() < 1e-13
