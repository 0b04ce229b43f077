"""End-to-end parity of the CUDA encoder forward (through the C ABI) with the fp64 oracle on the
five benchmark configurations, plus stress variants, edge cases and bitwise properties."""
import os

import numpy as np
import pytest

torch = pytest.importorskip("torch")

from gpu_common import cosine_rows, i32_dev, to_np64  # noqa: E402
from oracle import oracle  # noqa: E402
from synth.inputs import CONFIGS, EncoderConfig, make_inputs  # noqa: E402

pytestmark = pytest.mark.gpu

# Graded tolerance: cosine >= 0.9995 per embedding and max |err| <= 2e-2.  Honest bf16 error is
# ~100x smaller, so the tests also hold a tighter internal gate that catches subtle mistakes.
COS_MIN, ABS_MAX = 0.9995, 2e-2
COS_TIGHT, ABS_TIGHT = 0.9999, 4e-3


@pytest.fixture(scope="module")
def rlx():
    import paper_2609_37916_b200 as pkg
    from paper_2609_37916_b200.build import build
    build()
    return pkg


def run_gpu(rlx, inp, flags=0, host_io=False, weights=None, enc=None):
    c = inp.cfg
    own = enc is None
    if own:
        enc = rlx.Encoder.from_config(c, flags=flags, max_batch=c.batch, max_seq=c.seq)
    w = weights if weights is not None else rlx.upload_weights(inp.params, inp.layers)
    ws = enc.alloc_workspace(c.batch, c.seq)
    if host_io:
        out = torch.empty((c.batch, c.hidden), dtype=torch.float32).pin_memory()
        enc.forward_host(torch.from_numpy(inp.ids).pin_memory(), torch.from_numpy(inp.mask).pin_memory(), w, out, ws)
        res = out.numpy().astype(np.float64)
    else:
        out = torch.empty((c.batch, c.hidden), dtype=torch.float32, device="cuda")
        enc.forward(i32_dev(inp.ids), i32_dev(inp.mask), w, out, ws)
        torch.cuda.synchronize()
        res = to_np64(out)
    status = enc.last_device_status(ws)
    if own:
        enc.close()
    return res, status


def check(got, ref, lengths, tight=True):
    keep = np.asarray(lengths) > 0
    cos = cosine_rows(got[keep], ref[keep])
    err = np.abs(got - ref).max()
    assert np.all(np.isfinite(got))
    assert cos.min() >= COS_MIN and err <= ABS_MAX, (cos.min(), err)
    if tight:
        assert cos.min() >= COS_TIGHT and err <= ABS_TIGHT, (cos.min(), err)
    assert np.allclose(np.linalg.norm(got[keep], axis=1), 1.0, atol=1e-5)
    return float(cos.min()), float(err)


@pytest.mark.parametrize("name", ["c0", "c1", "c2"])
@pytest.mark.parametrize("mode", ["graph", "eager", "padded", "separate_ln", "separate_ln_eager", "attn_tcgen05", "cluster_ln",
                                  "fold_ln", "fold_ln_eager", "fold_ln_padded", "simt_gemm", "host_io"])
def test_full_config_matches_oracle(rlx, name, mode):
    if mode == "simt_gemm" and name == "c2":
        pytest.skip("bring-up GEMM is covered on c0/c1")
    inp = make_inputs(CONFIGS[name])
    flags = {"graph": 0, "eager": 1, "padded": 8, "separate_ln": 0x400, "separate_ln_eager": 0x401, "attn_tcgen05": 0x20, "cluster_ln": 0x80, "fold_ln": 0x200,
             "fold_ln_eager": 0x201, "fold_ln_padded": 0x208, "simt_gemm": 1 | 2, "host_io": 0}[mode]
    got, status = run_gpu(rlx, inp, flags=flags, host_io=(mode == "host_io"))
    assert status == 0
    ref = oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers)
    check(got, ref, inp.lengths)


def test_c0_matches_stored_golden(rlx):
    inp = make_inputs(CONFIGS["c0"])
    got, _ = run_gpu(rlx, inp)
    want = np.loadtxt(os.path.join(os.path.dirname(__file__), "golden", "c0_embedding.txt"), comments="#")
    check(got, want.reshape(1, -1), inp.lengths)


@pytest.mark.parametrize("flags", [0, 0x400, 0x20, 0x40, 0x80, 0x200], ids=["default", "separate_ln", "attn_tcgen05", "whole_row_ln", "cluster_ln", "fold_ln"])
@pytest.mark.parametrize("name,sample", [("c3", [0, 1, 100, 255]), ("c4", [0, 63])])
def test_large_config_sampled_sequences_match_oracle(rlx, name, sample, flags):
    """Full-size run in the benchmark's launch configuration; the oracle recomputes a sample of the
    sequences one by one (sequences are independent, so a batch-1 oracle call is the same function)."""
    inp = make_inputs(CONFIGS[name])
    got, status = run_gpu(rlx, inp, flags=flags)
    assert status == 0
    assert np.all(np.isfinite(got))
    assert np.allclose(np.linalg.norm(got, axis=1), 1.0, atol=1e-5)
    # always include the shortest and the longest sequence of the batch
    sample = sorted(set(sample) | {int(np.argmin(inp.lengths)), int(np.argmax(inp.lengths))})
    one = EncoderConfig(**{**inp.cfg.__dict__, "batch": len(sample)})
    ref = oracle.encoder_forward(one, inp.ids[sample], inp.mask[sample], inp.params, inp.layers)
    check(got[sample], ref, inp.lengths[sample])


def test_host_call_pinned_and_pageable_buffers_and_new_contents_between_calls(rlx):
    """rlx_encoder_forward_host with pinned and with pageable host buffers: both give the device call's
    bits, and a second call on the same buffers (the cached graph is replayed) reads what they hold at
    that moment."""
    a = make_inputs(CONFIGS["c1"], num_layers=2)
    c = a.cfg
    w = rlx.upload_weights(a.params, a.layers)
    enc = rlx.Encoder.from_config(c, max_batch=c.batch, max_seq=c.seq)
    ws = enc.alloc_workspace(c.batch, c.seq)
    want = torch.empty((c.batch, c.hidden), dtype=torch.float32, device="cuda")

    def device_result(ids, mask):
        enc.forward(i32_dev(ids), i32_dev(mask), w, want, ws)
        torch.cuda.synchronize()
        return want.cpu().numpy().copy()

    second_ids, second_mask = a.ids[::-1].copy(), a.mask[::-1].copy()   # the batch in reverse order
    for pinned in (True, False):
        ids = torch.from_numpy(a.ids.copy())
        mask = torch.from_numpy(a.mask.copy())
        out = torch.empty((c.batch, c.hidden), dtype=torch.float32)
        if pinned:
            ids, mask, out = ids.pin_memory(), mask.pin_memory(), out.pin_memory()
        enc.forward_host(ids, mask, w, out, ws)
        assert np.array_equal(out.numpy(), device_result(a.ids, a.mask))
        ids.copy_(torch.from_numpy(second_ids))       # same buffers, new contents: the cached graph is replayed
        mask.copy_(torch.from_numpy(second_mask))
        enc.forward_host(ids, mask, w, out, ws)
        assert np.array_equal(out.numpy(), device_result(second_ids, second_mask))
    assert enc.last_device_status(ws) == 0
    enc.close()


@pytest.mark.parametrize("flags", [0x800, 0x801], ids=["graph", "eager"])
def test_token_chunk_scheduling_is_bitwise_the_unchunked_forward(rlx, flags):
    """RLX_FLAG_CHUNKED: 200 sequences x 128 positions (25,600 padded tokens) run as two sub-batches through the
    same workspace; same kernels on fewer rows, so every bit must agree with the single-pass forward."""
    inp = make_inputs(CONFIGS["c2"], batch=200, num_layers=2)
    w = rlx.upload_weights(inp.params, inp.layers)
    whole, status = run_gpu(rlx, inp, weights=w, flags=flags & 1)
    assert status == 0
    parts, status = run_gpu(rlx, inp, weights=w, flags=flags)
    assert status == 0
    assert np.array_equal(whole, parts)
    again, status = run_gpu(rlx, inp, weights=w, flags=flags)      # a second call on a fresh encoder: same bits
    assert status == 0 and np.array_equal(again, parts)


@pytest.mark.parametrize("name", ["c3", "c4"])
def test_large_config_every_sequence_matches_oracle(rlx, name):
    """The two large configurations in the benchmark's launch configuration, EVERY sequence compared
    with the oracle (about 25 s and 100 s of oracle time on 16 host cores)."""
    oracle.set_threads(len(os.sched_getaffinity(0)))
    inp = make_inputs(CONFIGS[name])
    got, status = run_gpu(rlx, inp)
    assert status == 0
    ref = oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers)
    check(got, ref, inp.lengths)


@pytest.mark.parametrize("name", ["c0", "c1", "c2"])
def test_oracle_on_unrounded_weights_still_within_graded_tolerance(rlx, name):
    """Secondary reading of the weight precision: the oracle consumes the fp32 draws, the GPU their bf16
    roundings (the generator rounds; neither side does).  Weight quantisation then adds to the error,
    which must still clear the graded gate (cosine >= 0.9995, max |err| <= 2e-2); the tight internal
    gate belongs to the primary reading only."""
    rounded = make_inputs(CONFIGS[name])
    raw = make_inputs(CONFIGS[name], fp32_weights=True)
    assert np.array_equal(rounded.ids, raw.ids) and np.array_equal(rounded.mask, raw.mask)
    assert not np.array_equal(rounded.layers[0]["wqkv"], raw.layers[0]["wqkv"])
    got, status = run_gpu(rlx, rounded)
    assert status == 0
    ref = oracle.encoder_forward(raw.cfg, raw.ids, raw.mask, raw.params, raw.layers)
    check(got, ref, raw.lengths, tight=False)


@pytest.mark.parametrize("kw", [dict(qk_gain=8.0), dict(ln_affine_random=True), dict(mask_holes=0.3),
                                dict(qk_gain=8.0, ln_affine_random=True, mask_holes=0.2)],
                         ids=["peaky_softmax", "ln_affine", "mask_holes", "all"])
def test_stress_variants(rlx, kw):
    inp = make_inputs(CONFIGS["c1"], batch=4, seq=96, **kw)
    got, status = run_gpu(rlx, inp)
    assert status == 0
    padded, _ = run_gpu(rlx, inp, flags=8)           # padded layout: same function, other key blocking
    assert np.abs(got - padded).max() <= 2e-3
    ref = oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers)
    # a peaky softmax amplifies bf16 rounding of q and k: keep the graded gate, relax the internal one
    check(got, ref, inp.lengths, tight=("qk_gain" not in kw))


@pytest.mark.parametrize("B,S", [(1, 1), (3, 17), (2, 127), (2, 129), (1, 512), (5, 64)])
def test_odd_shapes(rlx, B, S):
    lengths = np.random.default_rng(B * 1000 + S).integers(1, S + 1, size=B)
    lengths[0] = S
    inp = make_inputs(CONFIGS["c1"], batch=B, seq=S, num_layers=2, lengths=lengths)
    got, status = run_gpu(rlx, inp)
    assert status == 0
    ref = oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers)
    check(got, ref, inp.lengths)


@pytest.mark.parametrize("seed", range(12))
def test_random_small_problems_match_oracle(rlx, seed):
    """Randomised sweep over batch, sequence length, valid lengths (incl. 0 and full), holes, LayerNorm
    affine parameters and layer count, each compared with the oracle and between the execution modes."""
    rng = np.random.default_rng(1000 + seed)
    B = int(rng.integers(1, 9))
    S = int(rng.choice([1, 2, 15, 16, 17, 31, 33, 63, 64, 65, 100, 128, 130, 200, 255, 256]))
    L = int(rng.integers(1, 4))
    lengths = rng.integers(0, S + 1, size=B)
    lengths[rng.integers(0, B)] = S
    inp = make_inputs(CONFIGS["c1"], batch=B, seq=S, num_layers=L, lengths=lengths,
                      ln_affine_random=bool(seed % 2), mask_holes=0.25 if seed % 3 == 0 else 0.0,
                      qk_gain=3.0 if seed % 4 == 0 else 1.0)
    ref = oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers)
    w = rlx.upload_weights(inp.params, inp.layers)
    base, status = run_gpu(rlx, inp, weights=w)
    assert status == 0
    check(base, ref, inp.lengths, tight=(seed % 4 != 0))
    assert np.array_equal(base[inp.lengths == 0], np.zeros_like(base[inp.lengths == 0]))
    for flags in (0x10, 0x100, 1, 0x400, 0x401, 0x420, 0x20, 0x80, 8, 0x408, 0x200, 0x201):   # no PDL, no prefetch, eager, tcgen05 attn, cluster LN, padded, folded LN (graph / eager)
        other, status = run_gpu(rlx, inp, weights=w, flags=flags)
        assert status == 0
        if flags in (0x10, 0x100, 1):
            assert np.array_equal(base, other), hex(flags)     # same kernels, other launch mechanics
        else:
            check(other, ref, inp.lengths, tight=(seed % 4 != 0))


def test_degenerate_lengths_zero_one_full(rlx):
    inp = make_inputs(CONFIGS["c1"], batch=3, seq=40, num_layers=2, lengths=[0, 1, 40])
    got, status = run_gpu(rlx, inp)
    assert status == 0
    assert np.array_equal(got[0], np.zeros(inp.cfg.hidden))   # no valid token -> zero embedding
    ref = oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers)
    check(got, ref, inp.lengths)


def test_all_sequences_empty_gives_zero_embeddings(rlx):
    """No valid token anywhere: zero packed rows, every kernel must cope with an empty problem."""
    inp = make_inputs(CONFIGS["c1"], batch=3, seq=33, num_layers=2, lengths=[0, 0, 0])
    for flags in (0, 8, 0x20):
        got, status = run_gpu(rlx, inp, flags=flags)
        assert status == 0
        assert np.array_equal(got, np.zeros_like(got))


def test_vocabulary_ends_and_out_of_range_ids(rlx):
    inp = make_inputs(CONFIGS["c0"])
    inp.ids[0, 0], inp.ids[0, 1] = 0, inp.cfg.vocab - 1
    got, status = run_gpu(rlx, inp)
    assert status == 0
    ref = oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers)
    check(got, ref, inp.lengths)
    bad = make_inputs(CONFIGS["c0"])
    bad.ids[0, 2] = bad.cfg.vocab + 7
    _, status = run_gpu(rlx, bad)
    assert status == 6  # RLX_ERR_TOKEN_RANGE: clamped and flagged, no fault


def test_padding_invariance_and_determinism_are_bitwise(rlx):
    inp = make_inputs(CONFIGS["c2"], batch=8)
    w = rlx.upload_weights(inp.params, inp.layers)
    a, _ = run_gpu(rlx, inp, weights=w)
    b, _ = run_gpu(rlx, inp, weights=w)
    assert np.array_equal(a, b)                        # run-to-run determinism
    e, _ = run_gpu(rlx, inp, weights=w, flags=1)
    assert np.array_equal(a, e)                        # graph replay == eager launches
    p, _ = run_gpu(rlx, inp, weights=w, flags=8)
    assert np.array_equal(a, p)                        # packed rows == padded layout (prefix masks)
    moved = make_inputs(CONFIGS["c2"], batch=8)
    pad = moved.mask == 0
    assert pad.any()
    moved.ids[pad] = (moved.ids[pad] + 12345) % moved.cfg.vocab
    c, _ = run_gpu(rlx, moved, weights=w)
    assert np.array_equal(a, c)                        # ids under mask 0 do not matter
    perm = np.random.default_rng(0).permutation(8)
    moved.ids, moved.mask = inp.ids[perm], inp.mask[perm]
    d, _ = run_gpu(rlx, moved, weights=w)
    assert np.array_equal(a[perm], d)                  # batch-permutation equivariance


def test_forward_refuses_an_encoder_bound_to_another_device(rlx):
    inp = make_inputs(CONFIGS["c0"])
    c = inp.cfg
    enc = rlx.Encoder.from_config(c, max_batch=1, max_seq=c.seq, device=torch.cuda.device_count())  # not current
    w = rlx.upload_weights(inp.params, inp.layers)
    out = torch.zeros((1, c.hidden), dtype=torch.float32, device="cuda")
    with pytest.raises(rlx.RlxError) as ei:
        enc.forward(i32_dev(inp.ids), i32_dev(inp.mask), w, out, enc.alloc_workspace(1, c.seq))
    assert ei.value.status == 1 and torch.count_nonzero(out) == 0
    enc.close()


def test_graph_cache_reuse_and_new_inputs(rlx):
    """Same encoder object, several calls: the captured graph must be replayed for the same
    pointer set and rebuilt when the buffers or the weights change."""
    inp = make_inputs(CONFIGS["c1"])
    c = inp.cfg
    enc = rlx.Encoder.from_config(c, max_batch=4, max_seq=c.seq)
    w = rlx.upload_weights(inp.params, inp.layers)
    ws = enc.alloc_workspace(1, c.seq)
    ids, mask = i32_dev(inp.ids), i32_dev(inp.mask)
    out = torch.empty((1, c.hidden), dtype=torch.float32, device="cuda")
    ref = oracle.encoder_forward(c, inp.ids, inp.mask, inp.params, inp.layers)
    for _ in range(3):
        out.zero_()
        enc.forward(ids, mask, w, out, ws)
        torch.cuda.synchronize()
        check(to_np64(out), ref, inp.lengths)
    # new contents in the same buffers: replay must read them
    ids2 = inp.ids.copy()
    ids2[0, :4] = [5, 6, 7, 8]
    ids.copy_(torch.from_numpy(ids2))
    enc.forward(ids, mask, w, out, ws)
    torch.cuda.synchronize()
    ref2 = oracle.encoder_forward(c, ids2, inp.mask, inp.params, inp.layers)
    check(to_np64(out), ref2, inp.lengths)
    # different weights -> different result, not a stale graph
    other = make_inputs(CONFIGS["c0"], batch=1, seq=c.seq, num_layers=c.num_layers, lengths=inp.lengths)
    w2 = rlx.upload_weights(other.params, other.layers)
    enc.forward(ids, mask, w2, out, ws)
    torch.cuda.synchronize()
    ref3 = oracle.encoder_forward(c, ids2, inp.mask, other.params, other.layers)
    check(to_np64(out), ref3, inp.lengths)
    enc.close()


@pytest.mark.parametrize("flags", [0x1400, 0x1401], ids=["graph", "eager"])
def test_fused_ffn_forward_against_the_two_kernel_forward(rlx, flags):
    """RLX_FLAG_FUSED_FFN: everything of a layer behind the attention in one kernel.  The products have the
    rounding points and the k order of the separate GEMMs; both LayerNorms work on unrounded sums (two bf16
    roundings fewer per layer), so the embeddings differ from the plain 7-kernel layer's by rounding noise only
    (0x400 keeps LayerNorm folding out of both)."""
    inp = make_inputs(CONFIGS["c2"])
    w = rlx.upload_weights(inp.params, inp.layers)
    plain, status = run_gpu(rlx, inp, weights=w, flags=0x400 | (flags & 1))
    assert status == 0
    fused, status = run_gpu(rlx, inp, weights=w, flags=flags)
    assert status == 0
    assert np.abs(plain - fused).max() <= 2e-3
    ref = oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers)
    check(fused, ref, inp.lengths)


def test_fused_ffn_is_chosen_from_32768_padded_tokens_on(rlx):
    """Without a flag the one-kernel layer tail takes over at batch*seq >= 32768; RLX_FLAG_NO_FUSED_FFN (0x2000)
    keeps the 7-kernel layer.  Four kernels less per layer, embeddings equal up to rounding noise."""
    inp = make_inputs(CONFIGS["c2"], batch=256, num_layers=2)
    w = rlx.upload_weights(inp.params, inp.layers)
    auto, status = run_gpu(rlx, inp, weights=w, flags=0)
    assert status == 0
    two, status = run_gpu(rlx, inp, weights=w, flags=0x2000)
    assert status == 0
    assert np.abs(auto - two).max() <= 2e-3
    ref = oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers)
    check(auto, ref, inp.lengths)
    c = inp.cfg
    assert c.batch * c.seq >= 32768
    a = rlx.Encoder.from_config(c, flags=0, max_batch=c.batch, max_seq=c.seq)
    b = rlx.Encoder.from_config(c, flags=0x2000, max_batch=c.batch, max_seq=c.seq)
    assert b.kernels_per_forward(256, 128) - a.kernels_per_forward(256, 128) == 4 * c.num_layers
    assert a.kernels_per_forward(255, 128) == b.kernels_per_forward(255, 128)
    a.close(); b.close()


def test_layer_tail_forward_on_random_shapes(rlx):
    """Random batches (1..40 sequences of 1..512 positions, empty sequences, masks with holes, random LayerNorm
    affine, 1..3 layers) through the forced 3-kernel layer, graph / eager / unpacked: against the oracle, run
    twice for bit-for-bit repeatability."""
    rng = np.random.default_rng(4242)
    for _ in range(10):
        B = int(rng.integers(1, 40))
        S = int(rng.choice([1, 7, 16, 33, 64, 65, 127, 128, 200, 256, 300, 512]))
        L = int(rng.integers(1, 4))
        lengths = rng.integers(0, S + 1, size=B)
        lengths[rng.integers(0, B)] = S
        inp = make_inputs(CONFIGS["c1"], batch=B, seq=S, num_layers=L, lengths=lengths,
                          ln_affine_random=bool(rng.integers(0, 2)), mask_holes=0.2 if rng.integers(0, 3) == 0 else 0.0)
        ref = oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers)
        w = rlx.upload_weights(inp.params, inp.layers)
        for flags in (0x1400, 0x1401, 0x1408):
            enc = rlx.Encoder.from_config(inp.cfg, flags=flags, max_batch=B, max_seq=S)
            assert enc.kernels_per_forward(B, S) == (2 if flags & 8 else 3) + 3 * L
            a, status = run_gpu(rlx, inp, weights=w, enc=enc)
            b, _ = run_gpu(rlx, inp, weights=w, enc=enc)
            enc.close()
            assert status == 0 and np.array_equal(a, b), (B, S, L, hex(flags))
            check(a, ref, inp.lengths, tight=False)


def test_captured_forward_chooses_the_layer_form_on_the_device(rlx):
    """RLX_FLAG_DEVICE_CHOICE (0x4000): from 12288 padded tokens on a captured forward carries both forms of the layer
    behind an IF / ELSE graph node; the packing kernel takes the layer tail when at least 9216 rows are valid.  Same call, same
    shapes, two masks: the dense batch gives bit for bit the forced layer-tail result, the sparse one the
    separate kernels' result."""
    B, S = 100, 128
    for lengths, forced in ((np.full(B, S), 0x1400), (np.full(B, 30), 0x2400)):
        inp = make_inputs(CONFIGS["c2"], batch=B, seq=S, num_layers=2, lengths=lengths)
        w = rlx.upload_weights(inp.params, inp.layers)
        auto, status = run_gpu(rlx, inp, weights=w, flags=0x4400)
        assert status == 0
        ref_path, status = run_gpu(rlx, inp, weights=w, flags=forced)
        assert status == 0
        assert np.array_equal(auto, ref_path), int(lengths.sum())
        again, _ = run_gpu(rlx, inp, weights=w, flags=0x4400)
        assert np.array_equal(auto, again)
        check(auto, oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers), inp.lengths)
