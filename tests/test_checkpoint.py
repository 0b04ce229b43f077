"""Checkpoint ingestion: the safetensors reader and the BERT name mapping, pinned against the
safetensors and transformers libraries (CPU), and the loaded model through the CUDA forward (GPU)."""
import json
import os
import struct

import numpy as np
import pytest

torch = pytest.importorskip("torch")
transformers = pytest.importorskip("transformers")
st = pytest.importorskip("safetensors.torch")

from oracle import oracle  # noqa: E402
from paper_2609_37916_b200 import checkpoint  # noqa: E402
from synth.inputs import round_to_bf16  # noqa: E402


def _tiny_bert(tmp_path, dtype=torch.float32, heads=4):
    torch.manual_seed(0)
    bc = transformers.BertConfig(vocab_size=97, hidden_size=128, num_hidden_layers=2, num_attention_heads=heads,
                                 intermediate_size=256, hidden_act="gelu", hidden_dropout_prob=0.0,
                                 attention_probs_dropout_prob=0.0, max_position_embeddings=40, type_vocab_size=2,
                                 layer_norm_eps=1e-12)
    model = transformers.BertModel(bc, add_pooling_layer=False).eval()
    with torch.no_grad():                       # make biases and LayerNorm parameters non-trivial
        for n, p in model.named_parameters():
            if n.endswith("bias") or "LayerNorm" in n:
                p.add_(0.1 * torch.randn_like(p))
    model = model.to(dtype)
    d = tmp_path / "ckpt"
    model.save_pretrained(str(d), safe_serialization=True)
    return model, str(d)


def test_reader_matches_the_safetensors_library(tmp_path):
    tensors = {"a": torch.randn(3, 5), "b.c": torch.randn(7).to(torch.bfloat16), "h": torch.randn(2, 2, 2).half(),
               "i": torch.arange(6, dtype=torch.int64).view(2, 3), "d": torch.randn(4).double(), "e": torch.zeros(0, 3)}
    path = str(tmp_path / "t.safetensors")
    st.save_file(tensors, path, metadata={"note": "x"})
    got = checkpoint.read_safetensors(path)
    assert set(got) == set(tensors)
    for k, v in tensors.items():
        assert got[k].shape == tuple(v.shape)
        assert np.array_equal(got[k].astype(np.float64), v.double().numpy()), k


def test_reader_rejects_truncated_and_inconsistent_files(tmp_path):
    path = str(tmp_path / "t.safetensors")
    st.save_file({"a": torch.randn(8, 8)}, path)
    raw = open(path, "rb").read()
    bad = str(tmp_path / "bad.safetensors")
    open(bad, "wb").write(raw[:-16])                         # data shorter than the header claims
    with pytest.raises(ValueError):
        checkpoint.read_safetensors(bad)
    open(bad, "wb").write(raw[:4])
    with pytest.raises(ValueError):
        checkpoint.read_safetensors(bad)
    hdr = json.dumps({"a": {"dtype": "F32", "shape": [9, 8], "data_offsets": [0, 256]}}).encode()
    open(bad, "wb").write(struct.pack("<Q", len(hdr)) + hdr + raw[-256:])
    with pytest.raises(ValueError):                           # shape and byte range disagree
        checkpoint.read_safetensors(bad)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_mapping_reproduces_the_library_model(tmp_path, dtype):
    """The oracle on the loaded arrays = the library's BertModel forward (fp64) on the same checkpoint."""
    model, d = _tiny_bert(tmp_path, dtype)
    cfg, params, layers = checkpoint.load_bert_checkpoint(d)
    assert (cfg.num_layers, cfg.hidden, cfg.num_heads, cfg.ffn, cfg.vocab, cfg.max_pos) == (2, 128, 4, 256, 97, 40)
    sd = model.state_dict()
    assert np.array_equal(params["word_emb"], sd["embeddings.word_embeddings.weight"].float().numpy())
    assert np.array_equal(layers[1]["wqkv"][128:256], sd["encoder.layer.1.attention.self.key.weight"].float().numpy())
    rng = np.random.default_rng(0)
    B, S = 3, 17
    ids = rng.integers(0, cfg.vocab, size=(B, S)).astype(np.int32)
    lengths = np.array([17, 5, 1])
    mask = (np.arange(S)[None, :] < lengths[:, None]).astype(np.int32)
    ours = oracle.encoder_forward(cfg, ids, mask, params, layers)
    with torch.no_grad():
        m64 = model.double()
        hid = m64(input_ids=torch.from_numpy(ids).long(), attention_mask=torch.from_numpy(mask).long()).last_hidden_state
        mm = torch.from_numpy(mask != 0).double()[..., None]
        ref = torch.nn.functional.normalize((hid * mm).sum(1) / mm.sum(1), p=2, dim=1).numpy()
    assert np.abs(ours - ref).max() < 1e-10


def test_head_count_is_required_without_a_config(tmp_path):
    _, d = _tiny_bert(tmp_path)
    with pytest.raises(ValueError):
        checkpoint.load_bert_checkpoint(os.path.join(d, "model.safetensors"))
    cfg, _, _ = checkpoint.load_bert_checkpoint(os.path.join(d, "model.safetensors"), num_heads=8)
    assert cfg.num_heads == 8 and cfg.head_dim == 16
    with pytest.raises(ValueError):
        checkpoint.load_bert_checkpoint(os.path.join(d, "model.safetensors"), num_heads=7)


@pytest.mark.gpu
def test_loaded_checkpoint_runs_through_the_cuda_forward(tmp_path):
    import paper_2609_37916_b200 as rlx
    from paper_2609_37916_b200.build import build
    build()
    _, d = _tiny_bert(tmp_path, torch.bfloat16, heads=4)      # head_dim 32
    cfg, params, layers = checkpoint.load_bert_checkpoint(d)
    rng = np.random.default_rng(1)
    B, S = 5, 33
    ids = rng.integers(0, cfg.vocab, size=(B, S)).astype(np.int32)
    lengths = rng.integers(1, S + 1, size=B)
    mask = (np.arange(S)[None, :] < lengths[:, None]).astype(np.int32)
    enc = rlx.Encoder.from_config(cfg, max_batch=B, max_seq=S)
    w = rlx.upload_weights(params, layers)
    ws = enc.alloc_workspace(B, S)
    out = torch.empty((B, cfg.hidden), dtype=torch.float32, device="cuda")
    enc.forward(torch.from_numpy(ids).cuda(), torch.from_numpy(mask).cuda(), w, out, ws)
    torch.cuda.synchronize()
    assert enc.last_device_status(ws) == 0
    # the oracle sees what the GPU stores: matrices and tables on the bf16 grid (exact here: a bf16 file)
    for k in ("word_emb", "pos_emb", "type_emb"):
        assert np.array_equal(params[k], round_to_bf16(params[k]))
    ref = oracle.encoder_forward(cfg, ids, mask, params, layers)
    got = out.double().cpu().numpy()
    cos = (got * ref).sum(1) / (np.linalg.norm(got, axis=1) * np.linalg.norm(ref, axis=1))
    assert cos.min() >= 0.9995 and np.abs(got - ref).max() <= 2e-2, (cos.min(), np.abs(got - ref).max())
    enc.close()
