"""Checkpoint ingestion: a safetensors file of a BERT-family encoder -> the arrays the C ABI takes.

The paper ingests safetensors as its native checkpoint format (Section 7, formats); the weight order it maps to is not
printed, so the mapping here is this library's own reading: `Linear` weights stay `[out, in]` row-major,
the query / key / value projections are stacked in that order into one `[3H, H]` matrix (head j = rows
j*d .. (j+1)*d of each third), LayerNorm weight / bias become gamma / beta.

Host-side marshalling only: the file is parsed here (8-byte little-endian header length, JSON header
with dtype / shape / byte range per tensor, raw little-endian data), nothing is computed beyond dtype
widening and concatenation, and the forward itself runs in the CUDA library.
"""
from __future__ import annotations

import json
import os
import struct
from typing import Dict, List, Optional, Tuple

import numpy as np

from synth.inputs import EncoderConfig

_DTYPES = {"F64": np.float64, "F32": np.float32, "F16": np.float16, "I64": np.int64, "I32": np.int32,
           "I16": np.int16, "I8": np.int8, "U8": np.uint8, "BOOL": np.bool_}


def read_safetensors(path: str) -> Dict[str, np.ndarray]:
    """Every tensor of the file as a numpy array (BF16 widened exactly to float32)."""
    with open(path, "rb") as f:
        raw = f.read()
    if len(raw) < 8:
        raise ValueError(f"{path}: too short for a safetensors header")
    (hlen,) = struct.unpack("<Q", raw[:8])
    if 8 + hlen > len(raw):
        raise ValueError(f"{path}: header length {hlen} exceeds the file")
    header = json.loads(raw[8:8 + hlen].decode("utf-8"))
    data = memoryview(raw)[8 + hlen:]
    out: Dict[str, np.ndarray] = {}
    for name, meta in header.items():
        if name == "__metadata__":
            continue
        lo, hi = meta["data_offsets"]
        shape = tuple(meta["shape"])
        if not (0 <= lo <= hi <= len(data)):
            raise ValueError(f"{path}: tensor {name} points outside the file")
        buf = data[lo:hi]
        if meta["dtype"] == "BF16":
            bits = np.frombuffer(buf, dtype="<u2").astype(np.uint32) << 16
            arr = bits.view(np.float32)
        elif meta["dtype"] in _DTYPES:
            arr = np.frombuffer(buf, dtype=np.dtype(_DTYPES[meta["dtype"]]).newbyteorder("<"))
        else:
            raise ValueError(f"{path}: tensor {name} has unsupported dtype {meta['dtype']}")
        if arr.size != int(np.prod(shape, dtype=np.int64)):
            raise ValueError(f"{path}: tensor {name} has {arr.size} elements for shape {shape}")
        out[name] = arr.reshape(shape)
    return out


def _strip_prefix(tensors: Dict[str, np.ndarray]) -> Dict[str, np.ndarray]:
    """Drop a leading model prefix ("bert.", "0.auto_model.", ...) so names start at "embeddings." / "encoder."."""
    key = next((k for k in tensors if k.endswith("embeddings.word_embeddings.weight")), None)
    if key is None:
        raise KeyError("no embeddings.word_embeddings.weight in the checkpoint: not a BERT-family encoder")
    prefix = key[: -len("embeddings.word_embeddings.weight")]
    return {k[len(prefix):]: v for k, v in tensors.items() if k.startswith(prefix)}


def bert_tensors_to_encoder(tensors: Dict[str, np.ndarray], num_heads: int, ln_eps: float = 1e-12
                            ) -> Tuple[EncoderConfig, Dict[str, np.ndarray], List[Dict[str, np.ndarray]]]:
    """HF-style BERT tensor names -> (config, params, layers) in this library's naming, float32."""
    t = _strip_prefix(tensors)
    f32 = lambda a: np.ascontiguousarray(a, dtype=np.float32)
    word = f32(t["embeddings.word_embeddings.weight"])
    pos = f32(t["embeddings.position_embeddings.weight"])
    typ = f32(t["embeddings.token_type_embeddings.weight"])
    H = word.shape[1]
    if H % num_heads:
        raise ValueError(f"hidden size {H} is not a multiple of {num_heads} heads")
    params = {"word_emb": word, "pos_emb": pos, "type_emb": typ,
              "emb_ln_g": f32(t["embeddings.LayerNorm.weight"]), "emb_ln_b": f32(t["embeddings.LayerNorm.bias"])}
    layers: List[Dict[str, np.ndarray]] = []
    while f"encoder.layer.{len(layers)}.attention.self.query.weight" in t:
        p = f"encoder.layer.{len(layers)}."
        qkv_w = [t[p + f"attention.self.{n}.weight"] for n in ("query", "key", "value")]
        qkv_b = [t[p + f"attention.self.{n}.bias"] for n in ("query", "key", "value")]
        layers.append({
            "wqkv": f32(np.concatenate(qkv_w, axis=0)), "bqkv": f32(np.concatenate(qkv_b, axis=0)),
            "wo": f32(t[p + "attention.output.dense.weight"]), "bo": f32(t[p + "attention.output.dense.bias"]),
            "ln1_g": f32(t[p + "attention.output.LayerNorm.weight"]), "ln1_b": f32(t[p + "attention.output.LayerNorm.bias"]),
            "w1": f32(t[p + "intermediate.dense.weight"]), "b1": f32(t[p + "intermediate.dense.bias"]),
            "w2": f32(t[p + "output.dense.weight"]), "b2": f32(t[p + "output.dense.bias"]),
            "ln2_g": f32(t[p + "output.LayerNorm.weight"]), "ln2_b": f32(t[p + "output.LayerNorm.bias"]),
        })
    if not layers:
        raise KeyError("no encoder.layer.0 in the checkpoint")
    for i, lw in enumerate(layers):
        if lw["wqkv"].shape != (3 * H, H) or lw["wo"].shape != (H, H) or lw["w2"].shape != (H, lw["w1"].shape[0]):
            raise ValueError(f"layer {i}: unexpected weight shapes")
    cfg = EncoderConfig(name="checkpoint", num_layers=len(layers), hidden=H, num_heads=num_heads,
                        ffn=layers[0]["w1"].shape[0], vocab=word.shape[0], max_pos=pos.shape[0],
                        type_vocab=typ.shape[0], ln_eps=ln_eps, batch=1, seq=min(128, pos.shape[0]),
                        len_lo=1, len_hi=min(128, pos.shape[0]), seed=0)
    return cfg, params, layers


def load_bert_checkpoint(path: str, num_heads: Optional[int] = None, ln_eps: Optional[float] = None):
    """`path`: a .safetensors file, or a directory holding model.safetensors (and, optionally, the
    config.json from which the head count and LayerNorm epsilon are read when not given)."""
    file = path
    if os.path.isdir(path):
        file = os.path.join(path, "model.safetensors")
        cfg_path = os.path.join(path, "config.json")
        if os.path.exists(cfg_path):
            with open(cfg_path) as f:
                meta = json.load(f)
            if meta.get("hidden_act", "gelu") != "gelu":
                raise ValueError(f"activation {meta['hidden_act']!r}: only the erf GELU is implemented")
            if meta.get("position_embedding_type", "absolute") != "absolute":
                raise ValueError("only absolute position embeddings are implemented")
            num_heads = num_heads or meta.get("num_attention_heads")
            ln_eps = ln_eps if ln_eps is not None else meta.get("layer_norm_eps")
    if num_heads is None:
        raise ValueError("num_heads is not stored in a safetensors file: pass it, or point at a directory with config.json")
    return bert_tensors_to_encoder(read_safetensors(file), int(num_heads), 1e-12 if ln_eps is None else float(ln_eps))
