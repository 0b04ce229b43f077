"""Seeded synthetic inputs for the masked-encoder forward path.

This module only DRAWS data (token ids, masks, parameter values) and rounds
parameter matrices to the bf16 grid.  It contains none of the encoder's
arithmetic, so both the CPU oracle's tests and the CUDA path's tests/bench can
read the very same bytes from it without sharing any method code.

Workload shapes follow the paper's inference benchmark (Section 8.2: a 384-d,
6-layer sentence-embedding encoder at sequence length 128, batch 1-32,
synthetic inputs); the trained checkpoint is not available offline, so seeded
N(0, 0.02) parameters of the same shapes stand in for it.

Draw order for a config with seed ``s`` (``rng = numpy.random.default_rng(s)``,
PCG64):
  1. lengths  = rng.integers(lo, hi + 1, size=B)
  2. ids      = rng.integers(0, vocab, size=(B, S), dtype=int32)  (also under mask 0)
  3. word_emb, pos_emb, type_emb, then per layer wqkv, bqkv, wo, bo, w1, b1, w2, b2,
     each ``rng.standard_normal(shape, dtype=float32) * 0.02``
  4. (optional stress draws, after everything above so the base stream is unchanged)
LayerNorm gamma = 1, beta = 0 unless ``ln_affine_random`` is set.

Precision convention shared by both sides: matrices and embedding tables are
rounded once, here, to the nearest-even bf16 value; biases and LayerNorm
gamma/beta stay fp32.  Every returned array is float32 holding exactly those
values, so widening to fp64 (oracle) or narrowing to bf16 (GPU) is lossless.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional

import numpy as np


@dataclass(frozen=True)
class EncoderConfig:
    name: str
    num_layers: int
    hidden: int
    num_heads: int
    ffn: int
    batch: int
    seq: int
    len_lo: int
    len_hi: int
    seed: int
    vocab: int = 30522
    max_pos: int = 512
    type_vocab: int = 2
    ln_eps: float = 1e-12

    @property
    def head_dim(self) -> int:
        return self.hidden // self.num_heads

    @property
    def tokens(self) -> int:
        return self.batch * self.seq


# The five benchmark configurations (index = seed).
CONFIGS: Dict[str, EncoderConfig] = {
    "c0": EncoderConfig("c0", 1, 384, 12, 1536, 1, 16, 11, 11, 0),
    "c1": EncoderConfig("c1", 6, 384, 12, 1536, 1, 128, 8, 128, 1),
    "c2": EncoderConfig("c2", 6, 384, 12, 1536, 32, 128, 8, 128, 2),
    "c3": EncoderConfig("c3", 6, 384, 12, 1536, 256, 256, 32, 256, 3),
    "c4": EncoderConfig("c4", 12, 768, 12, 3072, 64, 512, 64, 512, 4),
}

MATRIX_KEYS = ("wqkv", "wo", "w1", "w2")
VECTOR_KEYS = ("bqkv", "bo", "ln1_g", "ln1_b", "b1", "b2", "ln2_g", "ln2_b")
LAYER_KEYS = ("wqkv", "bqkv", "wo", "bo", "ln1_g", "ln1_b", "w1", "b1", "w2", "b2", "ln2_g", "ln2_b")
TABLE_KEYS = ("word_emb", "pos_emb", "type_emb")


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest-even bf16 value; result stays float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    r = (u + bias) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that already lie on the bf16 grid."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    assert not np.any(u & np.uint32(0xFFFF)), "values are not bf16-representable"
    return (u >> np.uint32(16)).astype(np.uint16)


@dataclass
class EncoderInputs:
    cfg: EncoderConfig
    ids: np.ndarray          # int32 [B, S]
    mask: np.ndarray         # int32 [B, S], nonzero = valid
    lengths: np.ndarray      # int64 [B]  (number of valid positions)
    params: Dict[str, np.ndarray] = field(default_factory=dict)   # tables + emb_ln_g/b
    layers: List[Dict[str, np.ndarray]] = field(default_factory=list)


def make_inputs(
    cfg: EncoderConfig,
    *,
    batch: Optional[int] = None,
    seq: Optional[int] = None,
    num_layers: Optional[int] = None,
    lengths: Optional[np.ndarray] = None,
    fp32_weights: bool = False,
    qk_gain: float = 1.0,
    ln_affine_random: bool = False,
    mask_holes: float = 0.0,
    weights: bool = True,
) -> EncoderInputs:
    """Draw ids, mask and parameters for ``cfg``.

    ``batch`` / ``seq`` / ``num_layers`` override the config's sizes (used by
    reduced test cases); ``lengths`` pins the valid lengths instead of drawing
    them.  Stress options: ``qk_gain`` multiplies the query and key rows of
    ``wqkv`` (peaky softmax), ``ln_affine_random`` draws gamma ~ N(1, 0.1),
    beta ~ N(0, 0.1), ``mask_holes`` zeroes that fraction of the valid
    positions at random (non-prefix masks).  ``fp32_weights`` skips the bf16
    rounding of the matrices (secondary reading of the weight precision).
    """
    if batch is not None or seq is not None or num_layers is not None:
        cfg = replace(
            cfg,
            batch=cfg.batch if batch is None else batch,
            seq=cfg.seq if seq is None else seq,
            num_layers=cfg.num_layers if num_layers is None else num_layers,
        )
    B, S, H, F, L = cfg.batch, cfg.seq, cfg.hidden, cfg.ffn, cfg.num_layers
    rng = np.random.default_rng(cfg.seed)
    drawn = rng.integers(min(cfg.len_lo, S), min(cfg.len_hi, S) + 1, size=B)
    if lengths is not None:
        drawn = np.asarray(lengths, dtype=np.int64).reshape(B)
    mask = (np.arange(S)[None, :] < drawn[:, None]).astype(np.int32)
    ids = rng.integers(0, cfg.vocab, size=(B, S), dtype=np.int32)
    out = EncoderInputs(cfg=cfg, ids=ids, mask=mask, lengths=drawn.astype(np.int64))
    if not weights:
        return out

    def draw(*shape):
        return rng.standard_normal(shape, dtype=np.float32) * np.float32(0.02)

    p = out.params
    p["word_emb"] = draw(cfg.vocab, H)
    p["pos_emb"] = draw(cfg.max_pos, H)
    p["type_emb"] = draw(cfg.type_vocab, H)
    p["emb_ln_g"] = np.ones(H, np.float32)
    p["emb_ln_b"] = np.zeros(H, np.float32)
    for _ in range(L):
        lw: Dict[str, np.ndarray] = {}
        lw["wqkv"] = draw(3 * H, H)
        lw["bqkv"] = draw(3 * H)
        lw["wo"] = draw(H, H)
        lw["bo"] = draw(H)
        lw["w1"] = draw(F, H)
        lw["b1"] = draw(F)
        lw["w2"] = draw(H, F)
        lw["b2"] = draw(H)
        for k in ("ln1_g", "ln2_g"):
            lw[k] = np.ones(H, np.float32)
        for k in ("ln1_b", "ln2_b"):
            lw[k] = np.zeros(H, np.float32)
        out.layers.append(lw)

    # ---- stress draws (after the base stream) ----
    if qk_gain != 1.0:
        for lw in out.layers:
            lw["wqkv"][: 2 * H] *= np.float32(qk_gain)
            lw["bqkv"][: 2 * H] *= np.float32(qk_gain)
    if ln_affine_random:
        p["emb_ln_g"] = (1.0 + 0.1 * rng.standard_normal(H)).astype(np.float32)
        p["emb_ln_b"] = (0.1 * rng.standard_normal(H)).astype(np.float32)
        for lw in out.layers:
            for k in ("ln1_g", "ln2_g"):
                lw[k] = (1.0 + 0.1 * rng.standard_normal(H)).astype(np.float32)
            for k in ("ln1_b", "ln2_b"):
                lw[k] = (0.1 * rng.standard_normal(H)).astype(np.float32)
    if mask_holes > 0.0:
        holes = rng.random((B, S)) < mask_holes
        out.mask = (out.mask * (~holes)).astype(np.int32)
        out.lengths = out.mask.sum(axis=1).astype(np.int64)

    if not fp32_weights:
        for k in TABLE_KEYS:
            p[k] = round_to_bf16(p[k])
        for lw in out.layers:
            for k in MATRIX_KEYS:
                lw[k] = round_to_bf16(lw[k])
    return out


def random_mask_case(seed: int, batch: int, seq: int, lo: int = 1) -> np.ndarray:
    """Prefix-mask lengths for ad-hoc test cases: uniform in [lo, seq]."""
    return np.random.default_rng(seed).integers(lo, seq + 1, size=batch)


def make_block_scaled_weights(seed: int, n: int, k: int, code_bits: int, max_magnitude: int,
                              scale_lo: int = 118, scale_hi: int = 136):
    """Seeded block-scaled minifloat weights: codes uint8 [n, k] with a random sign bit (bit code_bits-1)
    over a uniform magnitude code in [0, max_magnitude] (callers pass the largest magnitude code that is
    a finite number in their format), and one scale byte per 32 consecutive k drawn uniformly from
    [scale_lo, scale_hi].  Holds no decoding arithmetic."""
    rng = np.random.default_rng(seed)
    mag = rng.integers(0, max_magnitude + 1, size=(n, k))
    sign = rng.integers(0, 2, size=(n, k)) << (code_bits - 1)
    scales = rng.integers(scale_lo, scale_hi + 1, size=(n, k // 32))
    return (mag | sign).astype(np.uint8), scales.astype(np.uint8)


def pack_nibbles(codes: np.ndarray) -> np.ndarray:
    """[n, k] 4-bit codes -> [n, k/2] bytes, the element with the smaller k in the low nibble."""
    codes = np.asarray(codes, np.uint8)
    return (codes[:, 0::2] | (codes[:, 1::2] << 4)).astype(np.uint8)
