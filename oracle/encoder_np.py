"""Second, independently written fp64 statement of the encoder forward (numpy).

TEST INFRASTRUCTURE ONLY (see ``encoder_oracle.c`` for the readings it fixes).
It exists so that the C oracle is checked against something that is not
itself: this version is whole-tensor algebra (matmul / einsum / where) and was
written separately from the C loops; the two must agree to ~1e-12.  It follows
the same definition: the named model of the paper's inference benchmark
(Section 8.2) with key-padding-masked attention (Section 3.1 mask kinds) over
views of the packed q/k/v projection (Section 3.2).
"""
from __future__ import annotations

from math import sqrt
from typing import Dict, List

import numpy as np
from scipy.special import erf as _erf


def ln(v: np.ndarray, gamma, beta, eps: float) -> np.ndarray:
    mu = v.mean(axis=-1, keepdims=True)
    var = ((v - mu) ** 2).mean(axis=-1, keepdims=True)
    return (v - mu) / np.sqrt(var + eps) * np.asarray(gamma, np.float64) + np.asarray(beta, np.float64)


def gelu(u: np.ndarray) -> np.ndarray:
    return 0.5 * u * (1.0 + _erf(u / sqrt(2.0)))


def attention(qkv: np.ndarray, mask: np.ndarray, h: int) -> np.ndarray:
    """qkv [B,S,3H] -> ctx [B,S,H]; masked keys get probability exactly 0."""
    B, S, H3 = qkv.shape
    H = H3 // 3
    d = H // h
    q, k, v = (qkv[..., i * H:(i + 1) * H].reshape(B, S, h, d) for i in range(3))
    s = np.einsum("bihc,bkhc->bhik", q, k) / sqrt(d)
    valid = (np.asarray(mask) != 0)[:, None, None, :]
    s = np.where(valid, s, -np.inf)
    m = s.max(axis=-1, keepdims=True)
    m = np.where(np.isfinite(m), m, 0.0)
    e = np.where(valid, np.exp(s - m), 0.0)
    den = e.sum(axis=-1, keepdims=True)
    p = np.divide(e, den, out=np.zeros_like(e), where=den > 0)
    return np.einsum("bhik,bkhc->bihc", p, v).reshape(B, S, H)


def encoder_forward(cfg, ids, mask, params: Dict[str, np.ndarray], layers: List[Dict[str, np.ndarray]]):
    f8 = lambda a: np.asarray(a, np.float64)
    ids = np.asarray(ids)
    mask = np.asarray(mask)
    B, S = ids.shape
    e = f8(params["word_emb"])[ids] + f8(params["pos_emb"])[None, :S, :] + f8(params["type_emb"])[0]
    x = ln(e, params["emb_ln_g"], params["emb_ln_b"], cfg.ln_eps)
    for lw in layers:
        qkv = x @ f8(lw["wqkv"]).T + f8(lw["bqkv"])
        ctx = attention(qkv, mask, cfg.num_heads)
        x1 = ln(ctx @ f8(lw["wo"]).T + f8(lw["bo"]) + x, lw["ln1_g"], lw["ln1_b"], cfg.ln_eps)
        g = gelu(x1 @ f8(lw["w1"]).T + f8(lw["b1"]))
        x = ln(g @ f8(lw["w2"]).T + f8(lw["b2"]) + x1, lw["ln2_g"], lw["ln2_b"], cfg.ln_eps)
    m = (mask != 0).astype(np.float64)[..., None]
    pool = (x * m).sum(axis=1) / np.maximum(m.sum(axis=1), 1e-9)
    nrm = np.maximum(np.sqrt((pool ** 2).sum(axis=-1, keepdims=True)), 1e-12)
    return pool / nrm
