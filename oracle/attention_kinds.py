"""fp64 statement of scaled-dot-product attention under the paper's other mask kinds, with rotary
position embedding applied to q and k first.

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's CPU-baseline leg may import this
module; the product path never does, and it shares no code with the CUDA kernels.

What it follows.  Section 3.1 parameterises masked attention by MaskKind in {None, Causal,
SlidingWindow(w), Custom}; Section 3.2 names a fused QK-RoPE region ahead of attention.  The paper
defines none of them further, so the readings used here are the ones of the decoder families its model
zoo (Section 8.5) names:

  None              every key of the sequence is visible to every query.
  Causal            key k is visible to query i  iff  k <= i.
  SlidingWindow(w)  key k is visible to query i  iff  i - w < k <= i  (the w most recent positions,
                    the query's own included; w >= 1).
  RoPE              "rotate-half" pairing: component j < d/2 is paired with j + d/2 and the pair is
                    rotated by the angle  pos * theta^(-2j/d);  pos is the row's index in its sequence,
                    theta = 10000 unless given.  Applied to every head of q and k, never to v.

Everything is the plain definition in IEEE double precision: a dense score matrix, an explicit boolean
visibility matrix, a max-subtracted softmax over the visible keys only (invisible keys get probability
exactly 0), no blocking.
"""
from __future__ import annotations

from math import sqrt
from typing import Optional

import numpy as np

KIND_NONE, KIND_CAUSAL, KIND_SLIDING = 0, 1, 2


def visible(length: int, kind: int, window: int = 0) -> np.ndarray:
    """Boolean [length, length]: entry (i, k) says whether query i may look at key k."""
    i = np.arange(length)[:, None]
    k = np.arange(length)[None, :]
    if kind == KIND_NONE:
        return np.ones((length, length), dtype=bool)
    if kind == KIND_CAUSAL:
        return k <= i
    if kind == KIND_SLIDING:
        if window < 1:
            raise ValueError("window must be >= 1")
        return (k <= i) & (k > i - window)
    raise ValueError(f"unknown mask kind {kind}")


def rope(x: np.ndarray, theta: float = 10000.0, positions: Optional[np.ndarray] = None) -> np.ndarray:
    """x [L, h, d] -> rotated copy; pair (j, j + d/2) turns by positions[l] * theta**(-2j/d)."""
    x = np.asarray(x, np.float64)
    L, _, d = x.shape
    half = d // 2
    pos = np.arange(L, dtype=np.float64) if positions is None else np.asarray(positions, np.float64)
    inv_freq = theta ** (-2.0 * np.arange(half, dtype=np.float64) / d)
    ang = pos[:, None] * inv_freq[None, :]                      # [L, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    lo, hi = x[..., :half], x[..., half:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


def split_qkv(qkv: np.ndarray, num_heads: int, num_kv_heads: Optional[int] = None):
    """qkv [L, (hq + 2 hkv) d] -> q [L, hq, d], k [L, hkv, d], v [L, hkv, d]: q heads, then k heads, then v heads."""
    hkv = num_heads if num_kv_heads is None else num_kv_heads
    L, W = qkv.shape
    d = W // (num_heads + 2 * hkv)
    assert d * (num_heads + 2 * hkv) == W and num_heads % hkv == 0
    q = qkv[:, :num_heads * d].reshape(L, num_heads, d)
    k = qkv[:, num_heads * d:(num_heads + hkv) * d].reshape(L, hkv, d)
    v = qkv[:, (num_heads + hkv) * d:].reshape(L, hkv, d)
    return q, k, v


def attention_one(qkv: np.ndarray, num_heads: int, kind: int, window: int = 0,
                  rope_theta: Optional[float] = None, num_kv_heads: Optional[int] = None) -> np.ndarray:
    """One sequence: qkv [L, (hq + 2 hkv) d] (q | k | v column blocks, head j = columns j*d..(j+1)*d of its
    block) -> ctx [L, hq d].  With fewer k/v heads than q heads (grouped-query attention, the layout of the
    decoder families the paper's model zoo names), q head j reads k/v head j // (hq / hkv)."""
    qkv = np.asarray(qkv, np.float64)
    L = qkv.shape[0]
    q, k, v = split_qkv(qkv, num_heads, num_kv_heads)
    d = q.shape[2]
    group = num_heads // k.shape[1]
    if rope_theta is not None:
        q, k = rope(q, rope_theta), rope(k, rope_theta)
    vis = visible(L, kind, window)
    ctx = np.zeros((L, num_heads, d))
    for j in range(num_heads):
        s = (q[:, j, :] @ k[:, j // group, :].T) / sqrt(d)
        s = np.where(vis, s, -np.inf)
        m = s.max(axis=1, keepdims=True)                         # every row sees at least itself
        e = np.where(vis, np.exp(s - m), 0.0)
        ctx[:, j, :] = (e / e.sum(axis=1, keepdims=True)) @ v[:, j // group, :]
    return ctx.reshape(L, num_heads * d)


def attention_packed(qkv: np.ndarray, seq_start, seq_len, num_heads: int, kind: int, window: int = 0,
                     rope_theta: Optional[float] = None, num_kv_heads: Optional[int] = None) -> np.ndarray:
    """Packed rows: sequence b owns rows seq_start[b] .. seq_start[b]+seq_len[b]; other rows stay 0."""
    qkv = np.asarray(qkv, np.float64)
    hkv = num_heads if num_kv_heads is None else num_kv_heads
    out = np.zeros((qkv.shape[0], qkv.shape[1] // (num_heads + 2 * hkv) * num_heads))
    for s0, n in zip(np.asarray(seq_start), np.asarray(seq_len)):
        s0, n = int(s0), int(n)
        if n > 0:
            out[s0:s0 + n] = attention_one(qkv[s0:s0 + n], num_heads, kind, window, rope_theta, num_kv_heads)
    return out


def rope_qk_packed(qkv: np.ndarray, seq_start, seq_len, num_heads: int, theta: float = 10000.0,
                   num_kv_heads: Optional[int] = None) -> np.ndarray:
    """The QK-RoPE region on packed rows: q and k column blocks rotated by each row's position within its
    sequence, v and rows outside every sequence returned unchanged."""
    out = np.array(qkv, dtype=np.float64, copy=True)
    hkv = num_heads if num_kv_heads is None else num_kv_heads
    d = out.shape[1] // (num_heads + 2 * hkv)
    rot = (num_heads + hkv) * d                                   # q heads then k heads: one contiguous block
    for s0, n in zip(np.asarray(seq_start), np.asarray(seq_len)):
        s0, n = int(s0), int(n)
        blk = out[s0:s0 + n, :rot].reshape(n, num_heads + hkv, d)
        out[s0:s0 + n, :rot] = rope(blk, theta).reshape(n, rot)
    return out
