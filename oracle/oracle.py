"""ctypes front end of the fp64 C oracle (``encoder_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg.  Nothing on the CUDA product path may import it,
and it imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, List, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "encoder_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP, strict IEEE: no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-Wall", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class _Cfg(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("num_layers", "hidden", "num_heads", "ffn", "vocab", "max_pos", "type_vocab")] + \
               [("ln_eps", C.c_double)]


_FP = C.POINTER(C.c_float)
_DP = C.POINTER(C.c_double)
_IP = C.POINTER(C.c_int32)
_LAYER_FIELDS = ("wqkv", "bqkv", "wo", "bo", "ln1_g", "ln1_b", "w1", "b1", "w2", "b2", "ln2_g", "ln2_b")


class _Layer(C.Structure):
    _fields_ = [(n, _FP) for n in _LAYER_FIELDS]


class _Weights(C.Structure):
    _fields_ = [(n, _FP) for n in ("word_emb", "pos_emb", "type_emb", "emb_ln_g", "emb_ln_b")] + \
               [("layers", C.POINTER(_Layer))]


class _Dumps(C.Structure):
    _fields_ = [(n, _DP) for n in ("x_emb", "qkv", "ctx", "x1", "g", "x")]


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.rlx_oracle_encoder_forward.restype = C.c_int
    return _lib


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def _fp(a):
    return a.ctypes.data_as(_FP)


def _dp(a):
    return a.ctypes.data_as(_DP)


def _ip(a):
    return a.ctypes.data_as(_IP)


def set_threads(n: int) -> None:
    os.environ["OMP_NUM_THREADS"] = str(n)


def layernorm(v, gamma, beta, eps: float = 1e-12) -> np.ndarray:
    v = _f64(v)
    H = v.shape[-1]
    g, b = _f32(gamma), _f32(beta)
    out = np.empty_like(v)
    lib().rlx_oracle_layernorm(_dp(v), _fp(g), _fp(b), C.c_int64(v.size // H), C.c_int(H),
                               C.c_double(eps), _dp(out))
    return out


def linear(x, w, bias=None) -> np.ndarray:
    x = _f64(x)
    w = _f32(w)
    N, K = w.shape
    T = x.size // K
    out = np.empty(x.shape[:-1] + (N,), np.float64)
    b = _f32(bias) if bias is not None else None
    lib().rlx_oracle_linear(_dp(x), _fp(w), _fp(b) if b is not None else None, C.c_int64(T),
                            C.c_int(N), C.c_int(K), _dp(out))
    return out


def gelu(u) -> np.ndarray:
    u = _f64(u)
    out = np.empty_like(u)
    lib().rlx_oracle_gelu(_dp(u), C.c_int64(u.size), _dp(out))
    return out


def attention(qkv, mask, num_heads: int, compute_all_rows: bool = True, return_probs: bool = False):
    """qkv: [B,S,3H] packed; mask: [B,S] -> ctx [B,S,H] (and probs [B,h,S,S])."""
    qkv = _f64(qkv)
    mask = _i32(mask)
    B, S, H3 = qkv.shape
    H = H3 // 3
    d = H // num_heads
    ctx = np.empty((B, S, H), np.float64)
    probs = np.empty((B, num_heads, S, S), np.float64) if return_probs else None
    lib().rlx_oracle_attention(_dp(qkv), _ip(mask), B, S, num_heads, d, int(compute_all_rows), _dp(ctx),
                               _dp(probs) if probs is not None else None)
    return (ctx, probs) if return_probs else ctx


def pool_l2(x, mask) -> np.ndarray:
    x = _f64(x)
    mask = _i32(mask)
    B, S, H = x.shape
    out = np.empty((B, H), np.float64)
    lib().rlx_oracle_pool_l2(_dp(x), _ip(mask), B, S, H, _dp(out))
    return out


def encoder_forward(cfg, ids, mask, params: Dict[str, np.ndarray], layers: List[Dict[str, np.ndarray]],
                    compute_all_rows: bool = False, dumps: bool = False):
    """Run the whole encoder.  ``cfg`` needs num_layers, hidden, num_heads, ffn,
    vocab, max_pos, type_vocab, ln_eps attributes.  Returns out [B,H] fp64, or
    (out, dict of per-stage dumps) when ``dumps`` is set."""
    ids, mask = _i32(ids), _i32(mask)
    B, S = ids.shape
    L = len(layers)
    c = _Cfg(L, cfg.hidden, cfg.num_heads, cfg.ffn, cfg.vocab, cfg.max_pos, cfg.type_vocab, cfg.ln_eps)
    keep = []
    larr = (_Layer * max(L, 1))()
    for i, lw in enumerate(layers):
        for n in _LAYER_FIELDS:
            a = _f32(lw[n])
            keep.append(a)
            setattr(larr[i], n, _fp(a))
    w = _Weights()
    for n in ("word_emb", "pos_emb", "type_emb", "emb_ln_g", "emb_ln_b"):
        a = _f32(params[n])
        keep.append(a)
        setattr(w, n, _fp(a))
    w.layers = larr
    H, F, T = cfg.hidden, cfg.ffn, B * S
    out = np.empty((B, H), np.float64)
    d = None
    dd: Optional[Dict[str, np.ndarray]] = None
    if dumps:
        dd = {
            "x_emb": np.zeros((B, S, H)),
            "qkv": np.zeros((L, B, S, 3 * H)),
            "ctx": np.zeros((L, B, S, H)),
            "x1": np.zeros((L, B, S, H)),
            "g": np.zeros((L, B, S, F)),
            "x": np.zeros((L, B, S, H)),
        }
        d = _Dumps(*[_dp(dd[k]) for k in ("x_emb", "qkv", "ctx", "x1", "g", "x")])
    rc = lib().rlx_oracle_encoder_forward(C.byref(c), C.byref(w), _ip(ids), _ip(mask), B, S,
                                          int(compute_all_rows), _dp(out),
                                          C.byref(d) if d is not None else None)
    if rc != 0:
        raise ValueError("oracle rejected the arguments (id range, seq > max_pos, or hidden % heads)")
    return (out, dd) if dumps else out
