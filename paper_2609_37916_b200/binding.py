"""ctypes binding of ``librlx_encoder.so`` (declared in ``include/rlx_encoder.h``).

Argument marshalling only: every step of the encoder runs inside the CUDA
library.  PyTorch is used for device memory and streams, nothing else.  The
library must have been built (``python -m paper_2609_37916_b200.build``);
there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "librlx_encoder.so")

RLX_OK = 0
STATUS_NAMES = {0: "RLX_OK", 1: "RLX_ERR_INVALID_ARG", 2: "RLX_ERR_UNSUPPORTED", 3: "RLX_ERR_WORKSPACE",
                4: "RLX_ERR_CUDA", 5: "RLX_ERR_DEVICE_TIMEOUT", 6: "RLX_ERR_TOKEN_RANGE"}
FLAG_NO_GRAPH = 0x1
FLAG_GEMM_SIMT = 0x2
FLAG_KERNEL_EVENTS = 0x4
FLAG_NO_PACK = 0x8
FLAG_NO_PDL = 0x10
FLAG_ATTN_TCGEN05 = 0x20
FLAG_FUSED_LN = 0x40
FLAG_CLUSTER_LN = 0x80
FLAG_NO_PREFETCH = 0x100
FLAG_FOLD_LN = 0x200
FLAG_NO_AUTO_FOLD = 0x400
FLAG_CHUNKED = 0x800
FLAG_FUSED_FFN = 0x1000
FLAG_NO_FUSED_FFN = 0x2000
FLAG_DEVICE_CHOICE = 0x4000
EPI_BIAS, EPI_BIAS_GELU, EPI_BIAS_RESIDUAL = 0, 1, 2
GEMM_TCGEN05, GEMM_SIMT, GEMM_TCGEN05_PAIR, GEMM_TCGEN05_SINGLE, GEMM_TCGEN05_RESIDENT = 0, 1, 2, 3, 4
STATIC_WORKSPACE_BYTES = 16 << 20

EXPORTS = (
    "rlx_encoder_create", "rlx_encoder_destroy", "rlx_encoder_workspace_bytes", "rlx_encoder_forward",
    "rlx_encoder_forward_host", "rlx_encoder_forward_tp", "rlx_encoder_forward_static", "rlx_encoder_last_device_status", "rlx_encoder_kernels_per_forward", "rlx_encoder_kernel_times",
    "rlx_status_string", "rlx_pack_sequences", "rlx_embed_layernorm", "rlx_layernorm", "rlx_gemm_bf16", "rlx_gemm_residual_layernorm_bf16", "rlx_attention_bf16",
    "rlx_attention_f32", "rlx_attention_packed_bf16", "rlx_attention_kind_bf16", "rlx_rope_tables", "rlx_qk_rope_bf16", "rlx_dequant_block_scaled_bf16", "rlx_scaled_matmul_bf16", "rlx_quantise_mx", "rlx_mx_matmul_bf16", "rlx_ffn_fused_bf16", "rlx_layer_tail_bf16", "rlx_selftest_bounded_wait", "rlx_pool_l2norm",
)


class RlxError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}")


class _Config(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("num_layers", C.c_int32), ("hidden", C.c_int32),
                ("num_heads", C.c_int32), ("ffn", C.c_int32), ("vocab", C.c_int32), ("max_pos", C.c_int32),
                ("type_vocab", C.c_int32), ("ln_eps", C.c_float), ("max_batch", C.c_int32),
                ("max_seq", C.c_int32), ("device", C.c_int32), ("flags", C.c_uint32)]


LAYER_FIELDS = ("wqkv", "bqkv", "wo", "bo", "ln1_g", "ln1_b", "w1", "b1", "w2", "b2", "ln2_g", "ln2_b")
BF16_FIELDS = {"wqkv", "wo", "w1", "w2", "word_emb", "pos_emb", "type_emb"}


class _Layer(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in LAYER_FIELDS]


class _Weights(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("word_emb", C.c_void_p), ("pos_emb", C.c_void_p),
                ("type_emb", C.c_void_p), ("emb_ln_g", C.c_void_p), ("emb_ln_b", C.c_void_p),
                ("layers", C.POINTER(_Layer))]


ALLREDUCE_FN = C.CFUNCTYPE(C.c_int, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p)

_lib = None


def lib_path() -> str:
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2609_37916_b200.build` "
                              "(there is no fallback path)")
        _lib = C.CDLL(_LIB_PATH)
        _lib.rlx_encoder_workspace_bytes.restype = C.c_size_t
        _lib.rlx_status_string.restype = C.c_char_p
        _lib.rlx_encoder_destroy.restype = None
    return _lib


def _check(status: int, where: str) -> None:
    if status != RLX_OK:
        raise RlxError(status, where)


def _ptr(t: Optional[torch.Tensor]) -> C.c_void_p:
    return C.c_void_p(0 if t is None else t.data_ptr())


def _stream(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


class DeviceWeights:
    """Device-resident parameter set + the host struct of pointers the ABI takes."""

    def __init__(self, params: Dict[str, torch.Tensor], layers: Sequence[Dict[str, torch.Tensor]]):
        self.params = params
        self.layers = list(layers)
        self._layer_arr = (_Layer * max(len(self.layers), 1))()
        for i, lw in enumerate(self.layers):
            for n in LAYER_FIELDS:
                t = lw[n]
                want = torch.bfloat16 if n in BF16_FIELDS else torch.float32
                assert t.is_cuda and t.is_contiguous() and t.dtype == want, (n, t.dtype)
                setattr(self._layer_arr[i], n, t.data_ptr())
        self.c = _Weights()
        self.c.struct_size = C.sizeof(_Weights)
        for n in ("word_emb", "pos_emb", "type_emb", "emb_ln_g", "emb_ln_b"):
            t = params[n]
            want = torch.bfloat16 if n in BF16_FIELDS else torch.float32
            assert t.is_cuda and t.is_contiguous() and t.dtype == want, (n, t.dtype)
            setattr(self.c, n, t.data_ptr())
        self.c.layers = self._layer_arr


def upload_weights(params, layers, device="cuda") -> DeviceWeights:
    """Copy numpy float32 parameters (matrices already on the bf16 grid) to the device in the
    storage types the ABI expects: bf16 for tables / Linear weights, fp32 for biases and LN."""
    def put(name, a):
        t = torch.from_numpy(a).to(device)
        return t.to(torch.bfloat16).contiguous() if name in BF16_FIELDS else t.float().contiguous()

    p = {n: put(n, params[n]) for n in ("word_emb", "pos_emb", "type_emb", "emb_ln_g", "emb_ln_b")}
    ls = [{n: put(n, lw[n]) for n in LAYER_FIELDS} for lw in layers]
    return DeviceWeights(p, ls)


class Encoder:
    """rlx_encoder_create / _forward / _destroy."""

    def __init__(self, num_layers: int, hidden: int, num_heads: int, ffn: int, vocab: int = 30522,
                 max_pos: int = 512, type_vocab: int = 2, ln_eps: float = 1e-12, max_batch: int = 256,
                 max_seq: int = 512, device: int = 0, flags: int = 0):
        self._h = C.c_void_p()
        self.hidden = hidden
        self.cfg = _Config(C.sizeof(_Config), num_layers, hidden, num_heads, ffn, vocab, max_pos, type_vocab,
                           ln_eps, max_batch, max_seq, device, flags)
        _check(_load().rlx_encoder_create(C.byref(self.cfg), C.byref(self._h)), "rlx_encoder_create")

    @classmethod
    def from_config(cls, cfg, **kw) -> "Encoder":
        kw.setdefault("max_batch", max(cfg.batch, 1))
        kw.setdefault("max_seq", cfg.max_pos)
        return cls(cfg.num_layers, cfg.hidden, cfg.num_heads, cfg.ffn, cfg.vocab, cfg.max_pos, cfg.type_vocab,
                   cfg.ln_eps, **kw)

    def close(self) -> None:
        if self._h:
            _load().rlx_encoder_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def workspace_bytes(self, batch: int, seq: int) -> int:
        return int(_load().rlx_encoder_workspace_bytes(self._h, batch, seq))

    def kernels_per_forward(self, batch: int, seq: int) -> int:
        return int(_load().rlx_encoder_kernels_per_forward(self._h, batch, seq))

    def alloc_workspace(self, batch: int, seq: int, device="cuda") -> torch.Tensor:
        n = self.workspace_bytes(batch, seq)
        if n == 0:
            raise RlxError(1, "rlx_encoder_workspace_bytes")
        return torch.zeros(n, dtype=torch.uint8, device=device)

    def forward(self, ids: torch.Tensor, mask: torch.Tensor, weights: DeviceWeights, out: torch.Tensor,
                workspace: torch.Tensor, stream=None) -> torch.Tensor:
        B, S = ids.shape
        assert ids.dtype == torch.int32 and mask.dtype == torch.int32 and out.dtype == torch.float32
        assert ids.is_cuda and mask.is_cuda and out.is_cuda and ids.is_contiguous() and mask.is_contiguous()
        _check(_load().rlx_encoder_forward(self._h, _ptr(ids), _ptr(mask), B, S, C.byref(weights.c), _ptr(out),
                                           _ptr(workspace), C.c_size_t(workspace.numel()), _stream(stream)),
               "rlx_encoder_forward")
        return out

    def forward_tp(self, ids: torch.Tensor, mask: torch.Tensor, weights_shard: DeviceWeights, tp_rank: int, tp_size: int,
                   allreduce, out: torch.Tensor, workspace: torch.Tensor, stream=None) -> torch.Tensor:
        """rlx_encoder_forward_tp.  `allreduce(view)` receives a bf16 tensor VIEW of the workspace region that
        holds this rank's partial sums and must replace it, in place and ordered on the current stream, by the
        sum over all ranks (e.g. torch.distributed.all_reduce on an NCCL group)."""
        B, S = ids.shape
        assert ids.dtype == torch.int32 and mask.dtype == torch.int32 and out.dtype == torch.float32
        assert ids.is_cuda and mask.is_cuda and out.is_cuda and ids.is_contiguous() and mask.is_contiguous()
        base = workspace.data_ptr()
        failure = []

        def _cb(_user, buf, count, _stream):
            try:
                off = int(buf) - base
                allreduce(workspace[off:off + 2 * int(count)].view(torch.bfloat16))
                return 0
            except Exception as exc:   # an exception must not unwind through the C frames
                failure.append(exc)
                return 1

        cb = ALLREDUCE_FN(_cb)
        status = _load().rlx_encoder_forward_tp(self._h, _ptr(ids), _ptr(mask), B, S, C.byref(weights_shard.c), tp_rank,
                                                tp_size, cb, None, _ptr(out), _ptr(workspace),
                                                C.c_size_t(workspace.numel()), _stream(stream))
        if failure:
            raise failure[0]
        _check(status, "rlx_encoder_forward_tp")
        return out

    def forward_host(self, ids: torch.Tensor, mask: torch.Tensor, weights: DeviceWeights, out: torch.Tensor,
                     workspace: torch.Tensor, stream=None) -> torch.Tensor:
        B, S = ids.shape
        assert not ids.is_cuda and not mask.is_cuda and not out.is_cuda
        assert ids.dtype == torch.int32 and mask.dtype == torch.int32 and out.dtype == torch.float32
        _check(_load().rlx_encoder_forward_host(self._h, _ptr(ids), _ptr(mask), B, S, C.byref(weights.c),
                                                _ptr(out), _ptr(workspace), C.c_size_t(workspace.numel()),
                                                _stream(stream)), "rlx_encoder_forward_host")
        return out

    def forward_static(self, ids: torch.Tensor, mask: torch.Tensor, weights: DeviceWeights, out: torch.Tensor,
                       device_status: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """rlx_encoder_forward_static: the forward for callers that cannot allocate a workspace; the
        scratch lives in a fixed arena inside the library (STATIC_WORKSPACE_BYTES), shared by all
        calls, so calls must not overlap on the GPU.  Raises RlxError(RLX_ERR_WORKSPACE) when
        (batch, seq) needs more than the arena holds."""
        B, S = ids.shape
        assert ids.dtype == torch.int32 and mask.dtype == torch.int32 and out.dtype == torch.float32
        assert ids.is_cuda and mask.is_cuda and out.is_cuda and ids.is_contiguous() and mask.is_contiguous()
        _check(_load().rlx_encoder_forward_static(self._h, _ptr(ids), _ptr(mask), B, S, C.byref(weights.c),
                                                  _ptr(out), _ptr(device_status), _stream(stream)),
               "rlx_encoder_forward_static")
        return out

    def kernel_times(self, batch: int, seq: int) -> List[float]:
        """Milliseconds per kernel of the last forward (encoder created with FLAG_KERNEL_EVENTS)."""
        n = self.kernels_per_forward(batch, seq)
        buf = (C.c_float * n)()
        _check(_load().rlx_encoder_kernel_times(self._h, buf, n), "rlx_encoder_kernel_times")
        return list(buf)

    def last_device_status(self, workspace: torch.Tensor, stream=None) -> int:
        return int(_load().rlx_encoder_last_device_status(self._h, _ptr(workspace), _stream(stream)))


# ------------------------------------------------------------------ kernel-level entry points
def embed_layernorm(ids, word, pos, type_, gamma, beta, seq: int, vocab: int, eps: float, status=None, stream=None):
    T, H = ids.numel(), word.shape[1]
    out = torch.empty((T, H), dtype=torch.bfloat16, device=ids.device)
    _check(_load().rlx_embed_layernorm(_ptr(ids), _ptr(word), _ptr(pos), _ptr(type_), _ptr(gamma), _ptr(beta), T, seq,
                                       H, vocab, C.c_float(eps), _ptr(out), _ptr(status), _stream(stream)),
           "rlx_embed_layernorm")
    return out


def pack_sequences(mask: torch.Tensor, stream=None):
    """rlx_pack_sequences -> (seq_len [B], seq_start [B+1], pos_of_rank [B,S]) int32 device tensors."""
    B, S = mask.shape
    seq_len = torch.empty(B, dtype=torch.int32, device=mask.device)
    seq_start = torch.empty(B + 1, dtype=torch.int32, device=mask.device)
    pos_of_rank = torch.full((B, S), -1, dtype=torch.int32, device=mask.device)
    ticket = torch.zeros(1, dtype=torch.int32, device=mask.device)
    _check(_load().rlx_pack_sequences(_ptr(mask), B, S, _ptr(seq_len), _ptr(seq_start), _ptr(pos_of_rank),
                                      _ptr(ticket), _stream(stream)), "rlx_pack_sequences")
    return seq_len, seq_start, pos_of_rank, ticket


def layernorm(x, gamma, beta, eps: float, stream=None):
    rows, H = x.shape
    out = torch.empty_like(x)
    _check(_load().rlx_layernorm(_ptr(x), _ptr(gamma), _ptr(beta), rows, H, C.c_float(eps), _ptr(out), _stream(stream)),
           "rlx_layernorm")
    return out


def gemm_bf16(a, w, bias, residual=None, epilogue: int = EPI_BIAS, impl: int = GEMM_TCGEN05, status=None, stream=None):
    M, K = a.shape
    N = w.shape[0]
    out = torch.empty((M, N), dtype=torch.bfloat16, device=a.device)
    _check(_load().rlx_gemm_bf16(_ptr(a), _ptr(w), _ptr(bias), _ptr(residual), epilogue, M, N, K, _ptr(out), impl,
                                 _ptr(status), _stream(stream)), "rlx_gemm_bf16")
    return out


def gemm_residual_layernorm_bf16(a, w, bias, residual, gamma, beta, eps: float, impl: int = 0, status=None, stream=None):
    M, K = a.shape
    N = w.shape[0]
    out = torch.empty((M, N), dtype=torch.bfloat16, device=a.device)
    _check(_load().rlx_gemm_residual_layernorm_bf16(_ptr(a), _ptr(w), _ptr(bias), _ptr(residual), _ptr(gamma),
                                                    _ptr(beta), C.c_float(eps), M, N, K, _ptr(out), impl, _ptr(status),
                                                    _stream(stream)), "rlx_gemm_residual_layernorm_bf16")
    return out


def attention_bf16(qkv, mask, num_heads: int, stream=None):
    B, S, H3 = qkv.shape
    H = H3 // 3
    ctx = torch.empty((B, S, H), dtype=torch.bfloat16, device=qkv.device)
    _check(_load().rlx_attention_bf16(_ptr(qkv), _ptr(mask), B, S, num_heads, H // num_heads, _ptr(ctx), _stream(stream)),
           "rlx_attention_bf16")
    return ctx


def attention_packed_bf16(qkv, seq_start, seq_len, max_len: int, num_heads: int, impl: int = 0, status=None, stream=None):
    """qkv: packed [rows, 3H] bf16; returns ctx [rows, H] (rows outside every sequence stay zero)."""
    rows, H3 = qkv.shape
    H = H3 // 3
    ctx = torch.zeros((rows, H), dtype=torch.bfloat16, device=qkv.device)
    _check(_load().rlx_attention_packed_bf16(_ptr(qkv), rows, _ptr(seq_start), _ptr(seq_len), seq_len.numel(), max_len,
                                             num_heads, H // num_heads, _ptr(ctx), impl, _ptr(status), _stream(stream)),
           "rlx_attention_packed_bf16")
    return ctx


MASK_NONE, MASK_CAUSAL, MASK_SLIDING_WINDOW = 0, 1, 2
ATTENTION_KIND_MAX_LEN = 32768


def rope_tables(max_len: int, head_dim: int, theta: float = 10000.0, device="cuda", stream=None):
    """rlx_rope_tables: cos / sin of position * theta^(-2j/head_dim) as fp32 device tables
    [max_len, head_dim/2] (the constant inputs rlx_attention_kind_bf16 takes), built by the library."""
    cos = torch.empty((max_len, head_dim // 2), dtype=torch.float32, device=device)
    sin = torch.empty_like(cos)
    _check(_load().rlx_rope_tables(max_len, head_dim, C.c_double(theta), _ptr(cos), _ptr(sin), _stream(stream)),
           "rlx_rope_tables")
    return cos, sin


def attention_kind_bf16(qkv, seq_start, seq_len, max_len: int, num_heads: int, mask_kind: int, window: int = 0,
                        rope=None, out=None, stream=None, num_kv_heads: Optional[int] = None):
    """qkv: packed [rows, (hq + 2 hkv) d] bf16 (hkv = hq unless num_kv_heads is given); rope: None or the
    (cos, sin) pair of rope_tables; returns ctx [rows, hq d] (a fresh zero-filled tensor, or `out` with rows
    outside every sequence left as they were)."""
    rows, W = qkv.shape
    hkv = num_heads if num_kv_heads is None else num_kv_heads
    d = W // (num_heads + 2 * hkv)
    ctx = torch.zeros((rows, num_heads * d), dtype=torch.bfloat16, device=qkv.device) if out is None else out
    cos, sin = rope if rope is not None else (None, None)
    _check(_load().rlx_attention_kind_bf16(_ptr(qkv), rows, _ptr(seq_start), _ptr(seq_len), seq_len.numel(), max_len,
                                           num_heads, hkv, d, mask_kind, window, _ptr(cos), _ptr(sin),
                                           _ptr(ctx), _stream(stream)),
           "rlx_attention_kind_bf16")
    return ctx


def qk_rope_bf16(qkv, seq_start, seq_len, max_len: int, num_heads: int, rope, stream=None,
                 num_kv_heads: Optional[int] = None):
    """Rotates the q and k column blocks of packed qkv [rows, (hq + 2 hkv) d] bf16 IN PLACE; returns qkv."""
    rows, W = qkv.shape
    hkv = num_heads if num_kv_heads is None else num_kv_heads
    cos, sin = rope
    _check(_load().rlx_qk_rope_bf16(_ptr(qkv), rows, _ptr(seq_start), _ptr(seq_len), seq_len.numel(), max_len, num_heads,
                                    hkv, W // (num_heads + 2 * hkv), _ptr(cos), _ptr(sin), _stream(stream)),
           "rlx_qk_rope_bf16")
    return qkv


def selftest_bounded_wait(budget_us: int, status_word: torch.Tensor, waited_ns: Optional[torch.Tensor] = None, stream=None):
    """Runs the bounded-wait self-test kernel; status_word: int32 device tensor, waited_ns: int64 device tensor."""
    _check(_load().rlx_selftest_bounded_wait(C.c_uint32(budget_us), _ptr(status_word), _ptr(waited_ns), _stream(stream)),
           "rlx_selftest_bounded_wait")


def minifloat(ebits: int, mbits: int, special: int = 0, packed4: bool = False) -> int:
    """Format word of rlx_dequant_block_scaled_bf16 (special: 0 none, 1 all-ones magnitude NaN, 2 IEEE)."""
    return (ebits << 8) | (mbits << 4) | special | (0x1000 if packed4 else 0)


FMT_FP8_E4M3, FMT_FP8_E5M2 = minifloat(4, 3, 1), minifloat(5, 2, 2)
FMT_FP6_E3M2, FMT_FP6_E2M3 = minifloat(3, 2, 0), minifloat(2, 3, 0)
FMT_FP4_E2M1 = minifloat(2, 1, 0, packed4=True)


def dequant_block_scaled_bf16(codes, scales, N: int, K: int, fmt: int, out=None, stream=None):
    """codes uint8 [N,K] (or [N,K/2] packed nibbles), scales uint8 [N,K/32] -> W bf16 [N,K]."""
    w = torch.empty((N, K), dtype=torch.bfloat16, device=codes.device) if out is None else out
    _check(_load().rlx_dequant_block_scaled_bf16(_ptr(codes), _ptr(scales), N, K, fmt, _ptr(w), _stream(stream)),
           "rlx_dequant_block_scaled_bf16")
    return w


def scaled_matmul_bf16(a, codes, scales, fmt: int, bias, residual=None, epilogue: int = EPI_BIAS, w_scratch=None,
                       out=None, status=None, stream=None):
    """out bf16 [M,N] = epilogue(a [M,K] . dequant(codes, scales)^T + bias); N = rows of codes."""
    M, K = a.shape
    N = codes.shape[0]
    w = torch.empty((N, K), dtype=torch.bfloat16, device=a.device) if w_scratch is None else w_scratch
    out = torch.empty((M, N), dtype=torch.bfloat16, device=a.device) if out is None else out
    _check(_load().rlx_scaled_matmul_bf16(_ptr(a), _ptr(codes), _ptr(scales), fmt, _ptr(bias), _ptr(residual), epilogue,
                                          M, N, K, _ptr(w), _ptr(out), _ptr(status), _stream(stream)),
           "rlx_scaled_matmul_bf16")
    return out


def ffn_fused_bf16(x, w1, b1, w2, b2, ln_gamma=None, ln_beta=None, ln_eps=0.0, out=None, status=None, stream=None):
    """rlx_ffn_fused_bf16: out [M,H] = gelu(x w1^T + b1) w2^T + b2 + x in one kernel, through LayerNorm when
    ln_gamma / ln_beta are given."""
    M, H = x.shape
    F = w1.shape[0]
    out = torch.empty((M, H), dtype=torch.bfloat16, device=x.device) if out is None else out
    _check(_load().rlx_ffn_fused_bf16(_ptr(x), _ptr(w1), _ptr(b1), _ptr(w2), _ptr(b2), _ptr(ln_gamma), _ptr(ln_beta),
                                      C.c_float(ln_eps), M, H, F, _ptr(out), _ptr(status),
                                      _stream(stream)), "rlx_ffn_fused_bf16")
    return out


def layer_tail_bf16(ctx, h, wo, bo, ln1_gamma, ln1_beta, w1, b1, w2, b2, ln2_gamma, ln2_beta, ln_eps, out=None, status=None,
                    stream=None):
    """rlx_layer_tail_bf16: out-projection + residual + LayerNorm + feed-forward block + residual + LayerNorm of an
    encoder layer in one kernel; ctx, h, out bf16 [M,H]."""
    M, H = ctx.shape
    F = w1.shape[0]
    out = torch.empty((M, H), dtype=torch.bfloat16, device=ctx.device) if out is None else out
    _check(_load().rlx_layer_tail_bf16(_ptr(ctx), _ptr(h), _ptr(wo), _ptr(bo), _ptr(ln1_gamma), _ptr(ln1_beta), _ptr(w1),
                                       _ptr(b1), _ptr(w2), _ptr(b2), _ptr(ln2_gamma), _ptr(ln2_beta), C.c_float(ln_eps),
                                       M, H, F, _ptr(out), _ptr(status), _stream(stream)), "rlx_layer_tail_bf16")
    return out


def quantise_mx(x, fmt: int, stream=None):
    """rlx_quantise_mx: x bf16 [M,K] -> (codes uint8 [M,K], scales uint8 [M,K/32])."""
    M, K = x.shape
    codes = torch.empty((M, K), dtype=torch.uint8, device=x.device)
    scales = torch.empty((M, K // 32), dtype=torch.uint8, device=x.device)
    _check(_load().rlx_quantise_mx(_ptr(x), M, K, fmt, _ptr(codes), _ptr(scales), _stream(stream)), "rlx_quantise_mx")
    return codes, scales


def mx_matmul_bf16(a_codes, a_scales, a_fmt: int, w_codes, w_scales, w_fmt: int, bias=None, out=None, status=None,
                   stream=None):
    """rlx_mx_matmul_bf16: out bf16 [M,N] = A W^T (+ bias), both operands block-scaled FP8."""
    M, K = a_codes.shape
    N = w_codes.shape[0]
    out = torch.empty((M, N), dtype=torch.bfloat16, device=a_codes.device) if out is None else out
    _check(_load().rlx_mx_matmul_bf16(_ptr(a_codes), _ptr(a_scales), a_fmt, _ptr(w_codes), _ptr(w_scales), w_fmt,
                                      _ptr(bias), M, N, K, _ptr(out), _ptr(status), _stream(stream)),
           "rlx_mx_matmul_bf16")
    return out


def attention_f32(qkv, mask, num_heads: int, stream=None):
    B, S, H3 = qkv.shape
    H = H3 // 3
    ctx = torch.empty((B, S, H), dtype=torch.float32, device=qkv.device)
    _check(_load().rlx_attention_f32(_ptr(qkv), _ptr(mask), B, S, num_heads, H // num_heads, _ptr(ctx), _stream(stream)),
           "rlx_attention_f32")
    return ctx


def pool_l2norm(x, mask, stream=None):
    B, S, H = x.shape
    out = torch.empty((B, H), dtype=torch.float32, device=x.device)
    _check(_load().rlx_pool_l2norm(_ptr(x), _ptr(mask), B, S, H, _ptr(out), _stream(stream)), "rlx_pool_l2norm")
    return out
