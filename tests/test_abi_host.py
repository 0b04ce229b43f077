"""Host-side checks of the C ABI that need no GPU: the library loads, exports every
symbol the header declares, validates arguments before any launch, and sizes the workspace."""
import ctypes as C
import os
import re

import pytest

from paper_2609_37916_b200 import binding
from paper_2609_37916_b200.build import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build()
    return binding._load()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "rlx_encoder.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(rlx_[a-z0-9_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS), declared ^ set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    seen = {lib.rlx_status_string(i).decode() for i in range(7)}
    assert len(seen) == 7 and "ok" in seen
    assert lib.rlx_status_string(99).decode() == "unknown status"


def _cfg(**kw):
    base = dict(num_layers=6, hidden=384, num_heads=12, ffn=1536, vocab=30522, max_pos=512, type_vocab=2,
                ln_eps=1e-12, max_batch=32, max_seq=128, device=0, flags=0)
    base.update(kw)
    return base


def test_create_validates_shapes(lib):
    enc = binding.Encoder(**_cfg(max_batch=256))
    assert enc.kernels_per_forward(32, 128) == 3 + 5 * 6   # small batch: LayerNorm folded into the GEMMs automatically
    assert enc.kernels_per_forward(100, 128) == 3 + 7 * 6  # packing + embed + 7 per layer + pool
    assert enc.kernels_per_forward(128, 128) == 3 + 7 * 6
    assert enc.kernels_per_forward(256, 128) == 3 + 3 * 6  # from 32768 padded tokens on: everything behind the attention in one kernel
    enc.close()
    for bad, status in [
        (dict(hidden=400, num_heads=10), 2),    # H % 128
        (dict(hidden=384, num_heads=8), 2),     # head_dim 48
        (dict(hidden=2048, num_heads=32), 2),   # H > 1024
        (dict(ffn=1000), 2),                    # F % 64
        (dict(max_seq=1024, max_pos=512), 2),   # seq > max_pos
        (dict(num_layers=0), 1),
        (dict(max_batch=-1), 1),
    ]:
        with pytest.raises(binding.RlxError) as ei:
            binding.Encoder(**_cfg(**bad))
        assert ei.value.status == status, bad


def test_kernel_count_follows_the_layernorm_fusion_flags(lib):
    enc = binding.Encoder(**_cfg(max_batch=256, max_seq=256))
    assert enc.kernels_per_forward(256, 256) == 3 + 3 * 6     # default: QKV GEMM, attention, and one kernel for the rest of the layer
    enc.close()
    two = binding.Encoder(**_cfg(max_batch=256, max_seq=256, flags=binding.FLAG_NO_FUSED_FFN))
    assert two.kernels_per_forward(256, 256) == 3 + 7 * 6
    two.close()
    one = binding.Encoder(**_cfg(max_batch=256, max_seq=256, flags=binding.FLAG_FUSED_FFN | binding.FLAG_NO_AUTO_FOLD))
    assert one.kernels_per_forward(8, 64) == 3 + 3 * 6        # forced at every size
    one.close()
    cl = binding.Encoder(**_cfg(max_batch=256, max_seq=256, flags=binding.FLAG_CLUSTER_LN))
    assert cl.kernels_per_forward(256, 256) == 3 + 5 * 6      # folded into the GEMMs (cluster statistics)
    assert cl.kernels_per_forward(1, 16) == 3 + 5 * 6
    cl.close()
    whole = binding.Encoder(**_cfg(max_batch=256, max_seq=256, flags=binding.FLAG_FUSED_LN))
    assert whole.kernels_per_forward(256, 256) == 3 + 5 * 6   # whole-row variant: enough 128-row tiles for every SM
    assert whole.kernels_per_forward(32, 128) == 3 + 7 * 6    # an explicit fusion flag switches the automatic fold off
    whole.close()
    big = binding.Encoder(**_cfg(hidden=768, num_heads=12, ffn=3072, max_batch=64, max_seq=512,
                                 flags=binding.FLAG_CLUSTER_LN))
    assert big.kernels_per_forward(64, 512) == 3 + 5 * 6      # 768 = 4 slabs of 192 columns per cluster
    big.close()


def test_create_rejects_wrong_struct_size_and_null(lib):
    cfg = binding._Config(4, 6, 384, 12, 1536, 30522, 512, 2, 1e-12, 32, 128, 0, 0)
    h = C.c_void_p()
    assert lib.rlx_encoder_create(C.byref(cfg), C.byref(h)) == 1
    assert lib.rlx_encoder_create(None, C.byref(h)) == 1
    lib.rlx_encoder_destroy(None)  # no-op


def test_workspace_bytes_layout(lib):
    enc = binding.Encoder(**_cfg(max_batch=256, max_seq=256))
    T, H, F = 256 * 256, 384, 1536
    need = enc.workspace_bytes(256, 256)
    acts = T * (H + 3 * H + H + H + H + F) * 2
    assert acts <= need <= acts + 3 * T * 4 + (1 << 20)
    assert need % 256 == 0
    assert enc.workspace_bytes(257, 256) == 0 and enc.workspace_bytes(1, 0) == 0
    assert enc.workspace_bytes(1, 16) < enc.workspace_bytes(2, 16)
    enc.close()


def test_forward_rejects_bad_arguments_before_touching_the_device(lib):
    enc = binding.Encoder(**_cfg())
    w = binding._Weights()
    w.struct_size = C.sizeof(binding._Weights)
    fake = C.c_void_p(0x1000)
    # null pointers
    assert lib.rlx_encoder_forward(enc._h, None, fake, 1, 16, C.byref(w), fake, fake, C.c_size_t(1 << 30), None) == 1
    # sizes outside the configured bounds
    assert lib.rlx_encoder_forward(enc._h, fake, fake, 64, 16, C.byref(w), fake, fake, C.c_size_t(1 << 30), None) == 1
    assert lib.rlx_encoder_forward(enc._h, fake, fake, 1, 129, C.byref(w), fake, fake, C.c_size_t(1 << 30), None) == 1
    # weights struct without layers
    assert lib.rlx_encoder_forward(enc._h, fake, fake, 1, 16, C.byref(w), fake, fake, C.c_size_t(1 << 30), None) == 1
    # misaligned workspace / ids
    layers = (binding._Layer * 6)()
    for l in layers:
        for n in binding.LAYER_FIELDS:
            setattr(l, n, 0x2000)
    w.layers = layers
    for n in ("word_emb", "pos_emb", "type_emb", "emb_ln_g", "emb_ln_b"):
        setattr(w, n, 0x2000)
    assert lib.rlx_encoder_forward(enc._h, fake, fake, 1, 16, C.byref(w), fake, C.c_void_p(0x1010),
                                   C.c_size_t(1 << 30), None) == 1
    assert lib.rlx_encoder_forward(enc._h, C.c_void_p(0x1004), fake, 1, 16, C.byref(w), fake, fake,
                                   C.c_size_t(1 << 30), None) == 1
    # workspace too small
    assert lib.rlx_encoder_forward(enc._h, fake, fake, 1, 16, C.byref(w), fake, fake, C.c_size_t(1024), None) == 3
    # a null weight pointer inside a layer
    layers[3].w2 = 0
    assert lib.rlx_encoder_forward(enc._h, fake, fake, 1, 16, C.byref(w), fake, fake, C.c_size_t(1 << 30), None) == 1
    enc.close()


def test_kernel_entry_points_validate_on_the_host(lib):
    fake = C.c_void_p(0x1000)
    assert lib.rlx_layernorm(fake, fake, fake, 4, 100, C.c_float(1e-12), fake, None) == 2   # H % 128
    assert lib.rlx_layernorm(None, fake, fake, 4, 128, C.c_float(1e-12), fake, None) == 1
    assert lib.rlx_gemm_bf16(fake, fake, fake, None, 0, 8, 100, 64, fake, 0, None, None) == 2  # N % 64
    assert lib.rlx_gemm_bf16(fake, fake, fake, None, 0, 8, 128, 60, fake, 0, None, None) == 2  # K % 8
    assert lib.rlx_gemm_bf16(fake, fake, fake, None, 2, 8, 128, 64, fake, 0, None, None) == 1  # residual missing
    assert lib.rlx_attention_bf16(fake, fake, 1, 16, 12, 48, fake, None) == 2                   # head_dim
    assert lib.rlx_attention_bf16(fake, fake, 1, 1024, 12, 32, fake, None) == 2                 # seq > 512
    assert lib.rlx_attention_f32(fake, fake, 0, 16, 12, 32, fake, None) == 1
    assert lib.rlx_pool_l2norm(fake, fake, 1, 16, 100, fake, None) == 2
    assert lib.rlx_embed_layernorm(fake, fake, fake, fake, fake, fake, 16, 16, 2048, 100, C.c_float(0), fake,
                                   None, None) == 2


def test_attention_kind_validates_on_the_host(lib):
    fake, odd = C.c_void_p(0x1000), C.c_void_p(0x1004)
    call = lib.rlx_attention_kind_bf16
    ok_args = dict(rows=64, batch=1, max_len=64, h=2, hkv=2, d=32, kind=1, window=0, cos=None, sin=None)

    def run(qkv=fake, start=fake, length=fake, ctx=fake, **kw):
        a = dict(ok_args, **kw)
        return call(qkv, a["rows"], start, length, a["batch"], a["max_len"], a["h"], a["hkv"], a["d"], a["kind"],
                    a["window"], a["cos"], a["sin"], ctx, None)

    assert run(qkv=None) == 1 and run(start=None) == 1 and run(length=None) == 1 and run(ctx=None) == 1
    assert run(rows=0) == 1 and run(batch=0) == 1 and run(max_len=0) == 1
    assert run(kind=3) == 1 and run(kind=-1) == 1
    assert run(kind=2, window=0) == 1                      # sliding window needs w >= 1
    assert run(cos=fake, sin=None) == 1 and run(cos=None, sin=fake) == 1   # a lone table
    assert run(cos=odd, sin=fake) == 1                     # misaligned table
    assert run(h=6, hkv=4) == 1 and run(hkv=0) == 1       # k/v heads must divide the q heads
    assert run(d=48) == 2 and run(d=256) == 2              # head sizes other than 32 / 64 / 128
    assert run(max_len=32769) == 2                         # beyond RLX_ATTENTION_KIND_MAX_LEN


def test_qk_rope_validates_on_the_host(lib):
    fake, odd = C.c_void_p(0x1000), C.c_void_p(0x1008)
    call = lib.rlx_qk_rope_bf16
    assert call(None, 8, fake, fake, 1, 8, 2, 2, 32, fake, fake, None) == 1
    assert call(fake, 8, fake, fake, 1, 8, 2, 2, 32, None, fake, None) == 1      # both tables are required
    assert call(fake, 8, fake, fake, 1, 8, 2, 2, 32, fake, odd, None) == 1       # misaligned table
    assert call(fake, 0, fake, fake, 1, 8, 2, 2, 32, fake, fake, None) == 1
    assert call(fake, 8, fake, fake, 1, 8, 3, 2, 32, fake, fake, None) == 1      # 2 k/v heads do not divide 3
    assert call(fake, 8, fake, fake, 1, 8, 2, 2, 48, fake, fake, None) == 2      # head size
    assert call(fake, 8, fake, fake, 1, 40000, 2, 2, 32, fake, fake, None) == 2  # beyond the maximum length


def test_scaled_matmul_validates_on_the_host(lib):
    fake, odd = C.c_void_p(0x1000), C.c_void_p(0x1001)
    fmt = lambda e, m, s=0, p=False: (e << 8) | (m << 4) | s | (0x1000 if p else 0)
    dq = lib.rlx_dequant_block_scaled_bf16
    assert dq(None, fake, 8, 32, fmt(4, 3, 1), fake, None) == 1
    assert dq(odd, fake, 8, 32, fmt(4, 3, 1), fake, None) == 1                 # misaligned codes
    assert dq(fake, fake, 8, 32, fmt(0, 3), fake, None) == 1                    # no exponent bits
    assert dq(fake, fake, 8, 32, fmt(5, 3), fake, None) == 1                    # 9-bit code in a byte
    assert dq(fake, fake, 8, 32, fmt(2, 2, 0, True), fake, None) == 1           # 5-bit code in a nibble
    assert dq(fake, fake, 8, 32, fmt(4, 3, 3), fake, None) == 1                 # unknown special mode
    assert dq(fake, fake, 8, 48, fmt(4, 3, 1), fake, None) == 2                 # K % 32
    sm = lib.rlx_scaled_matmul_bf16
    assert sm(fake, fake, fake, fmt(4, 3, 1), fake, None, 2, 8, 64, 32, fake, fake, None, None) == 1   # residual missing
    assert sm(fake, fake, fake, fmt(4, 3, 1), fake, None, 0, 8, 100, 32, fake, fake, None, None) == 2  # N % 64
    assert sm(fake, fake, fake, fmt(4, 3, 1), fake, None, 0, 8, 64, 32, None, fake, None, None) == 1   # no scratch


def test_layer_tail_and_fused_ffn_validate_on_the_host(lib):
    fake, odd = C.c_void_p(0x1000), C.c_void_p(0x1008)
    eps = C.c_float(1e-12)
    ffn = lib.rlx_ffn_fused_bf16
    assert ffn(fake, fake, fake, fake, fake, None, None, C.c_float(0), 8, 384, 1536, None, None, None) == 1      # no output
    assert ffn(fake, fake, fake, fake, fake, fake, None, eps, 8, 384, 1536, fake, None, None) == 1               # gamma without beta
    assert ffn(fake, fake, fake, fake, fake, fake, fake, C.c_float(0), 8, 384, 1536, fake, None, None) == 1      # LayerNorm needs eps > 0
    assert ffn(odd, fake, fake, fake, fake, None, None, C.c_float(0), 8, 384, 1536, fake, None, None) == 1       # misaligned x
    assert ffn(fake, fake, fake, fake, fake, None, None, C.c_float(0), 8, 512, 2048, fake, None, None) == 2      # hidden 512: no room in tensor memory
    assert ffn(fake, fake, fake, fake, fake, None, None, C.c_float(0), 8, 384, 1600, fake, None, None) == 2      # F % 128
    tail = lib.rlx_layer_tail_bf16
    args = [fake] * 12
    assert tail(*args, eps, 8, 384, 1536, None, None, None) == 1
    assert tail(*args, C.c_float(0), 8, 384, 1536, fake, None, None) == 1
    assert tail(*(args[:5] + [None] + args[6:]), eps, 8, 384, 1536, fake, None, None) == 1                        # a LayerNorm vector missing
    assert tail(*args, eps, 8, 768, 3072, fake, None, None) == 2
    assert tail(*args, eps, 0, 384, 1536, fake, None, None) == 1
