"""B200 (sm_100a) masked transformer-encoder forward behind a C ABI.

``binding`` is a thin ctypes layer over ``librlx_encoder.so`` (same names as
``include/rlx_encoder.h``); it only marshals arguments.  There is no CPU or
library fallback: if the shared library has not been built, importing the
binding raises.
"""
from .binding import (  # noqa: F401
    DeviceWeights,
    Encoder,
    RlxError,
    attention_bf16,
    attention_f32,
    attention_kind_bf16,
    attention_packed_bf16,
    dequant_block_scaled_bf16,
    embed_layernorm,
    ffn_fused_bf16,
    layer_tail_bf16,
    gemm_bf16,
    gemm_residual_layernorm_bf16,
    layernorm,
    mx_matmul_bf16,
    quantise_mx,
    pack_sequences,
    lib_path,
    pool_l2norm,
    qk_rope_bf16,
    rope_tables,
    scaled_matmul_bf16,
    upload_weights,
)
