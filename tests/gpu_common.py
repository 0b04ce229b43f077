"""Helpers shared by the GPU parity tests (not a test module)."""
import numpy as np
import torch

from synth.inputs import round_to_bf16


def bf16_dev(a: np.ndarray) -> torch.Tensor:
    """float32 values on the bf16 grid -> device bf16 tensor (exact)."""
    return torch.from_numpy(np.ascontiguousarray(a, np.float32)).cuda().to(torch.bfloat16).contiguous()


def f32_dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, np.float32)).cuda().contiguous()


def i32_dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, np.int32)).cuda().contiguous()


def to_np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def rand_bf16(rng, shape, scale=1.0) -> np.ndarray:
    return round_to_bf16((rng.standard_normal(shape) * scale).astype(np.float32))


def cosine_rows(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    num = (a * b).sum(-1)
    den = np.linalg.norm(a, axis=-1) * np.linalg.norm(b, axis=-1)
    return num / np.maximum(den, 1e-300)


# unit round-off of bf16 (8 significand bits, round to nearest): 2^-9
BF16_U = 2.0 ** -9
