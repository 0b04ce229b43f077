"""fp64 statement of the block-scaled minifloat matmul ("ScaledMatMul").

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's CPU-baseline leg may import this
module; the product path never does, and it shares no code with the CUDA kernels.

What it follows.  Section 3.2 (numeric precision) lists weight-only quantisation down to "block-scaled
tensor-core minifloats -- the FP8/FP6/FP4 grids and arbitrary fNeXmY formats, selectable per matmul";
Section 6 names the operator (ScaledMatMul) and its bar: agreement with the F32 reference on the
dequantised grid.  The paper gives no layout, block size or scale format; the readings used here are
those of the open microscaling (MX) convention its llama.cpp scheme list also names:

  element    a minifloat code with 1 sign bit, X exponent bits, Y mantissa bits, exponent bias
             2^(X-1) - 1, gradual underflow (exponent field 0: subnormal, value = mantissa * 2^(1-bias-Y)).
             Special codes, by format:  "none"  every code is a finite number (FP4 E2M1, FP6 E2M3 / E3M2
             and generic fNeXmY);  "nan_only"  the all-ones magnitude is NaN, nothing is infinite
             (FP8 E4M3);  "ieee"  the top exponent is infinity (mantissa 0) or NaN (FP8 E5M2).
  block      32 consecutive elements along the contraction dimension K share one scale.
  scale      an E8M0 byte e: the power of two 2^(e - 127); e = 255 is NaN.
  weight     W[n, k] = value(code[n, k]) * 2^(scale[n, k // 32] - 127), a real number; the matmul is
             y = x W^T (+ bias) on those reals.

Everything here is the definition in IEEE double precision (every weight on these grids is exactly
representable in a double).
"""
from __future__ import annotations

from typing import NamedTuple, Optional

import numpy as np

BLOCK = 32


class MiniFloat(NamedTuple):
    ebits: int
    mbits: int
    special: str          # "none" | "nan_only" | "ieee"


E4M3 = MiniFloat(4, 3, "nan_only")
E5M2 = MiniFloat(5, 2, "ieee")
E3M2 = MiniFloat(3, 2, "none")
E2M3 = MiniFloat(2, 3, "none")
E2M1 = MiniFloat(2, 1, "none")


def decode_table(fmt: MiniFloat) -> np.ndarray:
    """value of every code 0 .. 2^(1+X+Y) - 1 (sign is the top bit)."""
    X, Y = fmt.ebits, fmt.mbits
    bias = 2 ** (X - 1) - 1
    out = np.empty(2 ** (1 + X + Y))
    for code in range(out.size):
        sign = -1.0 if code >> (X + Y) else 1.0
        e = (code >> Y) & (2 ** X - 1)
        m = code & (2 ** Y - 1)
        if fmt.special == "ieee" and e == 2 ** X - 1:
            v = np.inf if m == 0 else np.nan
        elif fmt.special == "nan_only" and e == 2 ** X - 1 and m == 2 ** Y - 1:
            v = np.nan
        elif e == 0:
            v = m * 2.0 ** (1 - bias - Y)
        else:
            v = (1.0 + m * 2.0 ** -Y) * 2.0 ** (e - bias)
        out[code] = sign * v
    return out


def scale_value(e8m0: np.ndarray) -> np.ndarray:
    e = np.asarray(e8m0).astype(np.int64)
    return np.where(e == 255, np.nan, np.ldexp(1.0, e - 127))


def dequantise(codes: np.ndarray, scales: np.ndarray, fmt: MiniFloat) -> np.ndarray:
    """codes [N, K] (one code per entry), scales [N, K/32] E8M0 bytes -> W [N, K] in fp64."""
    codes = np.asarray(codes)
    N, K = codes.shape
    assert K % BLOCK == 0 and np.asarray(scales).shape == (N, K // BLOCK)
    vals = decode_table(fmt)[codes.astype(np.int64)]
    return vals * np.repeat(scale_value(scales), BLOCK, axis=1)


def unpack_nibbles(packed: np.ndarray) -> np.ndarray:
    """[N, K/2] bytes -> [N, K] 4-bit codes; the low nibble holds the element with the smaller k."""
    packed = np.asarray(packed, np.uint8)
    out = np.empty((packed.shape[0], packed.shape[1] * 2), np.uint8)
    out[:, 0::2] = packed & 0xF
    out[:, 1::2] = packed >> 4
    return out


def scaled_matmul(x: np.ndarray, codes: np.ndarray, scales: np.ndarray, fmt: MiniFloat,
                  bias: Optional[np.ndarray] = None) -> np.ndarray:
    """y [M, N] = x [M, K] W^T (+ bias), W = dequantise(codes, scales)."""
    y = np.asarray(x, np.float64) @ dequantise(codes, scales, fmt).T
    return y if bias is None else y + np.asarray(bias, np.float64)


# ------------------------------------------------------------------------------------------------
# Quantised ACTIVATIONS (a reading: Section 3.2 is weight-only).  The tensor cores' block-scaled
# product takes BOTH operands as (element codes, one E8M0 scale per 32 elements along K), so running
# ScaledMatMul on that path needs a rule that puts a real activation row on such a grid.  The rule used
# is the microscaling convention's, per block of 32 consecutive elements of a row:
#   shared exponent  s = floor(log2(max |x_i|)) - emax(fmt),   emax = exponent of the largest finite
#                    element value (8 for E4M3: 448 = 1.75 * 2^8; 15 for E5M2);  clamped to the E8M0
#                    range [-127, 127];  an all-zero block takes s = 0
#   element          code of the grid value nearest to x_i / 2^s, ties to the even code, values beyond
#                    the largest finite element saturate to it (keeping the sign); never NaN / inf codes
# and the quantised activation is value(code) * 2^s.  Everything below is that definition in fp64.

def emax(fmt: MiniFloat) -> int:
    t = decode_table(fmt)
    return int(np.floor(np.log2(np.nanmax(t[np.isfinite(t)]))))


def _finite_grid(fmt: MiniFloat):
    """(values, codes) of the non-negative finite codes, ascending."""
    t = decode_table(fmt)
    half = t.size // 2
    codes = np.array([c for c in range(half) if np.isfinite(t[c])])
    return t[codes], codes


def quantise_elements(v: np.ndarray, fmt: MiniFloat) -> np.ndarray:
    """Nearest code on the element grid for every real v (ties to the even code, saturating)."""
    vals, codes = _finite_grid(fmt)
    v = np.asarray(v, np.float64)
    mag = np.minimum(np.abs(v), vals[-1])
    hi = np.searchsorted(vals, mag, side="left").clip(0, vals.size - 1)     # first grid value >= mag
    lo = np.maximum(hi - 1, 0)
    d_hi, d_lo = vals[hi] - mag, mag - vals[lo]
    take_lo = (d_lo < d_hi) | ((d_lo == d_hi) & (codes[lo] % 2 == 0))
    pick = np.where(take_lo, lo, hi)
    sign_bit = fmt.ebits + fmt.mbits
    return (codes[pick] | (np.signbit(v).astype(np.int64) << sign_bit)).astype(np.uint8)


def quantise_mx(x: np.ndarray, fmt: MiniFloat):
    """x [M, K] real -> (codes [M, K] uint8, scales [M, K/32] E8M0 bytes) by the rule above."""
    x = np.asarray(x, np.float64)
    M, K = x.shape
    assert K % BLOCK == 0
    blocks = x.reshape(M, K // BLOCK, BLOCK)
    amax = np.abs(blocks).max(axis=2)
    with np.errstate(divide="ignore"):
        s = np.where(amax > 0, np.floor(np.log2(np.where(amax > 0, amax, 1.0))) - emax(fmt), 0.0)
    s = np.clip(s, -127, 127)
    codes = quantise_elements(blocks / np.exp2(s)[:, :, None], fmt).reshape(M, K)
    return codes, (s + 127).astype(np.uint8)


def mx_matmul(a_codes, a_scales, a_fmt: MiniFloat, w_codes, w_scales, w_fmt: MiniFloat,
              bias: Optional[np.ndarray] = None) -> np.ndarray:
    """y [M, N] = A W^T (+ bias) with BOTH operands on block-scaled grids."""
    y = dequantise(a_codes, a_scales, a_fmt) @ dequantise(w_codes, w_scales, w_fmt).T
    return y if bias is None else y + np.asarray(bias, np.float64)
