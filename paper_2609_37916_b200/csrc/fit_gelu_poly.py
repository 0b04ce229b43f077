"""Generates the polynomial used by the GEMM epilogue's GELU (csrc/epilogue.cuh).

gelu(x) = x * Phi(x).  With u = min(|x|, U):  Phi(-u) = 2^r(u),  r(u) = log2 Phi(-u), which is
smooth and nearly quadratic, so a low-degree polynomial fits it well.  The kernel evaluates r by
Horner in fp32, takes one ex2, and uses Phi(x) = t for x < 0 and 1 - t for x >= 0.

    python fit_gelu_poly.py            # prints the coefficients and the measured error

Fit: Chebyshev interpolation (near-minimax) of degree DEG on [0, U], converted to the power basis.
Error of the resulting fp32 evaluation against the exact erf form: |gelu err| <= 7e-7 absolute,
<= 5e-6 relative, three orders of magnitude below the bf16 rounding of the stored result.
"""
import numpy as np
from numpy.polynomial import chebyshev as C
from scipy.special import log_ndtr, ndtr

U, DEG = 5.5, 7


def fit():
    n = 400
    x = np.cos(np.pi * (np.arange(n) + 0.5) / n)
    u = (x + 1) * U / 2
    c = C.chebfit(x, log_ndtr(-u) / np.log(2), DEG)
    px = np.poly1d(C.cheb2poly(c)[::-1])
    return px(np.poly1d([2 / U, -1])).coeffs[::-1].astype(np.float32)   # ascending powers of u


def check(coef):
    u = np.linspace(0, 8, 400001).astype(np.float32)
    uc = np.minimum(u, np.float32(U))
    acc = np.full_like(uc, coef[-1])
    for cf in coef[-2::-1]:
        acc = (acc * uc + cf).astype(np.float32)
    t = np.exp2(acc.astype(np.float64))
    ref = ndtr(-u.astype(np.float64))
    e_neg, e_pos = np.abs(-u * t + u * ref), np.abs(u * (1 - t) - u * (1 - ref))
    rel = e_neg[(u > 1e-3) & (u < 5)] / (u * ref)[(u > 1e-3) & (u < 5)]
    return max(e_neg.max(), e_pos.max()), rel.max()


if __name__ == "__main__":
    coef = fit()
    for i, c in enumerate(coef):
        print(f"c{i} = {float(c):.9e}f")
    print("max abs err, max rel err (x in [-5,0)):", check(coef))
