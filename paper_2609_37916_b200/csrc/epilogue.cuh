// Element-wise epilogue math shared by the GEMM kernels (fp32).
#pragma once
#include "common.cuh"

namespace rlx {

// Exact-form (erf) GELU, gelu(x) = x * Phi(x), evaluated without erff:
//   u = min(|x|, 5.5);  Phi(-u) = 2^r(u) with r a degree-7 polynomial fitted to log2 Phi(-u)
//   (coefficients from fit_gelu_poly.py next to this file);  Phi(x) = t for x < 0, 1 - t otherwise.
// fp32 Horner + one ex2: |error| <= 7e-7 absolute and <= 5e-6 relative against the erf form, far
// below the bf16 rounding of the stored result.  12 issue slots instead of ~30 for erff.
__device__ __forceinline__ float gelu_erf(float x) {
    const float u = fminf(fabsf(x), 5.5f);
    float r = -1.921234571e-06f;
    r = fmaf(r, u, 6.328849850e-05f);
    r = fmaf(r, u, -9.434208623e-04f);
    r = fmaf(r, u, 8.556271903e-03f);
    r = fmaf(r, u, -5.405228212e-02f);
    r = fmaf(r, u, -4.583817720e-01f);
    r = fmaf(r, u, -1.151278377e+00f);
    r = fmaf(r, u, -9.999938607e-01f);
    float t;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(r));
    const float phi = x < 0.f ? t : 1.0f - t;
    return x * phi;
}

}  // namespace rlx
