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

// The same function on two values at once with Blackwell's packed fp32 arithmetic (fma/add/mul
// .f32x2 operate on a 64-bit register pair): the Horner chain, the 0.5 - t step and the final
// products take one issue slot per PAIR.  Phi(x) = 0.5 + copysign(0.5 - t, x) avoids a select.
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t mul_f32x2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ void gelu_erf_x2(float& x0, float& x1) {
    const float u0 = fminf(fabsf(x0), 5.5f), u1 = fminf(fabsf(x1), 5.5f);
    const uint64_t u = pack_f32x2(u0, u1);
    uint64_t r = pack_f32x2(-1.921234571e-06f, -1.921234571e-06f);
    r = fma_f32x2(r, u, pack_f32x2(6.328849850e-05f, 6.328849850e-05f));
    r = fma_f32x2(r, u, pack_f32x2(-9.434208623e-04f, -9.434208623e-04f));
    r = fma_f32x2(r, u, pack_f32x2(8.556271903e-03f, 8.556271903e-03f));
    r = fma_f32x2(r, u, pack_f32x2(-5.405228212e-02f, -5.405228212e-02f));
    r = fma_f32x2(r, u, pack_f32x2(-4.583817720e-01f, -4.583817720e-01f));
    r = fma_f32x2(r, u, pack_f32x2(-1.151278377e+00f, -1.151278377e+00f));
    r = fma_f32x2(r, u, pack_f32x2(-9.999938607e-01f, -9.999938607e-01f));
    float r0, r1, t0, t1;
    unpack_f32x2(r, r0, r1);
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(t0) : "f"(r0));
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(t1) : "f"(r1));
    // h = 0.5 - t >= 0; give it the sign of x; phi = 0.5 + h
    const uint64_t h = fma_f32x2(pack_f32x2(t0, t1), pack_f32x2(-1.0f, -1.0f), pack_f32x2(0.5f, 0.5f));
    float h0, h1;
    unpack_f32x2(h, h0, h1);
    h0 = __uint_as_float(__float_as_uint(h0) | (__float_as_uint(x0) & 0x80000000u));
    h1 = __uint_as_float(__float_as_uint(h1) | (__float_as_uint(x1) & 0x80000000u));
    const uint64_t phi = add_f32x2(pack_f32x2(h0, h1), pack_f32x2(0.5f, 0.5f));
    unpack_f32x2(mul_f32x2(pack_f32x2(x0, x1), phi), x0, x1);
}

}  // namespace rlx
