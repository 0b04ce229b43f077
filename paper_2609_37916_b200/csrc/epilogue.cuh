// Element-wise epilogue math shared by the GEMM kernels (fp32).
#pragma once
#include "common.cuh"

namespace rlx {

// Exact-form (erf) GELU, gelu(x) = x * Phi(x), evaluated without erff:
//   u = min(|x|, 5.5);  Phi(-u) = 2^r(u) with r a degree-4 polynomial fitted to log2 Phi(-u), the fit
//   weighted by the sensitivity of the result to r (coefficients from fit_gelu_poly.py next to this
//   file);  gelu(x) = max(x, 0) - u * 2^r(u).
// The epilogue of a K = 384 GEMM is bound by the FP32 pipe (every output gets a handful of FP32
// operations against 384 tensor-core MACs), so every operation counts: 8 FP32-pipe operations and one
// ex2 per value.  |error| <= 6.2e-6 absolute against the erf form, far below the bf16 rounding of the
// stored result.
__device__ __forceinline__ float gelu_erf(float x) {
    const float u = fminf(fabsf(x), 5.5f);
    float r = 3.866270650e-03f;
    r = fmaf(r, u, -4.407931119e-02f);
    r = fmaf(r, u, -4.680147469e-01f);
    r = fmaf(r, u, -1.147372365e+00f);
    r = fmaf(r, u, -1.000479579e+00f);
    float t;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(r));
    return fmaf(-u, t, fmaxf(x, 0.f));
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
    // the polynomial runs on n = -u (odd coefficients change sign), so that the last step is the one
    // fused operation  max(x, 0) + n * t
    const float n0 = fmaxf(-fabsf(x0), -5.5f), n1 = fmaxf(-fabsf(x1), -5.5f);
    const uint64_t n = pack_f32x2(n0, n1);
    uint64_t r = pack_f32x2(3.866270650e-03f, 3.866270650e-03f);
    r = fma_f32x2(r, n, pack_f32x2(4.407931119e-02f, 4.407931119e-02f));
    r = fma_f32x2(r, n, pack_f32x2(-4.680147469e-01f, -4.680147469e-01f));
    r = fma_f32x2(r, n, pack_f32x2(1.147372365e+00f, 1.147372365e+00f));
    r = fma_f32x2(r, n, pack_f32x2(-1.000479579e+00f, -1.000479579e+00f));
    float r0, r1, t0, t1;
    unpack_f32x2(r, r0, r1);
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(t0) : "f"(r0));
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(t1) : "f"(r1));
    unpack_f32x2(fma_f32x2(n, pack_f32x2(t0, t1), pack_f32x2(fmaxf(x0, 0.f), fmaxf(x1, 0.f))), x0, x1);
}

}  // namespace rlx
