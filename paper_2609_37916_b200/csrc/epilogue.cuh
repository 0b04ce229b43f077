// Element-wise epilogue math shared by the GEMM kernels (fp32).
#pragma once
#include "common.cuh"

namespace rlx {

// Exact (erf) GELU: 0.5 u (1 + erf(u / sqrt 2)).
__device__ __forceinline__ float gelu_erf(float u) {
    return 0.5f * u * (1.0f + erff(u * 0.70710678118654752f));
}

}  // namespace rlx
