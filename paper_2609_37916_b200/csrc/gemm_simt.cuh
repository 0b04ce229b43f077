// Plain CUDA-core GEMM with the same fused epilogues as the tcgen05 kernel.  Bring-up and
// cross-check path only (selected by RLX_FLAG_GEMM_SIMT / RLX_GEMM_SIMT); never the default.
// out[M,N] = epilogue(A[M,K] * W[N,K]^T + bias), bf16 operands, fp32 accumulation.
#pragma once
#include "common.cuh"
#include "epilogue.cuh"

namespace rlx {

constexpr int kSimtTile = 64;
constexpr int kSimtBK = 32;

template <int EPI>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const __nv_bfloat16* __restrict__ A, const __nv_bfloat16* __restrict__ W,
                 const float* __restrict__ bias, const __nv_bfloat16* __restrict__ residual,
                 __nv_bfloat16* __restrict__ out, int M, int N, int K) {
    __shared__ float sa[kSimtBK][kSimtTile + 1];
    __shared__ float sw[kSimtBK][kSimtTile + 1];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int m0 = blockIdx.y * kSimtTile, n0 = blockIdx.x * kSimtTile;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < K; k0 += kSimtBK) {
        for (int i = threadIdx.x; i < kSimtTile * kSimtBK; i += 256) {
            const int r = i / kSimtBK, c = i % kSimtBK;
            const bool kin = k0 + c < K;
            sa[c][r] = (kin && m0 + r < M) ? __bfloat162float(A[(size_t)(m0 + r) * K + k0 + c]) : 0.f;
            sw[c][r] = (kin && n0 + r < N) ? __bfloat162float(W[(size_t)(n0 + r) * K + k0 + c]) : 0.f;
        }
        __syncthreads();
#pragma unroll 8
        for (int c = 0; c < kSimtBK; ++c) {
            float a[4], w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = sa[c][ty * 4 + i]; w[i] = sw[c][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] += a[i] * w[j];
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty * 4 + i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n >= N) continue;
            float v = acc[i][j] + bias[n];
            if (EPI == 1) v = gelu_erf(v);
            if (EPI == 2) v += __bfloat162float(residual[(size_t)m * N + n]);
            out[(size_t)m * N + n] = __float2bfloat16_rn(v);
        }
    }
}

}  // namespace rlx
