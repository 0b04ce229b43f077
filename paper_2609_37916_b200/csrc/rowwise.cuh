// Memory-bound row kernels: embedding gather + LayerNorm, LayerNorm, masked mean-pool + L2 norm.
// One warp owns one row of H = NV * 128 bf16 values; each lane holds NV vectors of 4 values
// (8-byte loads, a warp instruction covers 256 contiguous bytes).  Statistics in fp32, two-pass
// on registers (mean, then centred sum of squares), biased variance, eps inside the square root.
#pragma once
#include "common.cuh"

namespace rlx {

constexpr int kRowWarps = 8;  // rows per CTA

template <int NV>
__device__ __forceinline__ void ln_normalise_store(float (&v)[NV * 4], const float* __restrict__ gamma,
                                                   const float* __restrict__ beta, float eps, int lane,
                                                   __nv_bfloat16* __restrict__ out_row) {
    constexpr int H = NV * 128;
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < NV * 4; ++i) s += v[i];
    const float mean = warp_sum(s) / (float)H;  // true division: a constant row has exactly zero deviation
    float q = 0.f;
#pragma unroll
    for (int i = 0; i < NV * 4; ++i) {
        v[i] -= mean;
        q += v[i] * v[i];
    }
    const float var = warp_sum(q) / (float)H;
    const float rstd = 1.0f / sqrtf(var + eps);
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        const int col = (i * 32 + lane) * 4;
        const float4 g = __ldg(reinterpret_cast<const float4*>(gamma + col));
        const float4 b = __ldg(reinterpret_cast<const float4*>(beta + col));
        uint2 o;
        o.x = pack_bf16(v[i * 4 + 0] * rstd * g.x + b.x, v[i * 4 + 1] * rstd * g.y + b.y);
        o.y = pack_bf16(v[i * 4 + 2] * rstd * g.z + b.z, v[i * 4 + 3] * rstd * g.w + b.w);
        *reinterpret_cast<uint2*>(out_row + col) = o;
    }
}

// x[t] = LN(word[ids[t]] + pos[t % S] + type[0]).  Ids outside [0, V) are clamped and flagged.
template <int NV>
__global__ void __launch_bounds__(kRowWarps * 32)
embed_ln_kernel(const int32_t* __restrict__ ids, const __nv_bfloat16* __restrict__ word,
                const __nv_bfloat16* __restrict__ pos, const __nv_bfloat16* __restrict__ type,
                const float* __restrict__ gamma, const float* __restrict__ beta,
                __nv_bfloat16* __restrict__ out, int T, int S, int V, float eps, int32_t* status) {
    constexpr int H = NV * 128;
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * kRowWarps + (threadIdx.x >> 5);
    if (t >= T) return;
    int id = __ldg(ids + t);
    if (id < 0 || id >= V) {
        if (lane == 0 && status) atomicOr(status, RLX_DEVSTAT_TOKEN_RANGE_BIT);
        id = id < 0 ? 0 : V - 1;
    }
    const int s = t % S;
    const __nv_bfloat16* wrow = word + (size_t)id * H;
    const __nv_bfloat16* prow = pos + (size_t)s * H;
    float v[NV * 4];
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        const int col = (i * 32 + lane) * 4;
        const uint2 a = __ldg(reinterpret_cast<const uint2*>(wrow + col));
        const uint2 b = __ldg(reinterpret_cast<const uint2*>(prow + col));
        const uint2 c = __ldg(reinterpret_cast<const uint2*>(type + col));
        v[i * 4 + 0] = bf16lo(a.x) + bf16lo(b.x) + bf16lo(c.x);
        v[i * 4 + 1] = bf16hi(a.x) + bf16hi(b.x) + bf16hi(c.x);
        v[i * 4 + 2] = bf16lo(a.y) + bf16lo(b.y) + bf16lo(c.y);
        v[i * 4 + 3] = bf16hi(a.y) + bf16hi(b.y) + bf16hi(c.y);
    }
    ln_normalise_store<NV>(v, gamma, beta, eps, lane, out + (size_t)t * H);
}

// out = LN(x) row by row (the residual sum was already formed by the producing GEMM's epilogue).
template <int NV>
__global__ void __launch_bounds__(kRowWarps * 32)
layernorm_kernel(const __nv_bfloat16* __restrict__ x, const float* __restrict__ gamma,
                 const float* __restrict__ beta, __nv_bfloat16* __restrict__ out, int T, float eps) {
    constexpr int H = NV * 128;
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * kRowWarps + (threadIdx.x >> 5);
    if (t >= T) return;
    const __nv_bfloat16* row = x + (size_t)t * H;
    float v[NV * 4];
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        const int col = (i * 32 + lane) * 4;
        const uint2 a = __ldg(reinterpret_cast<const uint2*>(row + col));
        v[i * 4 + 0] = bf16lo(a.x);
        v[i * 4 + 1] = bf16hi(a.x);
        v[i * 4 + 2] = bf16lo(a.y);
        v[i * 4 + 3] = bf16hi(a.y);
    }
    ln_normalise_store<NV>(v, gamma, beta, eps, lane, out + (size_t)t * H);
}

// Masked mean-pool + L2 normalisation.  One CTA per sequence.  Thread (g, c) owns the 8-column
// vector c of the row and walks rows g, g+G, ... skipping rows with mask 0; the G partial sums per
// column vector are combined through shared memory in a fixed order (no atomics: deterministic).
constexpr int kPoolThreads = 384;

__global__ void __launch_bounds__(kPoolThreads)
pool_l2norm_kernel(const __nv_bfloat16* __restrict__ x, const int32_t* __restrict__ mask,
                   float* __restrict__ out, int S, int H) {
    extern __shared__ float pool_smem[];  // [G][H] partial sums, then [kPoolThreads/32] reductions
    const int b = blockIdx.x;
    const int vecs = H / 8;               // 16-byte vectors per row
    const int G = kPoolThreads / vecs;    // row groups (>= 1 since H <= 1024 -> vecs <= 128)
    const int g = threadIdx.x / vecs, c = threadIdx.x % vecs;
    const __nv_bfloat16* xb = x + (size_t)b * S * H;
    const int32_t* mb = mask + (size_t)b * S;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    int count = 0;
    if (g < G) {
        for (int s = g; s < S; s += G) {
            if (__ldg(mb + s) == 0) continue;
            ++count;
            const uint4 a = __ldg(reinterpret_cast<const uint4*>(xb + (size_t)s * H + c * 8));
            acc[0] += bf16lo(a.x); acc[1] += bf16hi(a.x);
            acc[2] += bf16lo(a.y); acc[3] += bf16hi(a.y);
            acc[4] += bf16lo(a.z); acc[5] += bf16hi(a.z);
            acc[6] += bf16lo(a.w); acc[7] += bf16hi(a.w);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) pool_smem[g * H + c * 8 + i] = acc[i];
    }
    __shared__ int s_count[kPoolThreads];
    s_count[threadIdx.x] = (g < G && c == 0) ? count : 0;
    __syncthreads();
    // column sums: thread j < H owns column j
    float n_valid = 0.f;
    for (int i = 0; i < kPoolThreads; ++i) n_valid += (float)s_count[i];  // same value in every thread
    float colsum[3] = {0.f, 0.f, 0.f};  // H <= 1024 -> at most ceil(1024/384) = 3 columns per thread
    float sq = 0.f;
    const float inv_n = 1.0f / fmaxf(n_valid, 1e-9f);
#pragma unroll
    for (int r = 0; r < 3; ++r) {
        const int j = threadIdx.x + r * kPoolThreads;
        if (j < H) {
            float t = 0.f;
            for (int gg = 0; gg < G; ++gg) t += pool_smem[gg * H + j];
            t *= inv_n;
            colsum[r] = t;
            sq += t * t;
        }
    }
    __syncthreads();
    float* red = pool_smem;  // reuse
    sq = warp_sum(sq);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = sq;
    __syncthreads();
    float tot = 0.f;
    for (int i = 0; i < kPoolThreads / 32; ++i) tot += red[i];
    const float inv_norm = 1.0f / fmaxf(sqrtf(tot), 1e-12f);
#pragma unroll
    for (int r = 0; r < 3; ++r) {
        const int j = threadIdx.x + r * kPoolThreads;
        if (j < H) out[(size_t)b * H + j] = colsum[r] * inv_norm;
    }
}

}  // namespace rlx
