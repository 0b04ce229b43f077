// Shared device helpers for the encoder kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#define RLX_DEVSTAT_TOKEN_RANGE_BIT 0x1
#define RLX_DEVSTAT_TIMEOUT_BIT 0x2

namespace rlx {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// two bf16 packed in a 32-bit word <-> two floats (exact widening)
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    // cvt.rn.bf16x2.f32 d, a, b : a -> upper half, b -> lower half (round to nearest even)
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// Rotary embedding of eight (lo, hi) column pairs held as 2 x 16 bytes of bf16: lo' = lo*cos - hi*sin,
// hi' = hi*cos + lo*sin with explicitly rounded fp32 products (no contraction), so every kernel that
// rotates gives the same bits.  cs / sn: the eight cosines / sines of the pairs' angles.
__device__ __forceinline__ void rope_rotate8(uint4& lo, uint4& hi, const float4 c0, const float4 c1, const float4 s0,
                                             const float4 s1) {
    const float cs[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
    const float sn[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
    const uint32_t lw[4] = {lo.x, lo.y, lo.z, lo.w}, hw[4] = {hi.x, hi.y, hi.z, hi.w};
    uint32_t ol[4], oh[4];
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        const float a0 = bf16lo(lw[w]), a1 = bf16hi(lw[w]), b0 = bf16lo(hw[w]), b1 = bf16hi(hw[w]);
        ol[w] = pack_bf16(__fsub_rn(__fmul_rn(a0, cs[2 * w]), __fmul_rn(b0, sn[2 * w])),
                          __fsub_rn(__fmul_rn(a1, cs[2 * w + 1]), __fmul_rn(b1, sn[2 * w + 1])));
        oh[w] = pack_bf16(__fadd_rn(__fmul_rn(b0, cs[2 * w]), __fmul_rn(a0, sn[2 * w])),
                          __fadd_rn(__fmul_rn(b1, cs[2 * w + 1]), __fmul_rn(a1, sn[2 * w + 1])));
    }
    lo = make_uint4(ol[0], ol[1], ol[2], ol[3]);
    hi = make_uint4(oh[0], oh[1], oh[2], oh[3]);
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// Programmatic dependent launch: a kernel launched with the programmatic-serialization attribute may
// start while its predecessor drains.  launch_dependents lets the successor's CTAs be scheduled early
// (they then park in their own pdl_wait); pdl_wait returns once every predecessor grid has completed
// and its writes are visible.  Both are no-ops for ordinary launches.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

}  // namespace rlx
