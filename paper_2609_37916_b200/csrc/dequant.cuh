// Block-scaled minifloat weights -> bf16 (the dequantisation half of ScaledMatMul).
//
// W[n,k] = value(code[n,k]) * 2^(scale[n, k/32] - 127): codes are sign | X exponent bits | Y mantissa bits
// with bias 2^(X-1)-1 and gradual underflow, one per byte or two per byte (4-bit formats, low nibble =
// smaller k); scales are E8M0 bytes shared by 32 consecutive k.  Every such product is exactly
// representable in bf16 whenever it lies in bf16's range (at most 7 significant bits), so the output is
// the exact weight; outside the range it is the correctly rounded one (a single rounding, see below).
//
// One CTA first builds the format's value table in shared memory (one code per thread, <= 256 codes),
// then every thread converts 16 consecutive k of one row: 16 (or 8) bytes in, 32 bytes out.  The scale
// 2^q is applied as two exact-power-of-two factors 2^floor(q/2) * 2^(q - floor(q/2)): the table values
// span 2^-40 .. 2^33, so the first product is always exact and only the second can round (when the
// result leaves fp32's normal range), which keeps the fp32 -> bf16 conversion the only other rounding.
#pragma once
#include "common.cuh"

namespace rlx {

constexpr int kDequantThreads = 256;
constexpr int kDequantElemsPerThread = 16;

struct MiniFloatFormat {
    int ebits, mbits, special;   // special: 0 none, 1 all-ones magnitude is NaN, 2 top exponent is inf / NaN
};

__device__ __forceinline__ float minifloat_value(int code, MiniFloatFormat f) {
    const int e_mask = (1 << f.ebits) - 1, m_mask = (1 << f.mbits) - 1;
    const int sign = (code >> (f.ebits + f.mbits)) & 1;
    const int e = (code >> f.mbits) & e_mask, m = code & m_mask;
    const int bias = (1 << (f.ebits - 1)) - 1;
    float v;
    if (f.special == 2 && e == e_mask) {
        v = m == 0 ? INFINITY : __int_as_float(0x7fc00000);
    } else if (f.special == 1 && e == e_mask && m == m_mask) {
        v = __int_as_float(0x7fc00000);
    } else {
        const int sig = (e ? (1 << f.mbits) : 0) | m;            // integer significand
        const int ex = (e ? e : 1) - bias - f.mbits;             // value = sig * 2^ex, |ex| <= 40: normal fp32
        v = (float)sig * __int_as_float((ex + 127) << 23);
    }
    return sign ? -v : v;   // keeps -0
}

__device__ __forceinline__ float pow2_normal(int p) { return __int_as_float((p + 127) << 23); }   // -126 <= p <= 127

template <bool PACKED4>
__global__ void __launch_bounds__(kDequantThreads)
dequant_block_scaled_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ scales,
                            __nv_bfloat16* __restrict__ out, int N, int K, MiniFloatFormat fmt) {
    __shared__ float lut[256];
    const int ncodes = 1 << (1 + fmt.ebits + fmt.mbits);
    if ((int)threadIdx.x < ncodes) lut[threadIdx.x] = minifloat_value(threadIdx.x, fmt);
    __syncthreads();
    const int chunks_per_row = K / kDequantElemsPerThread;
    const long long total = (long long)N * chunks_per_row;
    for (long long i = (long long)blockIdx.x * kDequantThreads + threadIdx.x; i < total;
         i += (long long)gridDim.x * kDequantThreads) {
        const int n = (int)(i / chunks_per_row), k0 = (int)(i % chunks_per_row) * kDequantElemsPerThread;
        const int se = __ldg(scales + (size_t)n * (K / 32) + k0 / 32);
        const int q = se - 127, q1 = q >> 1, q2 = q - q1;          // both within [-64, 64]
        const float s1 = se == 255 ? __int_as_float(0x7fc00000) : pow2_normal(q1), s2 = pow2_normal(q2);
        uint32_t c[4];
        if (PACKED4) {
            const uint2 raw = __ldg(reinterpret_cast<const uint2*>(codes + ((size_t)n * K + k0) / 2));
            c[0] = raw.x; c[1] = raw.y; c[2] = 0; c[3] = 0;
        } else {
            const uint4 raw = __ldg(reinterpret_cast<const uint4*>(codes + (size_t)n * K + k0));
            c[0] = raw.x; c[1] = raw.y; c[2] = raw.z; c[3] = raw.w;
        }
        uint32_t o[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            int a, b;   // codes of elements 2j and 2j+1
            if (PACKED4) {
                const uint32_t byte = (c[j >> 2] >> ((j & 3) * 8)) & 0xff;
                a = byte & 0xf; b = byte >> 4;
            } else {
                a = (c[j >> 1] >> ((j & 1) * 16)) & 0xff;
                b = (c[j >> 1] >> ((j & 1) * 16 + 8)) & 0xff;
            }
            o[j] = pack_bf16(__fmul_rn(__fmul_rn(lut[a], s1), s2), __fmul_rn(__fmul_rn(lut[b], s1), s2));
        }
        uint4* dst = reinterpret_cast<uint4*>(out + (size_t)n * K + k0);
        dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
        dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
    }
}

}  // namespace rlx
