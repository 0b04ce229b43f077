// Projection + bias + residual + LayerNorm in one kernel, for hidden sizes whose whole row fits in
// tensor memory (N = 2 * NH <= 512 fp32 columns: H = 256, 384 or 512):
//
//     out = LN(A W^T + bias + residual; gamma, beta)        A [M,K] bf16, W [N,K] bf16, out [M,N] bf16
//
// One persistent CTA per SM owns 128 complete output rows at a time, so the row statistics never
// leave the SM and neither the pre-LayerNorm sum nor a separate LayerNorm kernel touches HBM.
//   warp 0      TMA producer (A tile 128x64 and the full-width W slice as two NH-row boxes per k-block)
//   warp 1      MMA issuer: two tcgen05.mma (N = NH each) per 16-wide k-step into columns [0,NH) and [NH,2NH)
//   warps 2..9  epilogue, thread = (row, half of the columns), three sweeps over TMEM:
//                 1. v = acc + bias + residual, written back to TMEM in place; partial row sum
//                 2. partial sum of (v - mean)^2          (two-pass variance, like the row kernel)
//                 3. (v - mean) * rstd * gamma + beta -> bf16 -> swizzled transpose buffer -> 16-byte stores
//               the two warps that share a row exchange their partial sums through shared memory
//               and a 64-thread named barrier.
// The accumulator is single-buffered (2*NH columns leave no room for a second one), so the epilogue
// of a tile and the main loop of the next one do not overlap; the tile still costs far less than
// GEMM + store + reload + LayerNorm as separate kernels.  Waits are bounded as in the plain GEMM.
#pragma once
#include "gemm_tcgen05.cuh"

namespace rlx {
namespace tcln {

using namespace rlx::tc;

constexpr int kStageBuf = 32 * 32 * 2;            // one 32x32 bf16 chunk per epilogue warp
constexpr int kEpiWarps = 8;
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr int kStaging = kEpiWarps * kStageBuf;   // 16 KB
constexpr int kRedBytes = 2 * 128 * 2 * 4;        // [sum | sq][row][half] floats

template <int NH>
struct Cfg {
    static constexpr int N = 2 * NH;
    static constexpr int A_BYTES = BLOCK_M * BLOCK_K * 2;
    static constexpr int BH_BYTES = NH * BLOCK_K * 2;            // one half of the W slice
    static constexpr int STAGE_BYTES = A_BYTES + 2 * BH_BYTES;
    static constexpr int RING_BUDGET = 222 * 1024 - kStaging - kRedBytes;
    static constexpr int STAGES = RING_BUDGET / STAGE_BYTES;
    static constexpr int TMEM_COLS = N <= 256 ? 256 : 512;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + kStaging + kRedBytes + 256 + 1024;
    static_assert(NH % 32 == 0 && NH >= 64 && NH <= 256, "half width");
    static_assert(STAGES >= 2, "ring too shallow");
};

__device__ __forceinline__ void tmem_st_32x32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void pair_barrier(int id) { asm volatile("bar.sync %0, 64;" ::"r"(id) : "memory"); }

struct Params {
    const float* bias;               // [N]
    const __nv_bfloat16* residual;   // [M,N]
    const float* gamma;              // [N]
    const float* beta;               // [N]
    __nv_bfloat16* out;              // [M,N]
    float eps;
    int M, K;
    int32_t* status;
    const int32_t* m_ptr;            // optional device row count
};

template <int NH>
__global__ void __launch_bounds__(kThreads, 1)
gemm_ln_tcgen05_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b, const Params p) {
    using C = Cfg<NH>;
    constexpr int N = C::N;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* gbase = smem_raw + (base - raw);
    const uint32_t staging = base + C::STAGES * C::STAGE_BYTES;
    float* red = reinterpret_cast<float*>(gbase + C::STAGES * C::STAGE_BYTES + kStaging);   // [2][128][2]
    const uint32_t bars = staging + kStaging + kRedBytes;
    const uint32_t full_bar = bars, empty_bar = bars + 8 * C::STAGES;
    const uint32_t tfull_bar = bars + 16 * C::STAGES, tempty_bar = tfull_bar + 8;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gbase + C::STAGES * C::STAGE_BYTES + kStaging + kRedBytes +
                                                      16 * C::STAGES + 16);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* pair_ok = reinterpret_cast<volatile int*>(tmem_slot + 2);   // [kEpiWarps]: this tile's wait succeeded

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        for (int i = 0; i < C::STAGES; ++i) {
            mbar_init(full_bar + 8 * i, 1);
            mbar_init(empty_bar + 8 * i, 1);
        }
        mbar_init(tfull_bar, 1);
        mbar_init(tempty_bar, kEpiWarps);
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmap_a);
        prefetch_tmap(&tmap_b);
    }
    if (warp == 1) {
        tmem_alloc<1>(smem_u32(tmem_slot), C::TMEM_COLS);
        tmem_relinquish<1>();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    pdl_wait();
    int M = p.M;
    if (p.m_ptr != nullptr) M = min(M, __ldg(p.m_ptr));
    const int num_tiles = (M + BLOCK_M - 1) / BLOCK_M;
    const int num_kb = (p.K + BLOCK_K - 1) / BLOCK_K;

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(empty_bar + 8 * stage, phase ^ 1, abort_flag)) { ok = false; break; }
                    const uint32_t sa = base + stage * C::STAGE_BYTES, sb = sa + C::A_BYTES;
                    mbar_expect_tx(full_bar + 8 * stage, C::STAGE_BYTES);
                    tma_load_2d(sa, &tmap_a, kb * BLOCK_K, tile * BLOCK_M, full_bar + 8 * stage);
                    tma_load_2d(sb, &tmap_b, kb * BLOCK_K, 0, full_bar + 8 * stage);
                    tma_load_2d(sb + C::BH_BYTES, &tmap_b, kb * BLOCK_K, NH, full_bar + 8 * stage);
                    if (++stage == C::STAGES) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc(BLOCK_M, NH);
            int stage = 0;
            uint32_t phase = 0;
            int it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
                if (!mbar_wait(tempty_bar, (it & 1) ^ 1, abort_flag)) { ok = false; break; }
                tc_fence_after();
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(full_bar + 8 * stage, phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = base + stage * C::STAGE_BYTES, sb = sa + C::A_BYTES;
                    const uint64_t adesc = make_smem_desc(sa);
                    const uint64_t bdesc0 = make_smem_desc(sb), bdesc1 = make_smem_desc(sb + C::BH_BYTES);
#pragma unroll
                    for (int k = 0; k < BLOCK_K / UMMA_K; ++k) {
                        const uint32_t acc = (kb | k) != 0 ? 1u : 0u;
                        umma_bf16<1>(tmem_base, adesc + 2 * k, bdesc0 + 2 * k, idesc, acc);
                        umma_bf16<1>(tmem_base + NH, adesc + 2 * k, bdesc1 + 2 * k, idesc, acc);
                    }
                    umma_commit<1>(empty_bar + 8 * stage);
                    if (++stage == C::STAGES) { stage = 0; phase ^= 1; }
                }
                if (ok) umma_commit<1>(tfull_bar);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue
        constexpr int NC = NH / 32;
        const int ew = warp - 2;
        const int quad = warp & 3;
        const int hf = ew >> 2;
        const int row = quad * 32 + lane;                 // row inside the tile
        const uint32_t stg = staging + ew * kStageBuf;
        const uint32_t row_off = lane * 64;
        const uint32_t swz = (uint32_t)((lane >> 1) & 3);
        float* red_sum = red;
        float* red_sq = red + 256;
        int it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++it) {
            const int m = tile * BLOCK_M + row;
            const bool row_ok = m < M;
            const int n0 = hf * NH;
            const __nv_bfloat16* rrow = p.residual + (size_t)(row_ok ? m : 0) * N + n0;
            // first residual chunk is fetched before waiting for the accumulator
            uint4 rq[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) rq[i] = __ldg(reinterpret_cast<const uint4*>(rrow) + i);
            // The two warps that share a row quadrant meet at named barriers below, so they must also
            // give up together: each publishes whether its (bounded) wait succeeded and both leave if
            // either one did not -- a warp that left alone would strand its partner at the barrier.
            const bool got = mbar_wait(tfull_bar, it & 1, abort_flag);
            if (lane == 0) pair_ok[ew] = got ? 1 : 0;
            pair_barrier(1 + quad);
            if (!(pair_ok[ew] & pair_ok[ew ^ 4])) { ok = false; break; }
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + n0;
            uint32_t r[2][32];
            // ---- sweep 1: v = acc + bias + residual -> TMEM, partial row sum ----
            float sum = 0.f;
            tmem_ld_32x32(taddr, r[0]);
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                tmem_ld_wait();
                if (c + 1 < NC) tmem_ld_32x32(taddr + (c + 1) * 32, r[(c + 1) & 1]);
                uint4 rn[4];
                if (c + 1 < NC) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) rn[i] = __ldg(reinterpret_cast<const uint4*>(rrow + (c + 1) * 32) + i);
                }
                uint32_t(&acc)[32] = r[c & 1];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float4 b4 = __ldg(reinterpret_cast<const float4*>(p.bias + n0 + c * 32) + i);
                    const uint32_t w0 = (i & 1) ? rq[i >> 1].z : rq[i >> 1].x;
                    const uint32_t w1 = (i & 1) ? rq[i >> 1].w : rq[i >> 1].y;
                    const float v0 = __uint_as_float(acc[4 * i + 0]) + b4.x + bf16lo(w0);
                    const float v1 = __uint_as_float(acc[4 * i + 1]) + b4.y + bf16hi(w0);
                    const float v2 = __uint_as_float(acc[4 * i + 2]) + b4.z + bf16lo(w1);
                    const float v3 = __uint_as_float(acc[4 * i + 3]) + b4.w + bf16hi(w1);
                    sum += (v0 + v1) + (v2 + v3);
                    acc[4 * i + 0] = __float_as_uint(v0);
                    acc[4 * i + 1] = __float_as_uint(v1);
                    acc[4 * i + 2] = __float_as_uint(v2);
                    acc[4 * i + 3] = __float_as_uint(v3);
                }
                tmem_st_32x32(taddr + c * 32, acc);
                if (c + 1 < NC) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) rq[i] = rn[i];
                }
            }
            tmem_st_wait();
            red_sum[row * 2 + hf] = sum;
            pair_barrier(1 + quad);
            const float mean = (red_sum[row * 2] + red_sum[row * 2 + 1]) / (float)N;   // true division: constant rows stay exact
            // ---- sweep 2: centred sum of squares ----
            float sq = 0.f;
            tmem_ld_32x32(taddr, r[0]);
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                tmem_ld_wait();
                if (c + 1 < NC) tmem_ld_32x32(taddr + (c + 1) * 32, r[(c + 1) & 1]);
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const float d = __uint_as_float(r[c & 1][i]) - mean;
                    sq = fmaf(d, d, sq);
                }
            }
            red_sq[row * 2 + hf] = sq;
            pair_barrier(1 + quad);
            const float var = (red_sq[row * 2] + red_sq[row * 2 + 1]) / (float)N;
            const float rstd = 1.0f / sqrtf(var + p.eps);
            // ---- sweep 3: normalise, bf16, staged TMA store ----
            tmem_ld_32x32(taddr, r[0]);
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                tmem_ld_wait();
                if (c + 1 < NC) {
                    tmem_ld_32x32(taddr + (c + 1) * 32, r[(c + 1) & 1]);
                } else {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(tempty_bar);   // accumulator columns are free again
                }
                float y[32];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float4 g4 = __ldg(reinterpret_cast<const float4*>(p.gamma + n0 + c * 32) + i);
                    const float4 b4 = __ldg(reinterpret_cast<const float4*>(p.beta + n0 + c * 32) + i);
                    y[4 * i + 0] = (__uint_as_float(r[c & 1][4 * i + 0]) - mean) * rstd * g4.x + b4.x;
                    y[4 * i + 1] = (__uint_as_float(r[c & 1][4 * i + 1]) - mean) * rstd * g4.y + b4.y;
                    y[4 * i + 2] = (__uint_as_float(r[c & 1][4 * i + 2]) - mean) * rstd * g4.z + b4.z;
                    y[4 * i + 3] = (__uint_as_float(r[c & 1][4 * i + 3]) - mean) * rstd * g4.w + b4.w;
                }
                __syncwarp();   // the previous chunk has been read out of the buffer
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint4 q;
                    q.x = pack_bf16(y[8 * i + 0], y[8 * i + 1]);
                    q.y = pack_bf16(y[8 * i + 2], y[8 * i + 3]);
                    q.z = pack_bf16(y[8 * i + 4], y[8 * i + 5]);
                    q.w = pack_bf16(y[8 * i + 6], y[8 * i + 7]);
                    st_shared_v4(stg + row_off + (((uint32_t)i ^ swz) << 4), q);
                }
                __syncwarp();
                const int m_row0 = tile * BLOCK_M + quad * 32;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int rr = i * 8 + (lane >> 2), cc = lane & 3;
                    const uint4 q = ld_shared_v4(stg + rr * 64 + (((uint32_t)cc ^ (uint32_t)((rr >> 1) & 3)) << 4));
                    if (m_row0 + rr < M)
                        *reinterpret_cast<uint4*>(p.out + (size_t)(m_row0 + rr) * N + n0 + c * 32 + cc * 8) = q;
                }
            }
        }
    }

    if (*abort_flag) {
        if (threadIdx.x == 0 && p.status) atomicOr(p.status, RLX_DEVSTAT_TIMEOUT_BIT);
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc<1>(tmem_base, C::TMEM_COLS);
    }
}

}  // namespace tcln
}  // namespace rlx
