// Block-scaled FP8 product on the tensor cores' own block-scaled path (the Blackwell half of
// ScaledMatMul): out[M,N] = A W^T (+ bias) with BOTH operands given as (8-bit element codes, one E8M0
// scale byte per 32 consecutive k).  Three kernels (the product has a 128 x 128-tile form, described
// first, and a persistent 128 x 192-tile form further down for widths that are multiples of 192):
//
//  quantise_mx_kernel      bf16 activations -> (codes, scales) by the microscaling rule: per block of 32,
//                          shared exponent floor(log2 max|x|) - emax(format), elements rounded to the
//                          nearest even code with saturation.  One thread per block: 64 bytes in, 32 bytes
//                          of codes and one scale byte out.  Every step is exact (powers of two) except
//                          the final rounding, which is the hardware's round-to-nearest-even conversion.
//
//  gemm_mx_tcgen05_kernel  tcgen05.mma.kind::mxf8f6f4.block_scale: the tensor core multiplies the 8-bit
//                          elements and applies scale_A[row, k/32] * scale_B[col, k/32] per 32-wide
//                          k-group itself; the scale bytes have to sit in tensor memory.  One CTA = one
//                          128 x 128 output tile, six warps:
//    warp 0 (1 lane)   TMA: 128 x 128-byte operand tiles (128 k per stage, 128-byte swizzle)
//    warp 1 (1 lane)   MMA issue: four instructions (K = 32 each) per stage, scale slot selected by
//                      the instruction descriptor's scale-id fields
//    warps 2..5        scale feed, then the epilogue.  For every stage each warp copies the 4 scale
//                      bytes (one 32-bit word = 4 k-groups) of its rows into tensor memory in the layout
//                      the instruction expects: the 128 rows' words live in 32 lanes x 4 columns (lane l,
//                      column c = row 32c + l), replicated in all four lane quarters -- so each of the four
//                      warps writes the same 32 x 4 words into its own quarter with one tcgen05.st (and the
//                      same again for the 128 columns of W).  After the last stage the same warps read the
//                      fp32 accumulator (thread = row), add the bias, round to bf16 and store.
//  One mbarrier per stage collects the TMA bytes AND the four scale warps' arrivals, and one commit per
//  stage frees operands and scale slot together: the issuing thread pays for every barrier round.
//  TMEM: 128 accumulator columns + 3 scale slots of 8 columns = 152 -> 256 allocated, two CTAs per SM,
//  which is what overlaps one tile's epilogue with another's main loop.
// All mbarrier waits are bounded; on expiry the CTA sets the status bit and leaves.
#pragma once
#include <cuda.h>
#include "common.cuh"
#include "gemm_tcgen05.cuh"

namespace rlx {
namespace tcmx {

using namespace rlx::tc;

constexpr int kThreads = 192;
constexpr int kTileM = 128, kTileN = 128;
constexpr int kBlockK = 128;            // 8-bit elements per stage row = 128 bytes = one swizzle row
constexpr int kStages = 3;              // 3 x 32 KB: two CTAs fit an SM
constexpr int kTmemCols = 256;
constexpr int kColSf = kTileN;          // one scale slot (8 columns) per stage, behind the accumulator
constexpr int kOperandBytes = kTileM * kBlockK;
constexpr int kSmemBytes = kStages * 2 * kOperandBytes + 256 + 1024;

// element format ids of the instruction descriptor
constexpr int kFmtE4M3 = 0, kFmtE5M2 = 1;

// Instruction descriptor of kind::mxf8f6f4 with block scaling: [4,6) scale id of B, [7,10) A format,
// [10,13) B format, [15] / [16] A / B major (0 = K-major), [17,23) N >> 3, [23] scale format (1 = E8M0),
// [24,29) M >> 4, [29,31) scale id of A.  fp32 accumulation is implied.
__device__ __forceinline__ uint32_t idesc_mx(int a_fmt, int b_fmt, int sf_id) {
    return ((uint32_t)sf_id << 4) | ((uint32_t)a_fmt << 7) | ((uint32_t)b_fmt << 10) | ((uint32_t)(kTileN >> 3) << 17) |
           (1u << 23) | ((uint32_t)(kTileM >> 4) << 24) | ((uint32_t)sf_id << 29);
}
__device__ __forceinline__ void umma_mx(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                        uint32_t tmem_sfa, uint32_t tmem_sfb, uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %6, 0;\n"
        "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale.scale_vec::1X [%0], %1, %2, %3, [%4], [%5], p;\n"
        "}\n" ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(tmem_sfa), "r"(tmem_sfb), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_st_32x8(uint32_t taddr, const uint32_t (&r)[8]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]) : "memory");
}
__device__ __forceinline__ void tmem_st_wait_all() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

struct MxParams {
    const uint8_t* sfa;     // [M, K/32] scale bytes of A
    const uint8_t* sfw;     // [N, K/32] scale bytes of W
    const float* bias;      // [N] or nullptr
    __nv_bfloat16* out;     // [M, N]
    int M, N, K;
    int a_fmt, w_fmt;       // kFmtE4M3 / kFmtE5M2
    int32_t* status;
};

__global__ void __launch_bounds__(kThreads, 2)
gemm_mx_tcgen05_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w, MxParams p) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* gbase = smem_raw + (base - raw);
    const uint32_t bars = base + kStages * 2 * kOperandBytes;
    const uint32_t full = bars, empty = full + 8 * kStages, acc_full = empty + 8 * kStages;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gbase + kStages * 2 * kOperandBytes + 8 * (2 * kStages + 1));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles = p.N / kTileN;
    const int m0 = (blockIdx.x / n_tiles) * kTileM, n0 = (blockIdx.x % n_tiles) * kTileN;
    const int nkb = p.K / kBlockK;
    const int sf_ld = p.K / 32;   // scale bytes per row

    if (threadIdx.x == 0) {
        // full: the TMA lane's expect_tx arrival + one arrival per scale warp
        for (int i = 0; i < kStages; ++i) { mbar_init(full + 8 * i, 5); mbar_init(empty + 8 * i, 1); }
        mbar_init(acc_full, 1);
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmap_a);
        prefetch_tmap(&tmap_w);
    }
    if (warp == 1) {
        tmem_alloc<1>(smem_u32(tmem_slot), kTmemCols);
        tmem_relinquish<1>();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            for (int kb = 0; kb < nkb; ++kb) {
                const int st = kb % kStages, use = kb / kStages;
                if (use >= 1 && !mbar_wait(empty + 8 * st, (use - 1) & 1, abort_flag)) break;
                const uint32_t dst = base + st * 2 * kOperandBytes;
                mbar_expect_tx(full + 8 * st, 2 * kOperandBytes);
                tma_load_2d(dst, &tmap_a, kb * kBlockK, m0, full + 8 * st);
                tma_load_2d(dst + kOperandBytes, &tmap_w, kb * kBlockK, n0, full + 8 * st);
            }
        }
    } else if (warp == 1) {
        // warp-uniform loop, one elected lane issues (cheaper per instruction than a lone lane under a branch)
        bool ok = true;
        for (int kb = 0; kb < nkb && ok; ++kb) {
            const int st = kb % kStages;
            if (!(ok = mbar_wait_warp(full + 8 * st, (kb / kStages) & 1, abort_flag))) break;
            tc_fence_after();
            if (elect_one()) {
                const uint64_t adesc = make_smem_desc(base + st * 2 * kOperandBytes);
                const uint64_t bdesc = make_smem_desc(base + st * 2 * kOperandBytes + kOperandBytes);
                const uint32_t sfa = tmem + kColSf + st * 8, sfb = sfa + 4;
#pragma unroll
                for (int k = 0; k < kBlockK / 32; ++k)   // 32 bytes of k per instruction: descriptor start + 2
                    umma_mx(tmem, adesc + 2 * k, bdesc + 2 * k, idesc_mx(p.a_fmt, p.w_fmt, k), sfa, sfb, (kb | k) != 0 ? 1u : 0u);
                umma_commit<1>(empty + 8 * st);
                if (kb == nkb - 1) umma_commit<1>(acc_full);
            }
            __syncwarp();
        }
    } else {
        // ------------------------------------------------------------ scale feed, then epilogue
        const int quad = warp & 3;
        const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
        bool ok = true;
        for (int kb = 0; kb < nkb && ok; ++kb) {
            const int slot = kb % kStages, use = kb / kStages;
            uint32_t w[8];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int ar = m0 + 32 * c + lane, wr = n0 + 32 * c + lane;
                // rows past M are zero-filled operand rows: any finite scale will do
                w[c] = ar < p.M ? __ldg(reinterpret_cast<const uint32_t*>(p.sfa + (size_t)ar * sf_ld) + kb) : 0x7F7F7F7Fu;
                w[4 + c] = __ldg(reinterpret_cast<const uint32_t*>(p.sfw + (size_t)wr * sf_ld) + kb);
            }
            if (use >= 1 && !(ok = mbar_wait(empty + 8 * slot, (use - 1) & 1, abort_flag))) break;
            tc_fence_after();
            tmem_st_32x8(lane_addr + kColSf + slot * 8, w);
            tmem_st_wait_all();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(full + 8 * slot);
        }
        if (ok && (ok = mbar_wait(acc_full, 0, abort_flag))) {
            tc_fence_after();
            const int row = m0 + quad * 32 + lane;
            __nv_bfloat16* orow = p.out + (size_t)row * p.N + n0;
#pragma unroll 1
            for (int c0 = 0; c0 < kTileN; c0 += 32) {
                uint32_t r[32];
                tmem_ld_32x32(lane_addr + c0, r);
                tmem_ld_wait();
                if (row < p.M) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        float v[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            v[j] = __uint_as_float(r[8 * i + j]) + (p.bias ? __ldg(p.bias + n0 + c0 + 8 * i + j) : 0.f);
                        uint4 q;
                        q.x = pack_bf16(v[0], v[1]); q.y = pack_bf16(v[2], v[3]);
                        q.z = pack_bf16(v[4], v[5]); q.w = pack_bf16(v[6], v[7]);
                        *(reinterpret_cast<uint4*>(orow + c0) + i) = q;
                    }
                }
            }
        }
    }
    // ---------------------------------------------------------------- teardown
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
        tmem_dealloc<1>(tmem, kTmemCols);
    }
}

// ---------------------------------------------------------------------------- persistent 128 x 192 tiles
// The same product for N % 192 == 0 (the encoder's widths 384, 1152, 1536 and multiples): one persistent
// CTA per SM walks the tile list, the fp32 accumulators are double-buffered in tensor memory so that the
// epilogue of tile i overlaps the main loop of tile i + 1, the scale feed has its own four warps and the
// epilogue eight (one lane quarter x one 96-column half each).  A 128 x 192 tile moves 40 KB of operands
// per 384 tensor-core cycles (the 128 x 128 tile: 32 KB per 256), which is what the SM's fill rate can
// sustain.  TMEM: 2 x 192 accumulator columns + 4 scale slots of 12 columns (A's 4, W's 8) = 432 -> 512.
namespace wide {
constexpr int kTileNW = 192;
constexpr int kStagesW = 4;
constexpr int kThreadsW = 448;   // TMA, MMA, 4 scale warps, 8 epilogue warps
constexpr int kAccCols = 2 * kTileNW;
constexpr int kSfCols = 12;
constexpr int kWBytes = kTileNW * kBlockK;
constexpr int kStageBytesW = kOperandBytes + kWBytes;
constexpr int kEpiWarpsW = 8;
constexpr int kStagingW = kEpiWarpsW * kStageBufBytes;   // one 2 KB chunk buffer per epilogue warp (TMA-store source)
constexpr int kSmemBytesW = kStagesW * kStageBytesW + kStagingW + 256 + 1024;

__device__ __forceinline__ uint32_t idesc_mx_w(int a_fmt, int b_fmt, int sf_id) {
    return ((uint32_t)sf_id << 4) | ((uint32_t)a_fmt << 7) | ((uint32_t)b_fmt << 10) | ((uint32_t)(kTileNW >> 3) << 17) |
           (1u << 23) | ((uint32_t)(kTileM >> 4) << 24) | ((uint32_t)sf_id << 29);
}
__device__ __forceinline__ void tmem_st_32x4(uint32_t taddr, const uint32_t (&r)[4]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1, %2, %3, %4};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
}

__global__ void __launch_bounds__(kThreadsW, 1)
gemm_mx192_tcgen05_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_w,
                          const __grid_constant__ CUtensorMap tmap_out, MxParams p) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* gbase = smem_raw + (base - raw);
    const uint32_t staging = base + kStagesW * kStageBytesW;
    const uint32_t bars = staging + kStagingW;
    const uint32_t full = bars, empty = full + 8 * kStagesW, tfull = empty + 8 * kStagesW, tempty = tfull + 16;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gbase + kStagesW * kStageBytesW + kStagingW + 8 * (2 * kStagesW + 4));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles = p.N / kTileNW, m_tiles = (p.M + kTileM - 1) / kTileM, num_tiles = n_tiles * m_tiles;
    const int nkb = p.K / kBlockK;
    const int sf_ld = p.K / 32;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kStagesW; ++i) { mbar_init(full + 8 * i, 5); mbar_init(empty + 8 * i, 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(tfull + 8 * i, 1); mbar_init(tempty + 8 * i, 8); }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmap_a);
        prefetch_tmap(&tmap_w);
        prefetch_tmap(&tmap_out);
    }
    if (warp == 1) {
        tmem_alloc<1>(smem_u32(tmem_slot), 512);
        tmem_relinquish<1>();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            uint32_t it = 0;   // stages issued so far
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const int m0 = (tile / n_tiles) * kTileM, n0 = (tile % n_tiles) * kTileNW;
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const uint32_t st = it % kStagesW, use = it / kStagesW;
                    if (use >= 1 && !(ok = mbar_wait(empty + 8 * st, (use - 1) & 1, abort_flag))) break;
                    const uint32_t dst = base + st * kStageBytesW;
                    mbar_expect_tx(full + 8 * st, kStageBytesW);
                    tma_load_2d(dst, &tmap_a, kb * kBlockK, m0, full + 8 * st);
                    tma_load_2d(dst + kOperandBytes, &tmap_w, kb * kBlockK, n0, full + 8 * st);
                }
            }
        }
    } else if (warp == 1) {
        uint32_t it = 0, tcount = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++tcount) {
            const uint32_t as = tcount & 1, ause = tcount >> 1;
            if (ause >= 1 && !(ok = mbar_wait_warp(tempty + 8 * as, (ause - 1) & 1, abort_flag))) break;
            for (int kb = 0; kb < nkb; ++kb, ++it) {
                const uint32_t st = it % kStagesW;
                if (!(ok = mbar_wait_warp(full + 8 * st, (it / kStagesW) & 1, abort_flag))) break;
                tc_fence_after();
                if (elect_one()) {
                    const uint64_t adesc = make_smem_desc(base + st * kStageBytesW);
                    const uint64_t bdesc = make_smem_desc(base + st * kStageBytesW + kOperandBytes);
                    const uint32_t sfa = tmem + kAccCols + st * kSfCols, sfb = sfa + 4;
#pragma unroll
                    for (int k = 0; k < kBlockK / 32; ++k)
                        umma_mx(tmem + as * kTileNW, adesc + 2 * k, bdesc + 2 * k, idesc_mx_w(p.a_fmt, p.w_fmt, k), sfa, sfb,
                                (kb | k) != 0 ? 1u : 0u);
                    umma_commit<1>(empty + 8 * st);
                    if (kb == nkb - 1) umma_commit<1>(tfull + 8 * as);
                }
                __syncwarp();
            }
        }
    } else if (warp < 6) {
        // ------------------------------------------------------------ scale feed (one warp per lane quarter)
        // The scale words of a stage are requested kAhead stages before they are written to tensor memory,
        // so that their global-memory latency stays off the pipeline's critical path.
        constexpr int kAhead = 3;
        const int quad = warp & 3;
        const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
        const int my_tiles = blockIdx.x < num_tiles ? (num_tiles - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
        const long long total = (long long)my_tiles * nkb;
        uint32_t wa[kAhead][4], wb[kAhead][8];
        auto fetch = [&](long long i, uint32_t (&a4)[4], uint32_t (&b8)[8]) {
            const int tile = blockIdx.x + (int)(i / nkb) * gridDim.x, kb = (int)(i % nkb);
            const int m0 = (tile / n_tiles) * kTileM, n0 = (tile % n_tiles) * kTileNW;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int ar = m0 + 32 * c + lane;
                // rows past M are zero-filled operand rows: any finite scale will do
                a4[c] = ar < p.M ? __ldg(reinterpret_cast<const uint32_t*>(p.sfa + (size_t)ar * sf_ld) + kb) : 0x7F7F7F7Fu;
            }
#pragma unroll
            for (int c = 0; c < 8; ++c) {   // two 128-row groups of W's rows; the second is half used
                const int wr = 32 * c + lane;
                b8[c] = wr < kTileNW ? __ldg(reinterpret_cast<const uint32_t*>(p.sfw + (size_t)(n0 + wr) * sf_ld) + kb) : 0x7F7F7F7Fu;
            }
        };
#pragma unroll
        for (int i = 0; i < kAhead; ++i)
            if (i < total) fetch(i, wa[i], wb[i]);
        bool ok = true;
        for (long long i0 = 0; i0 < total && ok; i0 += kAhead) {
#pragma unroll
            for (int u = 0; u < kAhead; ++u) {
                const long long i = i0 + u;
                if (i >= total) break;
                const uint32_t slot = (uint32_t)(i % kStagesW), use = (uint32_t)(i / kStagesW);
                if (use >= 1 && !(ok = mbar_wait(empty + 8 * slot, (use - 1) & 1, abort_flag))) break;
                tc_fence_after();
                tmem_st_32x4(lane_addr + kAccCols + slot * kSfCols, wa[u]);
                tmem_st_32x8(lane_addr + kAccCols + slot * kSfCols + 4, wb[u]);
                tmem_st_wait_all();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(full + 8 * slot);
                if (i + kAhead < total) fetch(i + kAhead, wa[u], wb[u]);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue: lane quarter x 96-column half
        // the bf16 GEMM's epilogue tile: all three chunks to registers, accumulator handed back, bias, one
        // TMA store per 32 x 32 chunk out of the warp's swizzled staging buffer
        const int quad = warp & 3, half = (warp - 6) >> 2, ew = warp - 6;
        const uint32_t stg = staging + ew * kStageBufBytes;
        Params gp = {};
        gp.bias = p.bias; gp.out = p.out; gp.M = p.M; gp.N = p.N; gp.K = p.K; gp.status = p.status;
        uint32_t tcount = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++tcount) {
            const int m_row0 = (tile / n_tiles) * kTileM + quad * 32, n0 = (tile % n_tiles) * kTileNW + half * 96;
            const uint32_t as = tcount & 1;
            if (!(ok = mbar_wait(tfull + 8 * as, (tcount >> 1) & 1, abort_flag))) break;
            tc_fence_after();
            EpilogueTile<0, 3> et;
            et.template drain<1>(gp, &tmap_out, p.M, m_row0, n0, tmem + ((uint32_t)(quad * 32) << 16) + as * kTileNW + half * 96,
                                 stg, lane, tempty + 8 * as, 0u);
        }
        EpilogueTile<0, 3>::finish(lane);
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
        tmem_dealloc<1>(tmem, 512);
    }
}
}  // namespace wide

// ---------------------------------------------------------------------------- activation quantiser
template <bool E5M2>
__device__ __forceinline__ uint16_t cvt_fp8x2(float lo, float hi) {
    uint16_t r;
    if (E5M2) asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    else      asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}

constexpr int kQuantThreads = 256;

// x bf16 [M, K] -> codes [M, K] bytes, scales [M, K/32] bytes; one thread per 32-element block.
template <bool E5M2>
__global__ void __launch_bounds__(kQuantThreads)
quantise_mx_kernel(const __nv_bfloat16* __restrict__ x, uint8_t* __restrict__ codes, uint8_t* __restrict__ scales,
                   long long blocks) {
    const long long b = (long long)blockIdx.x * kQuantThreads + threadIdx.x;
    if (b >= blocks) return;
    constexpr int kEmax = E5M2 ? 15 : 8;
    const uint4* src = reinterpret_cast<const uint4*>(x + b * 32);
    uint4 in[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) in[i] = __ldg(src + i);
    const uint32_t* w = reinterpret_cast<const uint32_t*>(in);
    float amax = 0.f;
#pragma unroll
    for (int i = 0; i < 16; ++i) amax = fmaxf(amax, fmaxf(fabsf(bf16lo(w[i])), fabsf(bf16hi(w[i]))));
    int s = amax > 0.f ? ilogbf(amax) - kEmax : 0;
    s = max(-127, min(127, s));
    uint4 out[2];
    uint16_t* o = reinterpret_cast<uint16_t*>(out);
#pragma unroll
    for (int i = 0; i < 16; ++i) o[i] = cvt_fp8x2<E5M2>(scalbnf(bf16lo(w[i]), -s), scalbnf(bf16hi(w[i]), -s));
    uint4* dst = reinterpret_cast<uint4*>(codes + b * 32);
    dst[0] = out[0];
    dst[1] = out[1];
    scales[b] = (uint8_t)(s + 127);
}

}  // namespace tcmx
}  // namespace rlx
