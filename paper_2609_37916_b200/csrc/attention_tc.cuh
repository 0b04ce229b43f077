// Packed-sequence attention on the 5th-generation tensor cores (tcgen05 + TMEM), head_dim 32 or 64,
// up to 512 keys per sequence.  One CTA = 128 query rows of one (sequence, head):
//
//   warp 0 (1 lane)   TMA: Q tile and all K / V blocks of the sequence (64 keys each) straight out
//                     of the packed [rows, 3H] projection, one mbarrier per block
//   warp 1 (1 lane)   MMA issue:  S = Q K^T  (M=128, N=keys, K=d; both operands K-major)
//                                 O += P V    (M=128, N=d, K=keys; P read from TMEM, V MN-major)
//   warps 2..5        softmax, one thread per query row (TMEM lane = row, so row max / row sum are
//                     plain per-thread loops, no shuffles):
//                       pass 1  row max over all key blocks            (S from TMEM)
//                       pass 2  p = exp2(s*c - max*c), row sum, P (bf16) written back to TMEM
//                     then O / sum -> bf16 -> global.
// Two passes over S (the QK^T product is simply issued twice when there is more than one key block)
// mean the final row max is known before any exponential is taken: no running rescale of O.
// Keys come in blocks of 64; P overwrites S in place (chunk c of P lands in columns that chunk <= c
// of S occupied), so a CTA needs only 128 TMEM columns (S/P [0,64), O [64,64+d)) and four CTAs share
// an SM: each CTA is a chain of short dependent steps, and it is the number of chains in flight
// that fills the machine.
// All mbarrier waits are bounded; on expiry the CTA sets the status bit and leaves.
#pragma once
#include <cuda.h>
#include "common.cuh"
#include "gemm_tcgen05.cuh"

namespace rlx {
namespace tca {

using namespace rlx::tc;

constexpr int kThreads = 192;
constexpr int kBlockM = 128;   // query rows per CTA
constexpr int kBlockN = 64;    // keys per block
constexpr int kMaxBlocks = 8;  // 512 keys
constexpr int kTmemCols = 128; // four CTAs per SM: the kernel is a chain of short dependent steps, so
                               // throughput comes from many CTAs in flight, not from a long one
constexpr int kColS = 0, kColP = 0, kColO = 64;   // P (bf16) overwrites S in place, chunk by chunk

template <int D>
struct Smem {
    static constexpr int ROW_BYTES = D * 2;                  // 64 (64-byte swizzle) or 128 (128-byte swizzle)
    static constexpr int TILE_BYTES = kBlockN * ROW_BYTES;   // one 64-row tile of K or V (Q is two of them)
    // Q (128 rows), then nblk K tiles, then nblk V tiles, then the barrier block
    __host__ __device__ static constexpr int bar_offset(int nblk) { return (2 + 2 * nblk) * TILE_BYTES; }
    __host__ __device__ static constexpr int bytes(int nblk) { return bar_offset(nblk) + 256 + 1024; }
};

// K-major operand tile with rows of ROW_BYTES (= the swizzle span): 8-row groups are 8*ROW_BYTES apart.
template <int D>
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)((8 * D * 2) >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)(D == 64 ? 2 : 4) << 61;   // 128-byte / 64-byte swizzle
    return d;
}
// V as the B operand of O = P V: N (= head dim) is the contiguous direction, K (= keys) runs over
// rows; 8-key groups are 8*ROW_BYTES apart; the N extent is exactly one swizzle span.
template <int D>
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t smem_addr) { return desc_kmajor<D>(smem_addr); }

// fp32 accumulate, bf16 operands, A K-major (or TMEM), B K-major (b_mn = 0) or MN-major (b_mn = 1)
__device__ __forceinline__ uint32_t idesc_attn(int m, int n, int b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn << 16) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(m >> 4) << 24);
}
__device__ __forceinline__ void umma_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n"
        "}\n" ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void tmem_st_32x16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int D>
__global__ void __launch_bounds__(kThreads)
attention_tc_kernel(const __grid_constant__ CUtensorMap tmap_qkv, const int32_t* __restrict__ seq_start,
                    const int32_t* __restrict__ seq_len, __nv_bfloat16* __restrict__ ctx, int H,
                    float scale_log2e, int max_blocks, int32_t* status) {
    using SM = Smem<D>;
    pdl_launch_dependents();
    pdl_wait();
    const int q0 = blockIdx.x * kBlockM, head = blockIdx.y, b = blockIdx.z;
    const int len = __ldg(seq_len + b);
    if (q0 >= len) return;   // uniform: nothing allocated yet
    const int row0 = __ldg(seq_start + b);
    const int nkb = (len + kBlockN - 1) / kBlockN;

    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* gbase = smem_raw + (base - raw);
    const uint32_t sq = base, sk = base + 2 * SM::TILE_BYTES, sv = sk + max_blocks * SM::TILE_BYTES;
    const uint32_t bars = base + SM::bar_offset(max_blocks);
    // barriers: q_full, k_full[4], v_full[4], s_full, s_free, p_full, pv_done
    const uint32_t q_full = bars, k_full = bars + 8, v_full = bars + 8 + 8 * kMaxBlocks;
    const uint32_t s_full = bars + 8 + 16 * kMaxBlocks, s_free = s_full + 8, p_full = s_full + 16, pv_done = s_full + 24;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gbase + SM::bar_offset(max_blocks) + 8 + 16 * kMaxBlocks + 32);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        for (int i = 0; i < kMaxBlocks; ++i) { mbar_init(k_full + 8 * i, 1); mbar_init(v_full + 8 * i, 1); }
        mbar_init(s_full, 1);
        mbar_init(s_free, 4);
        mbar_init(p_full, 4);
        mbar_init(pv_done, 1);
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmap_qkv);
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
        // ------------------------------------------------------------ TMA: Q, then K_j and V_j
        if (lane == 0) {
            mbar_expect_tx(q_full, 2 * SM::TILE_BYTES);
            tma_load_2d(sq, &tmap_qkv, head * D, row0 + q0, q_full);
            tma_load_2d(sq + SM::TILE_BYTES, &tmap_qkv, head * D, row0 + q0 + kBlockN, q_full);
            for (int j = 0; j < nkb; ++j) {
                mbar_expect_tx(k_full + 8 * j, SM::TILE_BYTES);
                tma_load_2d(sk + j * SM::TILE_BYTES, &tmap_qkv, H + head * D, row0 + j * kBlockN, k_full + 8 * j);
            }
            for (int j = 0; j < nkb; ++j) {
                mbar_expect_tx(v_full + 8 * j, SM::TILE_BYTES);
                tma_load_2d(sv + j * SM::TILE_BYTES, &tmap_qkv, 2 * H + head * D, row0 + j * kBlockN, v_full + 8 * j);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issue
        if (lane == 0) {
            bool ok = mbar_wait(q_full, 0, abort_flag);
            uint32_t n_sfree = 0, n_pfull = 0;   // completed-phase counters of the barriers this thread waits on
            const uint64_t qdesc = desc_kmajor<D>(sq);
            auto issue_s = [&](int j) {
                const int keys = min(kBlockN, len - j * kBlockN);
                const int n = (keys + 15) & ~15;                       // UMMA N: multiple of 16
                const uint32_t idesc = idesc_attn(kBlockM, n, 0);
                const uint64_t kdesc = desc_kmajor<D>(sk + j * SM::TILE_BYTES);
#pragma unroll
                for (int k = 0; k < D / 16; ++k) umma_bf16<1>(tmem + kColS, qdesc + 2 * k, kdesc + 2 * k, idesc, k != 0);
                umma_commit<1>(s_full);
            };
            // pass 1: S_j for the row maxima
            for (int j = 0; j < nkb && ok; ++j) {
                if (!(ok = mbar_wait(k_full + 8 * j, 0, abort_flag))) break;
                if (j > 0) {
                    if (!(ok = mbar_wait(s_free, n_sfree & 1, abort_flag))) break;
                    ++n_sfree;
                }
                tc_fence_after();
                issue_s(j);
            }
            // pass 2: S_j again (unless the single block is still in TMEM), then O += P_j V_j.  P_j lives in
            // S_j's columns, so S_{j+1} may only be issued once P_j V_j has finished reading them.
            uint32_t n_pvdone = 0;
            for (int j = 0; j < nkb && ok; ++j) {
                if (nkb > 1) {
                    if (j == 0) {
                        if (!(ok = mbar_wait(s_free, n_sfree & 1, abort_flag))) break;   // last pass-1 read
                        ++n_sfree;
                    } else {
                        if (!(ok = mbar_wait(pv_done, n_pvdone & 1, abort_flag))) break;
                        ++n_pvdone;
                    }
                    tc_fence_after();
                    issue_s(j);
                }
                if (!(ok = mbar_wait(p_full, n_pfull & 1, abort_flag))) break;
                ++n_pfull;
                if (!(ok = mbar_wait(v_full + 8 * j, 0, abort_flag))) break;
                tc_fence_after();
                const int keys = min(kBlockN, len - j * kBlockN);
                const int ksteps = (keys + 15) >> 4;
                const uint32_t idesc = idesc_attn(kBlockM, D, 1);
                const uint64_t vdesc = desc_mnmajor<D>(sv + j * SM::TILE_BYTES);
                for (int kk = 0; kk < ksteps; ++kk) {
                    // 16 keys = two 8-row groups of ROW_BYTES rows further down the V tile
                    umma_ts(tmem + kColO, tmem + kColP + kk * 8, vdesc + (uint64_t)((16 * D * 2) >> 4) * kk, idesc,
                            (j | kk) != 0);
                }
                umma_commit<1>(pv_done);
            }
        }
    } else {
        // ------------------------------------------------------------ softmax warps (thread = query row)
        const int quad = warp & 3;
        const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
        const int qrow = q0 + quad * 32 + lane;
        uint32_t n_sfull = 0, n_pvdone = 0;
        bool ok = true;
        float m_row = -INFINITY;
        // ---- pass 1: row maximum of the raw scores ----
        for (int j = 0; j < nkb && ok; ++j) {
            if (!(ok = mbar_wait(s_full, n_sfull & 1, abort_flag))) break;
            ++n_sfull;
            tc_fence_after();
            const int keys = min(kBlockN, len - j * kBlockN);
            for (int c0 = 0; c0 < keys; c0 += 32) {
                uint32_t r[32];
                tmem_ld_32x32(lane_addr + kColS + c0, r);
                tmem_ld_wait();
                if (c0 + 32 <= keys) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) m_row = fmaxf(m_row, __uint_as_float(r[i]));
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (c0 + i < keys) m_row = fmaxf(m_row, __uint_as_float(r[i]));
                }
            }
            if (nkb > 1) {   // the single-block case keeps S in place for pass 2
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(s_free);
            }
        }
        const float m_scaled = m_row * scale_log2e;   // len >= 1, so m_row is finite
        float l_row = 0.f;
        // ---- pass 2: probabilities -> TMEM (bf16), row sum ----
        for (int j = 0; j < nkb && ok; ++j) {
            if (nkb > 1) {
                if (!(ok = mbar_wait(s_full, n_sfull & 1, abort_flag))) break;
                ++n_sfull;
                tc_fence_after();
            }
            if (j > 0) {   // keeps this thread's view of the pv_done phases in step (S_j was issued after it)
                if (!(ok = mbar_wait(pv_done, n_pvdone & 1, abort_flag))) break;
                ++n_pvdone;
                tc_fence_after();
            }
            const int keys = min(kBlockN, len - j * kBlockN);
            const int kpad = (keys + 15) & ~15;
            if (keys < kpad) {
                // keys of the last 16-group past the end of the sequence get probability 0, but the V
                // rows behind them are whatever follows in memory: clear them so that 0 * junk stays 0
                if (!(ok = mbar_wait(v_full + 8 * j, 0, abort_flag))) break;
                unsigned char* vt = gbase + (sv - base) + j * SM::TILE_BYTES;
                for (int i = threadIdx.x - 64; i < (kpad - keys) * (SM::ROW_BYTES / 16); i += 128)
                    *reinterpret_cast<uint4*>(vt + (size_t)keys * SM::ROW_BYTES + i * 16) = make_uint4(0, 0, 0, 0);
                fence_proxy_async();
            }
            for (int c0 = 0; c0 < kpad; c0 += 32) {
                uint32_t r[32];
                tmem_ld_32x32(lane_addr + kColS + c0, r);
                tmem_ld_wait();
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    float p0 = ex2f(fmaf(__uint_as_float(r[2 * i]), scale_log2e, -m_scaled));
                    float p1 = ex2f(fmaf(__uint_as_float(r[2 * i + 1]), scale_log2e, -m_scaled));
                    if (c0 + 2 * i >= keys) p0 = 0.f;
                    if (c0 + 2 * i + 1 >= keys) p1 = 0.f;
                    l_row += p0 + p1;
                    pk[i] = pack_bf16(p0, p1);
                }
                tmem_st_32x16(lane_addr + kColP + (c0 >> 1), pk);
            }
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(p_full);
        }
        // ---- O / sum -> bf16 -> global ----
        if (ok && (ok = mbar_wait(pv_done, n_pvdone & 1, abort_flag))) {
            tc_fence_after();
            const float inv = l_row > 0.f ? 1.0f / l_row : 0.f;
            __nv_bfloat16* orow = ctx + (size_t)(row0 + qrow) * H + head * D;
#pragma unroll
            for (int c0 = 0; c0 < D; c0 += 32) {
                uint32_t r[32];
                tmem_ld_32x32(lane_addr + kColO + c0, r);
                tmem_ld_wait();
                if (qrow < len) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        uint4 q;
                        q.x = pack_bf16(__uint_as_float(r[8 * i + 0]) * inv, __uint_as_float(r[8 * i + 1]) * inv);
                        q.y = pack_bf16(__uint_as_float(r[8 * i + 2]) * inv, __uint_as_float(r[8 * i + 3]) * inv);
                        q.z = pack_bf16(__uint_as_float(r[8 * i + 4]) * inv, __uint_as_float(r[8 * i + 5]) * inv);
                        q.w = pack_bf16(__uint_as_float(r[8 * i + 6]) * inv, __uint_as_float(r[8 * i + 7]) * inv);
                        *(reinterpret_cast<uint4*>(orow + c0) + i) = q;
                    }
                }
            }
        }
    }
    // ---------------------------------------------------------------- teardown
    if (*abort_flag) {
        if (threadIdx.x == 0 && status) atomicOr(status, RLX_DEVSTAT_TIMEOUT_BIT);
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

}  // namespace tca
}  // namespace rlx
