// Projection + bias + residual + LayerNorm with the row statistics formed ACROSS a thread-block
// cluster:  out = LN(A W^T + bias + residual; gamma, beta),  N = cluster_size * BLOCK_N.
//
// The CTAs of a cluster take the same 128 rows and one BLOCK_N-wide column slab each (cluster rank =
// column tile).  Every CTA is the ordinary pipelined GEMM (TMA ring -> tcgen05.mma -> double-buffered
// TMEM accumulators); only the epilogue differs: a warp reads its 32 rows x SLAB columns into
// registers, adds bias and residual, and the partial row sums go to every peer's shared memory with
// st.shared::cluster followed by a release-arrive on the peer's mbarrier (no multicast, no global
// round trip).  Two exchanges per tile (sum, then centred sum of squares: the same two-pass variance
// as the stand-alone kernel), then each CTA normalises and stores its own slab.  Tiles stay small
// (all SMs busy even for a few hundred rows) and the hidden size may be anything up to 8 slabs.
// The exchange buffers are safe to reuse tile after tile because a CTA can only run ahead of a peer
// by less than one exchange: it cannot pass barrier k+1 of a tile before every peer has arrived
// there, i.e. finished reading buffer k.
#pragma once
#include "gemm_tcgen05.cuh"

namespace rlx {
namespace tccl {

using namespace rlx::tc;

constexpr int kMaxCluster = 8;

template <int BLOCK_N>
struct Cfg {
    static constexpr int A_BYTES = BLOCK_M * BLOCK_K * 2;
    static constexpr int B_BYTES = BLOCK_N * BLOCK_K * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int EPI_SPLIT = BLOCK_N >= 192 ? BLOCK_N / 64 : 2;
    static constexpr int EPI_WARPS = 4 * EPI_SPLIT;
    static constexpr int THREADS = 64 + 32 * EPI_WARPS;
    static constexpr int SLAB = BLOCK_N / EPI_SPLIT;
    static constexpr int STAGING_BYTES = EPI_WARPS * kStageBufBytes;
    static constexpr int XCHG_FLOATS = kMaxCluster * EPI_SPLIT * BLOCK_M;   // one statistic: [rank][slab][row]
    static constexpr int XCHG_BYTES = 2 * XCHG_FLOATS * 4;                  // sum and centred squares
    static constexpr int RING_BUDGET = 222 * 1024 - STAGING_BYTES - XCHG_BYTES;
    static constexpr int STAGES = (RING_BUDGET / STAGE_BYTES) > 8 ? 8 : (RING_BUDGET / STAGE_BYTES);
    static constexpr int TMEM_COLS = (2 * BLOCK_N <= 128) ? 128 : (2 * BLOCK_N <= 256) ? 256 : 512;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + STAGING_BYTES + XCHG_BYTES + 256 + 1024;
    static_assert(BLOCK_N == 64 || BLOCK_N == 128 || BLOCK_N == 192, "slab widths of the clustered LayerNorm GEMM");
};

__device__ __forceinline__ uint32_t cluster_nctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void st_cluster_f32(uint32_t cluster_addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(cluster_addr), "f"(v) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    uint32_t spins = 0;
    while (!mbar_try_wait_cluster(bar, parity)) {
        if ((++spins & 0xff) == 0) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > kWaitBudgetNs) {
                *abort_flag = 1;
                return false;
            }
        }
    }
    return true;
}

struct Params {
    const float* bias;               // [N]
    const __nv_bfloat16* residual;   // [M,N]
    const float* gamma;              // [N]
    const float* beta;               // [N]
    __nv_bfloat16* out;              // [M,N]
    float eps;
    int M, N, K;
    int32_t* status;
    const int32_t* m_ptr;            // optional device row count
};

template <int BLOCK_N>
__global__ void __launch_bounds__((Cfg<BLOCK_N>::THREADS), 1)
gemm_cln_tcgen05_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b, const Params p) {
    using C = Cfg<BLOCK_N>;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* gbase = smem_raw + (base - raw);
    const uint32_t staging = base + C::STAGES * C::STAGE_BYTES;
    const uint32_t xchg = staging + C::STAGING_BYTES;                                 // shared::cta address
    const float* xchg_local = reinterpret_cast<const float*>(gbase + C::STAGES * C::STAGE_BYTES + C::STAGING_BYTES);
    const uint32_t bars = xchg + C::XCHG_BYTES;
    const uint32_t full_bar = bars, empty_bar = bars + 8 * C::STAGES;
    const uint32_t tfull_bar = bars + 16 * C::STAGES, tempty_bar = tfull_bar + 16, x_bar = tfull_bar + 32;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gbase + C::STAGES * C::STAGE_BYTES + C::STAGING_BYTES +
                                                      C::XCHG_BYTES + 16 * C::STAGES + 48);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank(), nranks = cluster_nctarank();
    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        for (int i = 0; i < C::STAGES; ++i) {
            mbar_init(full_bar + 8 * i, 1);
            mbar_init(empty_bar + 8 * i, 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(tfull_bar + 8 * i, 1);
            mbar_init(tempty_bar + 8 * i, C::EPI_WARPS);
            mbar_init(x_bar + 8 * i, C::EPI_WARPS * nranks);   // every epilogue warp of every CTA of the cluster
        }
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
    cluster_sync_all();   // peers' exchange barriers exist before anyone arrives on them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    pdl_wait();
    int M = p.M;
    if (p.m_ptr != nullptr) M = min(M, __ldg(p.m_ptr));
    const int m_tiles = (M + BLOCK_M - 1) / BLOCK_M;
    const int num_kb = (p.K + BLOCK_K - 1) / BLOCK_K;
    const int tile0 = blockIdx.x / nranks, tile_step = gridDim.x / nranks;   // the whole cluster walks the same row blocks
    const int n_blk = (int)rank;

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int mb = tile0; mb < m_tiles && ok; mb += tile_step) {
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(empty_bar + 8 * stage, phase ^ 1, abort_flag)) { ok = false; break; }
                    const uint32_t sa = base + stage * C::STAGE_BYTES, sb = sa + C::A_BYTES;
                    mbar_expect_tx(full_bar + 8 * stage, C::STAGE_BYTES);
                    tma_load_2d(sa, &tmap_a, kb * BLOCK_K, mb * BLOCK_M, full_bar + 8 * stage);
                    tma_load_2d(sb, &tmap_b, kb * BLOCK_K, n_blk * BLOCK_N, full_bar + 8 * stage);
                    if (++stage == C::STAGES) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc(BLOCK_M, BLOCK_N);
            int stage = 0;
            uint32_t phase = 0;
            int it = 0;
            bool ok = true;
            for (int mb = tile0; mb < m_tiles && ok; mb += tile_step, ++it) {
                const int as = it & 1;
                const uint32_t aphase = (it >> 1) & 1;
                if (!mbar_wait(tempty_bar + 8 * as, aphase ^ 1, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + as * BLOCK_N;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(full_bar + 8 * stage, phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = base + stage * C::STAGE_BYTES, sb = sa + C::A_BYTES;
                    const uint64_t adesc = make_smem_desc(sa), bdesc = make_smem_desc(sb);
#pragma unroll
                    for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
                        umma_bf16<1>(tmem_d, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
                    umma_commit<1>(empty_bar + 8 * stage);
                    if (++stage == C::STAGES) { stage = 0; phase ^= 1; }
                }
                if (ok) umma_commit<1>(tfull_bar + 8 * as);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue
        constexpr int SLAB = C::SLAB;
        constexpr int NC = SLAB / 32;
        const int ew = warp - 2;
        const int quad = warp & 3;
        const int slab = ew >> 2;
        const int row = quad * 32 + lane;
        const uint32_t stg = staging + ew * kStageBufBytes;
        const uint32_t row_off = lane * 64;
        const uint32_t swz = (uint32_t)((lane >> 1) & 3);
        const float inv_n = 1.0f;   // (division by N is done explicitly below)
        (void)inv_n;
        int it = 0;
        bool ok = true;
        for (int mb = tile0; mb < m_tiles && ok; mb += tile_step, ++it) {
            const int as = it & 1;
            const uint32_t aphase = (it >> 1) & 1;
            const int m = mb * BLOCK_M + row;
            const bool row_ok = m < M;
            const int n0 = n_blk * BLOCK_N + slab * SLAB;
            // residual first: its latency hides behind the accumulator wait
            uint4 res[NC][4];
            {
                const __nv_bfloat16* rrow = p.residual + (size_t)(row_ok ? m : 0) * p.N + n0;
#pragma unroll
                for (int c = 0; c < NC; ++c)
#pragma unroll
                    for (int i = 0; i < 4; ++i) res[c][i] = __ldg(reinterpret_cast<const uint4*>(rrow + c * 32) + i);
            }
            if (!mbar_wait(tfull_bar + 8 * as, aphase, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + as * BLOCK_N + slab * SLAB;
            float v[NC * 32];
            float sum = 0.f;
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                uint32_t r[32];
                tmem_ld_32x32(taddr + c * 32, r);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float4 b4 = __ldg(reinterpret_cast<const float4*>(p.bias + n0 + c * 32) + i);
                    const uint32_t w0 = (i & 1) ? res[c][i >> 1].z : res[c][i >> 1].x;
                    const uint32_t w1 = (i & 1) ? res[c][i >> 1].w : res[c][i >> 1].y;
                    v[c * 32 + 4 * i + 0] = __uint_as_float(r[4 * i + 0]) + b4.x + bf16lo(w0);
                    v[c * 32 + 4 * i + 1] = __uint_as_float(r[4 * i + 1]) + b4.y + bf16hi(w0);
                    v[c * 32 + 4 * i + 2] = __uint_as_float(r[4 * i + 2]) + b4.z + bf16lo(w1);
                    v[c * 32 + 4 * i + 3] = __uint_as_float(r[4 * i + 3]) + b4.w + bf16hi(w1);
                    sum += (v[c * 32 + 4 * i + 0] + v[c * 32 + 4 * i + 1]) + (v[c * 32 + 4 * i + 2] + v[c * 32 + 4 * i + 3]);
                }
            }
            // the accumulator is in registers: hand the TMEM buffer back to the MMA warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar + 8 * as);

            // ---- exchange 1: partial row sums to every CTA of the cluster ----
            const uint32_t slot = (uint32_t)(((int)rank * C::EPI_SPLIT + slab) * BLOCK_M + row) * 4u;
            for (uint32_t peer = 0; peer < nranks; ++peer) st_cluster_f32(map_to_cta(xchg + slot, peer), sum);
            __syncwarp();
            if (lane == 0)
                for (uint32_t peer = 0; peer < nranks; ++peer) mbar_arrive_cluster(map_to_cta(x_bar, peer));
            if (!mbar_wait_cluster(x_bar, it & 1, abort_flag)) { ok = false; break; }
            float tot = 0.f;
            for (uint32_t q = 0; q < nranks * C::EPI_SPLIT; ++q) tot += xchg_local[q * BLOCK_M + row];
            const float mean = tot / (float)p.N;
            // ---- exchange 2: centred sums of squares ----
            float sq = 0.f;
#pragma unroll
            for (int i = 0; i < NC * 32; ++i) {
                v[i] -= mean;
                sq = fmaf(v[i], v[i], sq);
            }
            for (uint32_t peer = 0; peer < nranks; ++peer)
                st_cluster_f32(map_to_cta(xchg + C::XCHG_FLOATS * 4 + slot, peer), sq);
            __syncwarp();
            if (lane == 0)
                for (uint32_t peer = 0; peer < nranks; ++peer) mbar_arrive_cluster(map_to_cta(x_bar + 8, peer));
            if (!mbar_wait_cluster(x_bar + 8, it & 1, abort_flag)) { ok = false; break; }
            float tsq = 0.f;
            for (uint32_t q = 0; q < nranks * C::EPI_SPLIT; ++q) tsq += xchg_local[C::XCHG_FLOATS + q * BLOCK_M + row];
            const float rstd = 1.0f / sqrtf(tsq / (float)p.N + p.eps);
            // ---- normalise, bf16, transposed stores ----
            const int m_row0 = mb * BLOCK_M + quad * 32;
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                __syncwarp();
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float4 g0 = __ldg(reinterpret_cast<const float4*>(p.gamma + n0 + c * 32) + 2 * i);
                    const float4 g1 = __ldg(reinterpret_cast<const float4*>(p.gamma + n0 + c * 32) + 2 * i + 1);
                    const float4 b0 = __ldg(reinterpret_cast<const float4*>(p.beta + n0 + c * 32) + 2 * i);
                    const float4 b1 = __ldg(reinterpret_cast<const float4*>(p.beta + n0 + c * 32) + 2 * i + 1);
                    const float* vv = v + c * 32 + 8 * i;
                    uint4 q;
                    q.x = pack_bf16(vv[0] * rstd * g0.x + b0.x, vv[1] * rstd * g0.y + b0.y);
                    q.y = pack_bf16(vv[2] * rstd * g0.z + b0.z, vv[3] * rstd * g0.w + b0.w);
                    q.z = pack_bf16(vv[4] * rstd * g1.x + b1.x, vv[5] * rstd * g1.y + b1.y);
                    q.w = pack_bf16(vv[6] * rstd * g1.z + b1.z, vv[7] * rstd * g1.w + b1.w);
                    st_shared_v4(stg + row_off + (((uint32_t)i ^ swz) << 4), q);
                }
                __syncwarp();
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int rr = i * 8 + (lane >> 2), cc = lane & 3;
                    const uint4 q = ld_shared_v4(stg + rr * 64 + (((uint32_t)cc ^ (uint32_t)((rr >> 1) & 3)) << 4));
                    if (m_row0 + rr < M)
                        *reinterpret_cast<uint4*>(p.out + (size_t)(m_row0 + rr) * p.N + n0 + c * 32 + cc * 8) = q;
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
    cluster_sync_all();   // no CTA leaves while a peer may still write into it or arrive on its barriers
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc<1>(tmem_base, C::TMEM_COLS);
    }
}

}  // namespace tccl
}  // namespace rlx
