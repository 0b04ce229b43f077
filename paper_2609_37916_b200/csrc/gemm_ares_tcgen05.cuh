// "Linear" GEMM with the activation block RESIDENT in shared memory, for short contractions
// (K <= 384, i.e. the QKV, attention-output and FFN-up projections of a 384-wide encoder):
//
//     out[M,N] = epilogue(A[M,K] W[N,K]^T + bias)          A, W, out bf16; fp32 accumulation
//
// Why: with K = 384 a 128 x 256 output tile has only six 64-wide k-blocks, and streaming A and W for
// every tile (48 KB per k-block) asks more of the L2 -> SM path than it delivers while the tensor pipe
// runs; the operand feed, not the MMA, paces the ordinary kernel.  Here a pair of CTAs (cta_group::2)
// keeps its 256 rows of A (all K columns, 96 KB per CTA) in shared memory and walks the n-tiles of
// those rows, so per k-block each CTA pulls only HALF of a W tile (BLOCK_N/2 x 64, 12 to 16 KB): a
// third of the bytes per MMA, A read from HBM exactly once, and a W ring deep enough (3 to 6 stages of
// two k-blocks each, one barrier round per stage) to hold a whole tile's operands in flight.
//   warp 0      TMA producer: the A k-blocks of the next row block are refilled one by one as the
//               last n-tile of the current block releases them (interleaved with that tile's W loads,
//               so the switch costs no bubble), W half-tiles stream through the ring
//   warp 1      leader CTA only: tcgen05.mma.cta_group::2 (M = 256, N = BLOCK_N, K = 16) into one of two
//               TMEM accumulator buffers; commits release ring stages, A k-blocks and accumulators in
//               both CTAs (multicast commit; no multicast load anywhere)
//   warps 2..   the epilogue of gemm_tcgen05.cuh (EpilogueTile), each CTA draining its own 128 rows
// Work unit = (256-row block, group of n-tiles); the group size is chosen on the device from the actual
// row count (packed batches) so that the pairs stay balanced.  Waits are bounded as in the plain GEMM.
#pragma once
#include "gemm_tcgen05.cuh"

namespace rlx {
namespace tcar {

using namespace rlx::tc;

constexpr int kMaxKB = 6;        // k-blocks of A kept resident: K <= 384
constexpr int kPairRows = 2 * BLOCK_M;

template <int BLOCK_N>
struct Cfg {
    static constexpr int A_BYTES = BLOCK_M * BLOCK_K * 2;        // one k-block of this CTA's 128 rows
    static constexpr int A_TOTAL = kMaxKB * A_BYTES;
    static constexpr int B_ROWS = BLOCK_N / 2;                   // W rows this CTA loads per k-block
    static constexpr int B_BYTES = B_ROWS * BLOCK_K * 2;
    static constexpr int KPS = 2;                                // k-blocks per ring stage (one barrier round per stage)
    static constexpr int STAGE_BYTES = KPS * B_BYTES;
    static constexpr int A_GROUPS = kMaxKB / KPS;                // A k-blocks are released in the same groups
    static constexpr int EPI_SPLIT = BLOCK_N >= 128 ? BLOCK_N / 64 : 2;
    static constexpr int EPI_WARPS = 4 * EPI_SPLIT;
    static constexpr int THREADS = 64 + 32 * EPI_WARPS;
    static constexpr int SLAB = BLOCK_N / EPI_SPLIT;
    static constexpr int STAGING_BYTES = EPI_WARPS * kStageBufBytes;   // one staging buffer per epilogue warp
    static constexpr int BAR_BYTES = 256;
    static constexpr int RING_BUDGET = 227 * 1024 - 1024 - BAR_BYTES - A_TOTAL - STAGING_BYTES;
    static constexpr int STAGES = (RING_BUDGET / STAGE_BYTES) > 8 ? 8 : (RING_BUDGET / STAGE_BYTES);
    static constexpr int TMEM_COLS = (2 * BLOCK_N <= 128) ? 128 : (2 * BLOCK_N <= 256) ? 256 : 512;
    static constexpr int SMEM_BYTES = A_TOTAL + STAGES * STAGE_BYTES + STAGING_BYTES + BAR_BYTES + 1024;
    static_assert(BLOCK_N % 32 == 0 && BLOCK_N >= 64 && BLOCK_N <= 256, "UMMA N for M = 256");
    static_assert(B_BYTES % 1024 == 0, "ring tiles must stay 1024-byte aligned");
    static_assert(kMaxKB % KPS == 0, "A release groups");
    static_assert(STAGES >= 3, "ring too shallow");
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory");
    static_assert(8 * (2 * STAGES + A_GROUPS + 4) + 16 <= BAR_BYTES, "barrier block");
};

// n-tiles per work unit: the largest divisor of n_tiles whose unit count fills the pairs to at least
// 85 % in the last round, else the one that fills them best.  Same result in every thread.
__device__ __forceinline__ int pick_group(int m_blocks, int n_tiles, int pairs) {
    int best = 1, best_eff = -1;
    for (int g = n_tiles; g >= 1; --g) {
        if (n_tiles % g) continue;
        const int units = m_blocks * (n_tiles / g);
        const int rounds = (units + pairs - 1) / pairs;
        const int eff = units * 1000 / (rounds * pairs);
        if (eff >= 850) return g;
        if (eff > best_eff) { best_eff = eff; best = g; }
    }
    return best;
}

template <int BLOCK_N, int EPI>
__global__ void __launch_bounds__((Cfg<BLOCK_N>::THREADS), 1)
gemm_ares_tcgen05_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                         const __grid_constant__ CUtensorMap tmap_out, const Params p) {
    using C = Cfg<BLOCK_N>;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;   // 128-byte swizzle atoms need 1024-byte alignment
    unsigned char* gbase = smem_raw + (base - raw);
    const uint32_t a_smem = base;
    const uint32_t ring = base + C::A_TOTAL;
    const uint32_t staging = ring + C::STAGES * C::STAGE_BYTES;
    const uint32_t bars = staging + C::STAGING_BYTES;
    // barrier block: full[STAGES], empty[STAGES], a_empty[A_GROUPS], tmem_full[2], tmem_empty[2], tmem slot, abort flag
    const uint32_t full_bar = bars, empty_bar = bars + 8 * C::STAGES, aempty_bar = bars + 16 * C::STAGES;
    const uint32_t tfull_bar = aempty_bar + 8 * C::A_GROUPS, tempty_bar = tfull_bar + 16;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gbase + C::A_TOTAL + C::STAGES * C::STAGE_BYTES + C::STAGING_BYTES +
                                                      16 * C::STAGES + 8 * C::A_GROUPS + 32);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta_rank = cluster_ctarank();   // rank 0 leads the pair
    pdl_launch_dependents();
    if (threadIdx.x == 0) RLX_TRACE(p, 0);

    if (threadIdx.x == 0) {
        for (int i = 0; i < C::STAGES; ++i) {
            mbar_init(full_bar + 8 * i, 1);
            mbar_init(empty_bar + 8 * i, 1);
        }
        for (int i = 0; i < C::A_GROUPS; ++i) mbar_init(aempty_bar + 8 * i, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(tfull_bar + 8 * i, 1);
            mbar_init(tempty_bar + 8 * i, C::EPI_WARPS * 2);   // the leader's barrier collects both CTAs' warps
        }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmap_a);
        prefetch_tmap(&tmap_b);
        prefetch_tmap(&tmap_out);
    }
    if (warp == 1) {
        tmem_alloc<2>(smem_u32(tmem_slot), C::TMEM_COLS);
        tmem_relinquish<2>();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();   // the peer's barriers are initialised before any remote use
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (threadIdx.x == 0) RLX_TRACE(p, 1);
    pdl_wait();   // the previous kernel's outputs are read only from here on
    if (threadIdx.x == 0) RLX_TRACE(p, 2);
    int M = p.M;
    if (p.m_ptr != nullptr) M = min(M, __ldg(p.m_ptr));   // packed activations: only sum(len) rows exist
    const int n_tiles = p.N / BLOCK_N;
    const int m_blocks = (M + kPairRows - 1) / kPairRows;
    const int num_kb = (p.K + BLOCK_K - 1) / BLOCK_K;     // <= kMaxKB (checked by the launcher)
    const int pairs = gridDim.x / 2, pair0 = blockIdx.x / 2;
    const int group = pick_group(m_blocks, n_tiles, pairs);
    const int n_groups = n_tiles / group;
    const int units = m_blocks * n_groups;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (both CTAs; whole warp, one lane issues)
        {
            int stage = 0;
            uint32_t phase = 0, uit = 0;
            bool ok = true;
            for (int unit = pair0; unit < units && ok; unit += pairs, ++uit) {
                const int m_blk = unit / n_groups, ng = unit % n_groups;
                for (int j = 0; j < group && ok; ++j) {
                    const int n_blk = ng * group + (j + pair0) % group;   // staggered start: see the epilogue
                    for (int kb = 0; kb < num_kb; kb += C::KPS) {
                        const int cnt = min(C::KPS, num_kb - kb);   // k-blocks in this stage
                        if (!mbar_wait_warp(empty_bar + 8 * stage, phase ^ 1, abort_flag)) { ok = false; break; }
                        // the first n-tile of a unit brings the unit's A k-blocks in with it, each group as
                        // soon as the previous unit's last MMAs on it have released the buffers
                        const bool load_a = j == 0;
                        if (load_a && !mbar_wait_warp(aempty_bar + 8 * (kb / C::KPS), (uit & 1) ^ 1, abort_flag)) { ok = false; break; }
                        const uint32_t sb = ring + stage * C::STAGE_BYTES;
                        if (elect_one()) {
                            // while the unit's first tile streams in, pull the NEXT unit's A block into L2 so
                            // that its loads, one unit later, do not pay an HBM round trip on the critical path
                            if (load_a && unit + pairs < units) {
                                const int next_m = (unit + pairs) / n_groups;
                                const int nrow = next_m * kPairRows + (int)cta_rank * BLOCK_M;
                                if (p.kblock_maps) tma_prefetch_3d(&tmap_a, 0, nrow, kb);
                                else for (int i = 0; i < cnt; ++i) tma_prefetch_2d(&tmap_a, (kb + i) * BLOCK_K, nrow);
                            }
                            // both CTAs' copies complete on the LEADER's full barrier, which expects all bytes
                            const uint32_t lead_full = map_to_cta(full_bar + 8 * stage, 0);
                            if (RLX_DBG(p, kDbgNoLoad)) {
                                if (cta_rank == 0) mbar_arrive(full_bar + 8 * stage);
                            } else {
                                const bool k3 = p.kblock_maps != 0;   // one 3-D load per operand and stage
                                const int nkb = k3 ? C::KPS : cnt;
                                if (cta_rank == 0)
                                    mbar_expect_tx(full_bar + 8 * stage, 2 * nkb * (C::B_BYTES + (load_a ? C::A_BYTES : 0)));
                                const int arow = m_blk * kPairRows + (int)cta_rank * BLOCK_M;
                                const int brow = n_blk * BLOCK_N + (int)cta_rank * C::B_ROWS;
                                if (k3) {
                                    if (load_a) tma_load_3d_cg2(a_smem + kb * C::A_BYTES, &tmap_a, 0, arow, kb, lead_full);
                                    tma_load_3d_cg2(sb, &tmap_b, 0, brow, kb, lead_full);
                                } else {
                                    for (int i = 0; i < cnt; ++i) {
                                        if (load_a) tma_load_2d_cg2(a_smem + (kb + i) * C::A_BYTES, &tmap_a, (kb + i) * BLOCK_K, arow, lead_full);
                                        tma_load_2d_cg2(sb + i * C::B_BYTES, &tmap_b, (kb + i) * BLOCK_K, brow, lead_full);
                                    }
                                }
                            }
                            if (uit == 0 && j == 0 && kb == 0) RLX_TRACE(p, 3);
                        }
                        __syncwarp();
                        if (++stage == C::STAGES) { stage = 0; phase ^= 1; }
                    }
                }
            }
            if (lane == 0) RLX_TRACE(p, 4);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA; whole warp, one lane issues)
        if (cta_rank == 0) {
            constexpr uint32_t idesc = make_idesc(kPairRows, BLOCK_N);
            int stage = 0;
            uint32_t phase = 0;
            int it = 0;
            bool ok = true;
            if (lane == 0) { RLX_TRACE(p, 9); RLX_TRACE_CLK(p, 14); }
            RLX_CLK_DECL(clk_full);
            RLX_CLK_DECL(clk_tempty);
            for (int unit = pair0; unit < units && ok; unit += pairs) {
                for (int j = 0; j < group && ok; ++j, ++it) {
                    const int as = it & 1;
                    const uint32_t aphase = (it >> 1) & 1;
                    bool got_acc;
                    RLX_CLK_ADD(clk_tempty, got_acc = mbar_wait_warp(tempty_bar + 8 * as, aphase ^ 1, abort_flag));
                    if (!got_acc) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t tmem_d = tmem_base + as * BLOCK_N;
                    for (int kb = 0; kb < num_kb; kb += C::KPS) {
                        const int cnt = min(C::KPS, num_kb - kb);
                        bool got_ops;
                        RLX_CLK_ADD(clk_full, got_ops = mbar_wait_warp(full_bar + 8 * stage, phase, abort_flag));
                        if (!got_ops) { ok = false; break; }
                        tc_fence_after();
                        if (elect_one()) {
                            if (it == 0 && kb == 0) RLX_TRACE(p, 5);
                            if (!RLX_DBG(p, kDbgNoMma)) {
                                for (int i = 0; i < cnt; ++i) {
                                    const uint64_t adesc = make_smem_desc(a_smem + (kb + i) * C::A_BYTES);
                                    const uint64_t bdesc = make_smem_desc(ring + stage * C::STAGE_BYTES + i * C::B_BYTES);
#pragma unroll
                                    for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
                                        umma_bf16<2>(tmem_d, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | i | k) != 0 ? 1u : 0u);
                                }
                            }
                            umma_commit<2>(empty_bar + 8 * stage);                                   // ring stage reusable
                            if (j == group - 1) umma_commit<2>(aempty_bar + 8 * (kb / C::KPS));      // last reader of these A k-blocks
                        }
                        __syncwarp();
                        if (++stage == C::STAGES) { stage = 0; phase ^= 1; }
                    }
                    if (ok && elect_one()) {
                        umma_commit<2>(tfull_bar + 8 * as);   // accumulator complete
                        if (it == 0) RLX_TRACE(p, 6);
                    }
                    __syncwarp();
                }
            }
            if (lane == 0) {
                RLX_TRACE(p, 7);
                RLX_TRACE_CLK(p, 15);
                RLX_TRACE_VAL(p, 10, clk_full);
                RLX_TRACE_VAL(p, 11, clk_tempty);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue warps
        const int ew = warp - 2;
        const int quad = warp & 3;            // TMEM lane quadrant this warp may read
        const int slab = ew >> 2;             // which column slab of the tile
        const uint32_t stg = staging + ew * kStageBufBytes;
        int it = 0;
        bool ok = true;
        for (int unit = pair0; unit < units && ok; unit += pairs) {
            const int m_blk = unit / n_groups, ng = unit % n_groups;
            const int m_row0 = m_blk * kPairRows + (int)cta_rank * BLOCK_M + quad * 32;
            for (int j = 0; j < group; ++j, ++it) {
                const int as = it & 1;
                const uint32_t aphase = (it >> 1) & 1;
                // pairs start their walk over the n-tiles at different tiles, so that at any moment they
                // pull different parts of W through L2 instead of all hitting the same lines
                const int n0 = (ng * group + (j + pair0) % group) * BLOCK_N + slab * C::SLAB;
                {   // bias of the tile after this one (the next n-tile of the unit, else the next unit's first)
                    const int nj = j + 1 < group ? j + 1 : 0;
                    const int nng = j + 1 < group ? ng : ((unit + pairs) % n_groups);
                    EpilogueTile<EPI, C::SLAB / 32>::prefetch_bias(p, (nng * group + (nj + pair0) % group) * BLOCK_N + slab * C::SLAB);
                }
                const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + as * BLOCK_N + slab * C::SLAB;
                EpilogueTile<EPI, C::SLAB / 32> et;
                et.prefetch(p, M, m_row0 + lane, n0);
                if (!mbar_wait(tfull_bar + 8 * as, aphase, abort_flag)) { ok = false; break; }
                tc_fence_after();
                if (ew == 0 && lane == 0 && it < 12) RLX_TRACE(p, 16 + it);
                et.template drain<2>(p, &tmap_out, M, m_row0, n0, taddr, stg, lane, tempty_bar + 8 * as, cta_rank,
                                     (ew == 0 && lane == 0 && (it == 1 || it == 5)) ? 40 + 2 * (it - 1) : -1);
                if (ew == 0 && lane == 0 && it < 12) RLX_TRACE(p, 28 + it);
            }
        }
        EpilogueTile<EPI, C::SLAB / 32>::finish(lane);
        if (ew == 0 && lane == 0) RLX_TRACE(p, 8);
    }

    // ---------------------------------------------------------------- teardown
    if (*abort_flag) {
        if (threadIdx.x == 0 && p.status) atomicOr(p.status, RLX_DEVSTAT_TIMEOUT_BIT);
        // give copies that may still be in flight time to land before shared memory is released
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) RLX_TRACE(p, 12);
    cluster_sync_all();   // neither CTA leaves while the pair still uses its memory
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc<2>(tmem_base, C::TMEM_COLS);
        if (lane == 0) RLX_TRACE(p, 13);
    }
}

}  // namespace tcar
}  // namespace rlx
