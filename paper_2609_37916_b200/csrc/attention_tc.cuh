// Packed-sequence attention on the 5th-generation tensor cores (tcgen05 + TMEM), head_dim 32 or 64,
// up to 512 keys per sequence, ONE pass over the keys, persistent CTAs (two per SM).
//
// A work item is 128 query rows of one (sequence, head), numbered batch x query tile x head.  The TMA
// lane hands out items -- from a global ticket counter when the caller provides one (long and short
// sequences then balance by themselves), else with a fixed stride -- skips tiles past a sequence's
// end and publishes each item number through a small ring in shared memory; the other roles follow.
//
//   warp 0 (1 lane)   item ring + TMA: the item's Q tile (two-slot ring) and its K / V blocks of 64
//                     keys (ring of stages shared by all items), straight out of the packed
//                     [rows, 3H] projection; it runs ahead of the math across item boundaries
//   warp 1 (1 lane)   MMA issue:  S = Q K^T  (M=128, N=keys, K=d) into a ring of S buffers in tensor
//                                 memory, ahead of the softmax;
//                                 O += P V     (M=128, N=d, K=keys; P read from TMEM, V MN-major)
//   warps 2..5        softmax, one thread per query row (TMEM lane = row: row max and row sum are
//                     per-thread loops, no shuffles).  The 64 scores of a block sit in registers as two
//                     halves; the next block's halves are requested as soon as a half's exponentials
//                     have been taken, so the tensor-memory latency hides behind the MUFU work.
//
// Online softmax without a correction step in the common case: the reference maximum m of a row is the
// maximum of its first block; a later block keeps it unless its own maximum exceeds it by more than 8
// in the exponent of two (then p <= 256: well inside bf16's range, and the row sum stays far from
// overflow).  Only then does the warp wait for the products already issued, scale its rows of O in
// tensor memory by 2^(m_old - m_new) and move m.  The final division by the row sum removes the common
// factor, so the result does not depend on which m was used.
// TMEM per CTA (256 columns): (256 - 2d)/64 S/P buffers of 64 columns, then two O accumulators (d
// columns each, alternating between items so that the next item's products need not wait for the
// previous item's output rows to be read).
// All mbarrier waits are bounded; on expiry the CTA sets the status bit and leaves.
#pragma once
#include <cuda.h>
#include "common.cuh"
#include "gemm_tcgen05.cuh"

namespace rlx {
namespace tca {

using namespace rlx::tc;

constexpr int kThreads = 192;  // TMA warp, MMA warp, four softmax warps
constexpr int kBlockM = 128;   // query rows per work item
constexpr int kBlockN = 64;    // keys per block
constexpr int kMaxBlocks = 8;  // 512 keys
constexpr int kTmemCols = 256;
constexpr int kPvRing = 8;     // completion barriers of the P V products, indexed by block number
constexpr int kItemRing = 8;   // published item numbers
constexpr float kRescaleAbove = 8.f;   // exp2 units a block maximum may exceed the row's reference maximum

template <int D>
struct Smem {
    static constexpr int ROW_BYTES = D * 2;                  // 64 (64-byte swizzle) or 128 (128-byte swizzle)
    static constexpr int TILE_BYTES = kBlockN * ROW_BYTES;   // one 64-row tile of K or V (Q is two of them)
    static constexpr int S_BUFS = (kTmemCols - 2 * D) / kBlockN;
    static constexpr int COL_O = S_BUFS * kBlockN;
    static constexpr int STAGES = D == 32 ? 10 : 5;          // K+V stages: 80 KB, Q ring 16 / 32 KB
    static constexpr int Q_OFF = 0, KV_OFF = 4 * TILE_BYTES, BAR_OFF = KV_OFF + STAGES * 2 * TILE_BYTES;
    static constexpr int BYTES = BAR_OFF + 512 + 1024;
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
__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ float max3f(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2f_pinned(float x) {
    float y;
    asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}


// One work item, decoded from its number.
struct Item {
    int head, q0, len, row0, nkb;
    __device__ bool decode(int cand, int qtiles, int heads, const int32_t* seq_start, const int32_t* seq_len) {
        const int b = cand / (qtiles * heads), rem = cand % (qtiles * heads);
        q0 = (rem / heads) * kBlockM;
        len = __ldg(seq_len + b);
        if (q0 >= len) return false;
        head = rem % heads;
        row0 = __ldg(seq_start + b);
        nkb = (len + kBlockN - 1) / kBlockN;
        return true;
    }
};

// A consumer's view of the item ring: items in publication order, -1 ends the list.
struct ItemReader {
    uint32_t n;        // items read so far
    uint32_t g0;       // key blocks of all earlier items
    Item it;
    // returns 1: item ready, 0: end of list, -1: a wait ran out.  WARP: all 32 lanes read together and
    // `arrive` is true in one of them; otherwise a single lane calls.
    template <bool WARP>
    __device__ int next(uint32_t item_full, uint32_t item_free, const volatile int* ring, bool arrive, int qtiles,
                        int heads, const int32_t* seq_start, const int32_t* seq_len, volatile int* abort_flag) {
        const uint32_t slot = n % kItemRing;
        if (!mbar_wait(item_full + 8 * slot, (n / kItemRing) & 1, abort_flag)) return -1;
        const int cand = ring[slot];
        if (WARP) __syncwarp();
        if (arrive) mbar_arrive(item_free + 8 * slot);
        g0 += it.nkb;
        ++n;
        if (cand < 0) return 0;
        it.decode(cand, qtiles, heads, seq_start, seq_len);
        return 1;
    }
};

#ifdef RLX_ATTN_TRACE
#define ATT_TR(role, code) do { if (blockIdx.x == 0 && tr_cnt < 250) { \
    reinterpret_cast<unsigned long long*>(status)[(role) * 256 + tr_cnt++] = ((unsigned long long)clock64() << 8) | (code); } } while (0)
#else
#define ATT_TR(role, code) do { } while (0)
#endif

template <int D>
__global__ void __launch_bounds__(kThreads, 2)
attention_tc_kernel(const __grid_constant__ CUtensorMap tmap_qkv, const int32_t* __restrict__ seq_start,
                    const int32_t* __restrict__ seq_len, __nv_bfloat16* __restrict__ ctx, int H,
                    float scale_log2e, int batch, int qtiles, unsigned int* ticket, int32_t* status) {
    using SM = Smem<D>;
    constexpr int NSB = SM::S_BUFS, NST = SM::STAGES, COL_O = SM::COL_O;
    pdl_launch_dependents();
    pdl_wait();
    const int heads = H / D;

    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* gbase = smem_raw + (base - raw);
    const uint32_t sq = base + SM::Q_OFF, skv = base + SM::KV_OFF;
    const uint32_t bars = base + SM::BAR_OFF;
    const uint32_t q_full = bars, q_free = q_full + 16, kv_full = q_free + 16, kv_free = kv_full + 8 * NST;
    const uint32_t s_full = kv_free + 8 * NST, p_full = s_full + 8 * NSB, pv_done = p_full + 8 * NSB;
    const uint32_t o_free = pv_done + 8 * kPvRing, item_full = o_free + 16, item_free = item_full + 8 * kItemRing;
    constexpr int kBarBytes = 8 * (4 + 2 * NST + 2 * NSB + kPvRing + 2 + 2 * kItemRing);
    static_assert(kBarBytes + 4 * kItemRing + 8 <= 512, "barrier block");
    volatile int* ring = reinterpret_cast<volatile int*>(gbase + SM::BAR_OFF + kBarBytes);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gbase + SM::BAR_OFF + kBarBytes + 4 * kItemRing);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int i = 0; i < 2; ++i) { mbar_init(q_full + 8 * i, 1); mbar_init(q_free + 8 * i, 1); mbar_init(o_free + 8 * i, 4); }
        for (int i = 0; i < NST; ++i) { mbar_init(kv_full + 8 * i, 1); mbar_init(kv_free + 8 * i, 1); }
        for (int i = 0; i < NSB; ++i) { mbar_init(s_full + 8 * i, 1); mbar_init(p_full + 8 * i, 4); }
        for (int i = 0; i < kPvRing; ++i) mbar_init(pv_done + 8 * i, 1);
        for (int i = 0; i < kItemRing; ++i) { mbar_init(item_full + 8 * i, 1); mbar_init(item_free + 8 * i, 5); }
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
    const int n_cand = batch * qtiles * heads;
    int tr_cnt = 0;
    (void)tr_cnt;

    if (warp == 0) {
        // ------------------------------------------------------------ items, then TMA: Q, K_j, V_j
        if (lane == 0) {
            bool ok = true;
            uint32_t n = 0, g0 = 0;      // items published, key blocks of all earlier items
            int next_static = blockIdx.x;
            for (;;) {
                Item it;
                int cand;
                for (;;) {               // draw until a tile that exists, or the end of the list
                    if (ticket) {
                        cand = (int)atomicAdd(ticket, 1u);
                        // every CTA draws exactly one ticket >= n_cand; the last of those re-arms the counter
                        if (cand == n_cand + (int)gridDim.x - 1) atomicExch(ticket, 0u);
                    } else {
                        cand = next_static;
                        next_static += gridDim.x;
                    }
                    if (cand >= n_cand) { cand = -1; break; }
                    if (it.decode(cand, qtiles, heads, seq_start, seq_len)) break;
                }
                const uint32_t slot = n % kItemRing;
                if (n >= kItemRing && !(ok = mbar_wait(item_free + 8 * slot, ((n / kItemRing) - 1) & 1, abort_flag))) break;
                ring[slot] = cand;
                mbar_arrive(item_full + 8 * slot);   // release: orders the store above
                if (cand < 0) break;
                const uint32_t qs = n & 1;
                if (n >= 2 && !(ok = mbar_wait(q_free + 8 * qs, ((n >> 1) - 1) & 1, abort_flag))) break;
                const uint32_t qdst = sq + qs * 2 * SM::TILE_BYTES;
                mbar_expect_tx(q_full + 8 * qs, 2 * SM::TILE_BYTES);
                tma_load_2d(qdst, &tmap_qkv, it.head * D, it.row0 + it.q0, q_full + 8 * qs);
                tma_load_2d(qdst + SM::TILE_BYTES, &tmap_qkv, it.head * D, it.row0 + it.q0 + kBlockN, q_full + 8 * qs);
                for (int j = 0; j < it.nkb; ++j) {
                    const uint32_t g = g0 + j, st = g % NST, use = g / NST;
                    if (use >= 1 && !(ok = mbar_wait(kv_free + 8 * st, (use - 1) & 1, abort_flag))) break;
                    const uint32_t dst = skv + st * 2 * SM::TILE_BYTES;
                    mbar_expect_tx(kv_full + 8 * st, 2 * SM::TILE_BYTES);
                    tma_load_2d(dst, &tmap_qkv, H + it.head * D, it.row0 + j * kBlockN, kv_full + 8 * st);
                    tma_load_2d(dst + SM::TILE_BYTES, &tmap_qkv, 2 * H + it.head * D, it.row0 + j * kBlockN, kv_full + 8 * st);
                }
                if (!ok) break;
                g0 += it.nkb;
                ++n;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issue
        if (lane == 0) {
            // The ring is read once, by the S cursor; the P V cursor replays the items from a private queue
            // (it is at most S_BUFS blocks, hence at most S_BUFS items, behind).
            ItemReader sc;
            sc.n = 0; sc.g0 = 0; sc.it.nkb = 0;
            Item q_items[4];
            uint32_t q_g0[4];
            uint32_t s_items = 0;        // items the S cursor has opened
            int s_state = sc.next<false>(item_full, item_free, ring, true, qtiles, heads, seq_start, seq_len, abort_flag);
            if (s_state == 1) { q_items[0] = sc.it; q_g0[0] = sc.g0; s_items = 1; }
            int sj = 0;
            bool ok = s_state >= 0;
            auto issue_next_s = [&]() -> bool {
                if (s_state != 1) return s_state == 0;
                const uint32_t item_no = sc.n - 1;
                const uint32_t g = sc.g0 + sj, st = g % NST, sb = g % NSB, qs = item_no & 1;
                if (sj == 0 && !mbar_wait(q_full + 8 * qs, (item_no >> 1) & 1, abort_flag)) return false;
                if (!mbar_wait(kv_full + 8 * st, (g / NST) & 1, abort_flag)) return false;
                tc_fence_after();
                const int keys = min(kBlockN, sc.it.len - sj * kBlockN);
                const int n = (keys + 15) & ~15;                       // UMMA N: multiple of 16
                const uint32_t idesc = idesc_attn(kBlockM, n, 0);
                const uint64_t qdesc = desc_kmajor<D>(sq + qs * 2 * SM::TILE_BYTES);
                const uint64_t kdesc = desc_kmajor<D>(skv + st * 2 * SM::TILE_BYTES);
#pragma unroll
                for (int k = 0; k < D / 16; ++k)
                    umma_bf16<1>(tmem + sb * kBlockN, qdesc + 2 * k, kdesc + 2 * k, idesc, k != 0);
                umma_commit<1>(s_full + 8 * sb);
                if (++sj == sc.it.nkb) {
                    umma_commit<1>(q_free + 8 * qs);   // the item's last read of its Q tile
                    s_state = sc.next<false>(item_full, item_free, ring, true, qtiles, heads, seq_start, seq_len, abort_flag);
                    if (s_state == 1) { q_items[s_items & 3] = sc.it; q_g0[s_items & 3] = sc.g0; ++s_items; }
                    sj = 0;
                    if (s_state < 0) return false;
                }
                return true;
            };
            for (int i = 0; i < NSB - 1 && ok; ++i) ok = issue_next_s();
            for (uint32_t pi = 0; ok && pi < s_items; ++pi) {   // s_items grows while the S cursor runs ahead
                const Item it = q_items[pi & 3];
                const uint32_t pg0 = q_g0[pi & 3];
                const uint32_t os = pi & 1;
                for (int j = 0; j < it.nkb; ++j) {
                    const uint32_t g = pg0 + j, st = g % NST, sb = g % NSB;
                    // the next S goes where P_{g-1} lives: the product that reads it must have finished
                    if (g >= 1 && !(ok = mbar_wait(pv_done + 8 * ((g - 1) % kPvRing), ((g - 1) / kPvRing) & 1, abort_flag))) break;
                    ATT_TR(1, 1);
                    if (!(ok = issue_next_s())) break;
                    ATT_TR(1, 2);
                    if (!(ok = mbar_wait(p_full + 8 * sb, (g / NSB) & 1, abort_flag))) break;
                    ATT_TR(1, 3);
                    // first product into this O accumulator since the item two back: its rows must have been read
                    if (j == 0 && pi >= 2 && !(ok = mbar_wait(o_free + 8 * os, ((pi >> 1) - 1) & 1, abort_flag))) break;
                    tc_fence_after();
                    const int keys = min(kBlockN, it.len - j * kBlockN);
                    const int ksteps = (keys + 15) >> 4;
                    const uint32_t idesc = idesc_attn(kBlockM, D, 1);
                    const uint64_t vdesc = desc_mnmajor<D>(skv + st * 2 * SM::TILE_BYTES + SM::TILE_BYTES);
                    for (int kk = 0; kk < ksteps; ++kk) {
                        // 16 keys = two 8-row groups of ROW_BYTES rows further down the V tile
                        umma_ts(tmem + COL_O + os * D, tmem + sb * kBlockN + kk * 8,
                                vdesc + (uint64_t)((16 * D * 2) >> 4) * kk, idesc, (j | kk) != 0);
                    }
                    umma_commit<1>(kv_free + 8 * st);
                    umma_commit<1>(pv_done + 8 * (g % kPvRing));
                    ATT_TR(1, 4);
                }
            }
        }
    } else {
        // ------------------------------------------------------------ softmax warps (thread = query row)
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
        ItemReader rd;
        rd.n = 0; rd.g0 = 0; rd.it.nkb = 0;
        bool ok = true;
        for (;;) {
            const int state = rd.next<true>(item_full, item_free, ring, lane == 0, qtiles, heads, seq_start, seq_len, abort_flag);
            if (state != 1) { ok = state == 0; break; }
            const Item it = rd.it;
            const uint32_t os = (rd.n - 1) & 1, ouse = (rd.n - 1) >> 1;
            const uint32_t o_acc = lane_addr + COL_O + os * D;
            const bool warp_live = it.q0 + quad * 32 < it.len;   // a warp whose 32 rows lie past the sequence only signals
            float m_ref = -INFINITY;   // reference maximum of the row, in exp2 units (score * scale_log2e)
            float l_row = 0.f;
            uint32_t ra[32], rb[32];   // the two halves of a block's scores
            if (!(ok = mbar_wait(s_full + 8 * (rd.g0 % NSB), (rd.g0 / NSB) & 1, abort_flag))) break;
            if (warp_live) {
                tc_fence_after();
                const uint32_t sbuf = lane_addr + (rd.g0 % NSB) * kBlockN;
                tmem_ld_32x32(sbuf, ra);
                if (it.len > 32) tmem_ld_32x32(sbuf + 32, rb);
            }
            for (int j = 0; j < it.nkb && ok; ++j) {
                const uint32_t g = rd.g0 + j, st = g % NST, sb = g % NSB;
                const int keys = min(kBlockN, it.len - j * kBlockN);
                const int kpad = (keys + 15) & ~15;
                const bool more = j + 1 < it.nkb;
                if (keys < kpad) {
                    // keys of the last 16-group past the end of the sequence get probability 0, but the V
                    // rows behind them are whatever follows in memory: clear them so that 0 * junk stays 0
                    // (S_j is complete, so the stage's K and V have landed)
                    unsigned char* vt = gbase + SM::KV_OFF + st * 2 * SM::TILE_BYTES + SM::TILE_BYTES;
                    for (int i = (int)threadIdx.x - 64; i < (kpad - keys) * (SM::ROW_BYTES / 16); i += 128)
                        *reinterpret_cast<uint4*>(vt + (size_t)keys * SM::ROW_BYTES + i * 16) = make_uint4(0, 0, 0, 0);
                    fence_proxy_async();
                }
                // the next block's S: passed here by every warp, so that no parity wait is ever a phase behind
                if (warp == 2 && lane == 0) ATT_TR(2, 1);
                if (more && !(ok = mbar_wait(s_full + 8 * ((g + 1) % NSB), ((g + 1) / NSB) & 1, abort_flag))) break;
                if (warp == 2 && lane == 0) ATT_TR(2, 2);
                if (warp_live) {
                    const uint32_t sbuf = lane_addr + sb * kBlockN;
                    const uint32_t snext = lane_addr + ((g + 1) % NSB) * kBlockN;
                    const int keys_next = min(kBlockN, it.len - (j + 1) * kBlockN);
                    tmem_ld_wait();
                    if (warp == 2 && lane == 0) ATT_TR(2, 3);
                    if (keys < kBlockN) {   // last block: columns past the sequence never count
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            if (i >= keys) ra[i] = 0xFF800000u;        // -inf
                            if (32 + i >= keys) rb[i] = 0xFF800000u;
                        }
                    }
                    float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int i = 0; i < 32; i += 4) {
                        mx[0] = max3f(mx[0], __uint_as_float(ra[i]), __uint_as_float(ra[i + 1]));
                        mx[1] = max3f(mx[1], __uint_as_float(ra[i + 2]), __uint_as_float(ra[i + 3]));
                        mx[2] = max3f(mx[2], __uint_as_float(rb[i]), __uint_as_float(rb[i + 1]));
                        mx[3] = max3f(mx[3], __uint_as_float(rb[i + 2]), __uint_as_float(rb[i + 3]));
                    }
                    const float m_blk = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * scale_log2e;
                    if (j == 0) {
                        m_ref = m_blk;
                    } else {
                        const bool need = m_blk > m_ref + kRescaleAbove;
                        if (__any_sync(0xffffffffu, need)) {
                            // the products issued so far must have landed in O before it is scaled
                            if (!(ok = mbar_wait(pv_done + 8 * ((g - 1) % kPvRing), ((g - 1) / kPvRing) & 1, abort_flag))) break;
                            tc_fence_after();
                            const float alpha = need ? ex2f(m_ref - m_blk) : 1.f;
                            if (need) m_ref = m_blk;
                            l_row *= alpha;
#pragma unroll
                            for (int c0 = 0; c0 < D; c0 += 16) {
                                uint32_t o[16];
                                tmem_ld_32x16(o_acc + c0, o);
                                tmem_ld_wait();
#pragma unroll
                                for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                                tmem_st_32x16(o_acc + c0, o);
                            }
                        }
                    }
                    // Exponentials in an explicit software pipeline: every step pairs one MUFU instruction
                    // with independent FMA-pipe work of the other half, in place in the score registers, so
                    // that a warp keeps the MUFU fed by itself (the ex2 statements are volatile: their order
                    // among the other instructions is the order written here).
                    const float neg_m = -m_ref;
                    float acc[4] = {0.f, 0.f, 0.f, 0.f};
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 32; ++i) ra[i] = __float_as_uint(fmaf(__uint_as_float(ra[i]), scale_log2e, neg_m));
                    if (kpad > 32) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            ra[i] = __float_as_uint(ex2f_pinned(__uint_as_float(ra[i])));
                            rb[i] = __float_as_uint(fmaf(__uint_as_float(rb[i]), scale_log2e, neg_m));
                        }
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            rb[i] = __float_as_uint(ex2f_pinned(__uint_as_float(rb[i])));
                            acc[i & 3] += __uint_as_float(ra[i]);
                            if (i & 1) pk[i >> 1] = pack_bf16(__uint_as_float(ra[i - 1]), __uint_as_float(ra[i]));
                        }
                        tmem_st_32x16(sbuf, pk);
                        if (more) tmem_ld_32x32(snext, ra);        // next block, first half
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            acc[i & 3] += __uint_as_float(rb[i]);
                            if (i & 1) pk[i >> 1] = pack_bf16(__uint_as_float(rb[i - 1]), __uint_as_float(rb[i]));
                        }
                        tmem_st_32x16(sbuf + 16, pk);
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) ra[i] = __float_as_uint(ex2f_pinned(__uint_as_float(ra[i])));
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            acc[i & 3] += __uint_as_float(ra[i]);
                            if (i & 1) pk[i >> 1] = pack_bf16(__uint_as_float(ra[i - 1]), __uint_as_float(ra[i]));
                        }
                        tmem_st_32x16(sbuf, pk);
                        if (more) tmem_ld_32x32(snext, ra);
                    }
                    if (more && keys_next > 32) tmem_ld_32x32(snext + 32, rb);
                    l_row += (acc[0] + acc[1]) + (acc[2] + acc[3]);
                    if (warp == 2 && lane == 0) ATT_TR(2, 5);
                    tmem_st_wait();
                    tc_fence_before();
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full + 8 * sb);
                if (warp == 2 && lane == 0) ATT_TR(2, 6);
            }
            if (!ok) break;
            // ---- O / sum -> bf16 -> global ----
            const uint32_t gl = rd.g0 + it.nkb - 1;   // completions are in order: the last one covers all
            if (!(ok = mbar_wait(pv_done + 8 * (gl % kPvRing), (gl / kPvRing) & 1, abort_flag))) break;
            tc_fence_after();
            const float inv = l_row > 0.f ? 1.0f / l_row : 0.f;
            const int qrow = it.q0 + row;
            __nv_bfloat16* orow = ctx + (size_t)(it.row0 + qrow) * H + it.head * D;
            (void)ouse;
#pragma unroll
            for (int c0 = 0; c0 < D; c0 += 32) {
                uint32_t a[32];
                if (warp_live) {
                    tmem_ld_32x32(o_acc + c0, a);
                    tmem_ld_wait();
                }
                if (c0 + 32 >= D) {   // last read of this O accumulator: hand it back
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(o_free + 8 * os);
                }
                if (warp_live && qrow < it.len) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        uint4 q;
                        q.x = pack_bf16(__uint_as_float(a[8 * i + 0]) * inv, __uint_as_float(a[8 * i + 1]) * inv);
                        q.y = pack_bf16(__uint_as_float(a[8 * i + 2]) * inv, __uint_as_float(a[8 * i + 3]) * inv);
                        q.z = pack_bf16(__uint_as_float(a[8 * i + 4]) * inv, __uint_as_float(a[8 * i + 5]) * inv);
                        q.w = pack_bf16(__uint_as_float(a[8 * i + 6]) * inv, __uint_as_float(a[8 * i + 7]) * inv);
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
