// The part of an encoder layer behind the attention in one kernel (Section 3.2, operator fusion), in three forms
// (template switches LN, PRE):
//   plain        out = gelu(X W1^T + b1) W2^T + b2 + X                        X [M, H] is input AND residual
//   LN           out = LayerNorm(gelu(X W1^T + b1) W2^T + b2 + X)
//   LN + PRE     X   = LayerNorm(ctx Wo^T + bo + h) first (ctx: the attention's context rows, h: the layer's input
//                rows), then the LN form: the whole layer tail; X never reaches global memory
// W1 [F, H], W2 [H, F], Wo [H, H]; erf GELU.  The F-wide hidden activation never reaches global memory either: it
// is produced and consumed in chunks of 64 columns.
//
// A CTA pair (tcgen05 cta_group::2, M = 256) owns a block of 256 rows at a time:
//   front (PRE)  the ctx rows land in the X tiles (H/64 swizzled k-block tiles per CTA, one barrier per tile);
//                O = ctx Wo^T with Wo's k-block tiles through the W2 ring; the residual rows h are loaded over
//                each ctx tile as soon as the products on it have completed; row epilogue: X = bf16(LayerNorm(O +
//                bo + h)) written over h in the same swizzled slots -- the A operand of what follows
//   X block      resident in shared memory for the whole block; the A operand of every first product and, at the
//                end, the residual (read from shared memory)
//   chunk c      S_c = X W1[64c .. 64c+63, :]^T            M = 256, N = 64, K = H       -> TMEM (two S buffers)
//                G_c = bf16(gelu(S_c + b1))                 epilogue warps: TMEM -> registers -> shared memory,
//                                                           written in the K-major 128-byte-swizzled layout the
//                                                           tensor core reads (two G buffers of one k-block)
//                O  += G_c W2[:, 64c .. 64c+63]^T           M = 256, N = H (two instructions of H/2), K = 64
//   end          out = [LayerNorm](O + b2 + X) -> bf16, written back over the X tile slots the residual was read
//                from, and stored from there with one TMA store per warp and 64-column tile (the shared memory is
//                full; the X tiles are the only staging room and already have the store's layout)
// Roles (per CTA, 13 warps): warp 0 loads X and the W1 chunks, another warp the W2 chunks, Wo's tiles and the
// residual tiles (so a late W2 slot never holds back W1); in the leader CTA two warps issue the first products
// (even / odd chunks) and a third the second products and the projection in front -- a thread pays ~100 cycles
// per tcgen05.mma, and one thread for a chunk's 32 instructions paced the kernel; eight epilogue warps turn S_c
// into G_c in a software pipeline that overlaps the barrier probes and the tensor-memory load of S_{c+1} with
// the GELU arithmetic of S_c, and run the row epilogues (two passes over tensor memory for a LayerNorm: pivoted
// row sums, then normalise).  W1 / W2 chunks stream through two-stage rings, each CTA loading its half of the
// rows.  TMEM: O (H columns) + 2 x 64 columns of S = 512 at H = 384.
// Rounding points of the products are those of the separate GEMMs (G and X rounded to bf16 once, fp32
// accumulation in the same k order): without LayerNorm the result is bit for bit the two-GEMM form's.  The
// LayerNorms work on the unrounded fp32 sums.
// All mbarrier waits are bounded; on expiry the CTA sets the status bit and leaves.
#pragma once
#include <cuda.h>
#include "common.cuh"
#include "epilogue.cuh"
#include "gemm_tcgen05.cuh"

namespace rlx {
namespace tcff {

using namespace rlx::tc;

constexpr int kPairRows = 256;
constexpr int kChunk = 64;          // hidden columns per chunk = one k-block of the second product
constexpr int kEpiWarps = 8;        // per CTA: lane quarter x column half of a 64-column S chunk
constexpr int kThreads = 64 + 32 * kEpiWarps + 96;   // TMA, first products (even chunks), epilogue warps, second products, first products (odd chunks), W2 loads

template <int HID>
struct Cfg {
    static_assert(HID % 128 == 0 && HID <= 384, "hidden size");
    static constexpr int KB1 = HID / BLOCK_K;                       // k-blocks of the first product
    static constexpr int X_BYTES = KB1 * BLOCK_M * 128;             // this CTA's 128 rows of X
    static constexpr int W1_ROWS = kChunk / 2;                      // this CTA's half of a chunk's W1 rows
    static constexpr int W1_STAGE = KB1 * W1_ROWS * 128;
    static constexpr int W2_ROWS = HID / 4;                         // per instruction (N = HID/2), this CTA's half
    static constexpr int W2_STAGE = 2 * W2_ROWS * 128;              // two instructions' halves, one k-block
    static constexpr int G_BYTES = BLOCK_M * 128;                   // one k-block tile of G
    static constexpr int X_OFF = 0, W1_OFF = X_BYTES, W2_OFF = W1_OFF + 2 * W1_STAGE, G_OFF = W2_OFF + 2 * W2_STAGE;
    static constexpr int BAR_OFF = G_OFF + 2 * G_BYTES;
    static constexpr int B1_OFF = BAR_OFF + 512;                    // per epilogue warp: the 32 bias values of its chunk half
    static constexpr int SMEM_BYTES = B1_OFF + kEpiWarps * 128 + 1024;
    static constexpr int COL_S = HID;                               // S buffers behind O
    static constexpr int TMEM_COLS = 512;
    static_assert(HID + 2 * kChunk <= 512, "tensor memory");
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory");
};

struct FfnParams {
    const float* b1;            // [F]
    const float* b2;            // [H]
    __nv_bfloat16* out;         // [M, H]
    int M, F;
    const int32_t* m_ptr;       // optional device row count
    const float* bo;            // [H]  PRE variant: bias of the projection in front, and the LayerNorm behind it
    const float* ln1_gamma;     // [H]
    const float* ln1_beta;      // [H]
    const float* ln_gamma;      // [H]  LayerNorm over the rows of the result (kernel variant LN only)
    const float* ln_beta;       // [H]
    float ln_eps;
    int32_t* status;
};

// byte offset of 16-byte chunk j of row r in a K-major tile of 128-byte rows with the 128-byte swizzle
__device__ __forceinline__ uint32_t sw128(int r, int j) { return (uint32_t)(r * 128 + ((j ^ (r & 7)) << 4)); }

// v[j] = accumulator + bias + residual for eight consecutive columns (x: the eight bf16 residual values)
__device__ __forceinline__ void residual_row8(const uint32_t* acc, const uint4& x, const float4& ba, const float4& bb, float* v) {
    v[0] = __uint_as_float(acc[0]) + ba.x + bf16lo(x.x); v[1] = __uint_as_float(acc[1]) + ba.y + bf16hi(x.x);
    v[2] = __uint_as_float(acc[2]) + ba.z + bf16lo(x.y); v[3] = __uint_as_float(acc[3]) + ba.w + bf16hi(x.y);
    v[4] = __uint_as_float(acc[4]) + bb.x + bf16lo(x.z); v[5] = __uint_as_float(acc[5]) + bb.y + bf16hi(x.z);
    v[6] = __uint_as_float(acc[6]) + bb.z + bf16lo(x.w); v[7] = __uint_as_float(acc[7]) + bb.w + bf16hi(x.w);
}
// the same as four packed pairs (Blackwell's f32x2 arithmetic: one issue slot per pair)
__device__ __forceinline__ void residual_row8_x2(const uint32_t* acc, const uint4& x, const float4& ba, const float4& bb, uint64_t* v) {
    v[0] = add_f32x2(add_f32x2(pack_f32x2(__uint_as_float(acc[0]), __uint_as_float(acc[1])), pack_f32x2(ba.x, ba.y)), pack_f32x2(bf16lo(x.x), bf16hi(x.x)));
    v[1] = add_f32x2(add_f32x2(pack_f32x2(__uint_as_float(acc[2]), __uint_as_float(acc[3])), pack_f32x2(ba.z, ba.w)), pack_f32x2(bf16lo(x.y), bf16hi(x.y)));
    v[2] = add_f32x2(add_f32x2(pack_f32x2(__uint_as_float(acc[4]), __uint_as_float(acc[5])), pack_f32x2(bb.x, bb.y)), pack_f32x2(bf16lo(x.z), bf16hi(x.z)));
    v[3] = add_f32x2(add_f32x2(pack_f32x2(__uint_as_float(acc[6]), __uint_as_float(acc[7])), pack_f32x2(bb.z, bb.w)), pack_f32x2(bf16lo(x.w), bf16hi(x.w)));
}
__device__ __forceinline__ uint32_t pack_bf16_pair(uint64_t v) {
    float lo, hi;
    unpack_f32x2(v, lo, hi);
    return pack_bf16(lo, hi);
}
__device__ __forceinline__ void st_shared_f32(uint32_t addr, float a) {
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(a) : "memory");
}
__device__ __forceinline__ float4 ld_shared_f32x4(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void st_shared_f32x4(uint32_t addr, const float4& v) {
    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
__device__ __forceinline__ void st_shared_f32x2(uint32_t addr, float a, float b) {
    asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(addr), "f"(a), "f"(b) : "memory");
}
__device__ __forceinline__ void ld_shared_f32x2(uint32_t addr, float& a, float& b) {
    asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(a), "=f"(b) : "r"(addr) : "memory");
}

// What a warp of the row epilogue knows about its place: tensor-memory lanes, shared-memory regions, barriers.
struct RowCtx {
    uint32_t lane_addr;      // tensor-memory address of the warp's lane quarter, column 0 (the accumulator O)
    uint32_t xs, gs;         // X tiles (residual in, result out), G buffers (scratch)
    uint32_t ln_bar;         // [4] per lane quarter
    uint32_t lead_o_empty;   // leader CTA's barrier: O has been read
    volatile int* abort_flag;
    int r, wslot, quad, grp, lane;   // row in the CTA; index of the warp's parameter copy; lane quarter; column group
};

// Row epilogue of a 128 x HID accumulator block:  v = O + bias + residual (the bf16 values in the X tiles),
// optionally through LayerNorm, rounded to bf16 and written back over the residual's slots; with STORE each
// warp then stores its 32-row slice of every 64-column tile with one TMA store (row0 = the slice's first global
// row).  Returns false when a bounded wait ran out.
template <int HID, bool DO_LN, bool STORE, int GROUPS>
__device__ __noinline__ bool row_epilogue(const RowCtx rc, const float* bias, const float* gamma, const float* beta, float eps,
                                             uint32_t ln_parity, const CUtensorMap* tmap_out, int row0) {
    const uint32_t lane_addr = rc.lane_addr, xs = rc.xs, gs = rc.gs, ln_bar = rc.ln_bar, lead_o_empty = rc.lead_o_empty;
    volatile int* abort_flag = rc.abort_flag;
    const int r = rc.r, wslot = rc.wslot, quad = rc.quad, grp = rc.grp, lane = rc.lane;
    // The columns are split over GROUPS warps per lane quarter (two with the eight epilogue warps alone, three when
    // the producer and MMA-issuing warps, idle while rows are finished, form a third group).
    static_assert(HID % (64 * GROUPS) == 0, "whole 64-column tiles per group");
    constexpr int kTilesPerWarp = HID / 64 / GROUPS;
    // LN variant: the row then goes through LayerNorm before it is rounded.  A row's H values sit with two
    // threads (same lane quarter and lane, the two column halves): a first pass over O and X sums v and
    // v^2 per thread, the pair swaps its sums through shared memory (the first G buffer, idle until the
    // next block's first chunk, which cannot start before every warp here has released X), and the
    // second pass recomputes v and normalises it.  Tensor memory is read twice; nothing else moves.
    // Both passes walk the warp's column half in chunks of 32 columns with the tensor-memory load of the
    // next chunk in flight while the current one is worked on (two register buffers).
    constexpr int kColChunks = 2 * kTilesPerWarp;
    static_assert(kColChunks % 2 == 0, "chunk pairs");
    // b2 (and gamma, beta) of the warp's column half go to a private copy in the idle G buffers first
    // (behind the 2 KB the row sums are swapped through): every thread needs every value, and broadcast
    // reads from shared memory are several times cheaper than same-address global loads.
    constexpr int kParamVecs = DO_LN ? 3 : 1, kHalfCols = HID / GROUPS;
    constexpr int kScratch = GROUPS * BLOCK_M * 8;   // (mean, M2) per row and group
    const uint32_t par = gs + kScratch + wslot * (3 * kHalfCols * 4);
    static_assert(kScratch + 4 * GROUPS * 3 * kHalfCols * 4 <= 2 * Cfg<HID>::G_BYTES, "parameter copies fit in the G buffers");
    for (int idx = lane; idx < kParamVecs * (kHalfCols / 4); idx += 32) {
        const int a = idx / (kHalfCols / 4), w4 = idx - a * (kHalfCols / 4);
        const float* src = (a == 0 ? bias : a == 1 ? gamma : beta) + grp * kHalfCols;
        st_shared_f32x4(par + (a * kHalfCols + w4 * 4) * 4, __ldg(reinterpret_cast<const float4*>(src) + w4));
    }
    __syncwarp();
    const auto param4 = [&](int a, int col0, int i4) {   // 4 values of vector a at columns col0 + 4*i4 ..
        return ld_shared_f32x4(par + (a * kHalfCols + (col0 - grp * kHalfCols) + 4 * i4) * 4);
    };
    const auto chunk_col = [&](int cidx) { return (grp * kTilesPerWarp + (cidx >> 1)) * 64 + (cidx & 1) * 32; };
    float ln_a = 1.f, ln_c = 0.f;    // y = (v * ln_a + ln_c) * gamma + beta
    if constexpr (DO_LN) {
        // sums of (v - pivot) and (v - pivot)^2 with the thread's first value as the pivot: no cancellation
        // when a row's mean is large against its spread
        uint64_t sum2 = pack_f32x2(0.f, 0.f), sq2 = sum2, npivot2 = sum2;
        float pivot = 0.f;
        bool have_pivot = false;
        const auto stats_chunk = [&](const uint32_t* acc, int cidx) {
            const int col0 = chunk_col(cidx);
            const uint32_t tile = xs + (col0 >> 6) * BLOCK_M * 128;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint4 x = ld_shared_v4(tile + sw128(r, (cidx & 1) * 4 + i));
                const float4 ba = param4(0, col0, 2 * i), bb = param4(0, col0, 2 * i + 1);
                uint64_t v[4];
                residual_row8_x2(acc + 8 * i, x, ba, bb, v);
                if (!have_pivot) {
                    float hi;
                    unpack_f32x2(v[0], pivot, hi);
                    npivot2 = pack_f32x2(-pivot, -pivot);
                    have_pivot = true;
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint64_t dv = add_f32x2(v[j], npivot2);
                    sum2 = add_f32x2(sum2, dv);
                    sq2 = fma_f32x2(dv, dv, sq2);
                }
            }
        };
        {
            uint32_t acc_a[32], acc_b[32];
            tmem_ld_32x32(lane_addr + chunk_col(0), acc_a);
#pragma unroll 1
            for (int cidx = 0; cidx < kColChunks; cidx += 2) {
                tmem_ld_wait();
                tmem_ld_32x32(lane_addr + chunk_col(cidx + 1), acc_b);
                stats_chunk(acc_a, cidx);
                tmem_ld_wait();
                if (cidx + 2 < kColChunks) tmem_ld_32x32(lane_addr + chunk_col(cidx + 2), acc_a);
                stats_chunk(acc_b, cidx + 1);
            }
        }
        float sum, sq;
        {
            float a0, a1, q0, q1;
            unpack_f32x2(sum2, a0, a1);
            unpack_f32x2(sq2, q0, q1);
            sum = a0 + a1; sq = q0 + q1;
        }
        // this thread's part of the row: mean and sum of squared deviations; the parts are combined in group order
        // by every thread of the row, so that all of them normalise with the same two numbers
        constexpr float kPart = (float)kHalfCols;
        const float my_mean = pivot + sum * (1.f / kPart);
        const float my_m2 = fmaxf(sq - sum * sum * (1.f / kPart), 0.f);
        st_shared_f32x2(gs + (uint32_t)((grp * BLOCK_M + r) * 8), my_mean, my_m2);
        __syncwarp();
        if (lane == 0) mbar_arrive(ln_bar + 8 * quad);
        if (!mbar_wait(ln_bar + 8 * quad, ln_parity, abort_flag)) return false;
        float mean, m2;
        ld_shared_f32x2(gs + (uint32_t)(r * 8), mean, m2);
#pragma unroll
        for (int g = 1; g < GROUPS; ++g) {
            float o_mean, o_m2;
            ld_shared_f32x2(gs + (uint32_t)((g * BLOCK_M + r) * 8), o_mean, o_m2);
            const float dm = o_mean - mean;
            mean += dm * (1.f / (g + 1));                              // g parts of kPart columns so far, one more
            m2 += o_m2 + dm * dm * (kPart * (float)g / (float)(g + 1));
        }
        const float var = m2 * (1.f / HID);
        ln_a = rsqrtf(var + eps);
        ln_c = -mean * ln_a;
    }
    const uint64_t ln_a2 = pack_f32x2(ln_a, ln_a), ln_c2 = pack_f32x2(ln_c, ln_c);
    const auto out_chunk = [&](const uint32_t* acc, int cidx) {
        const int col0 = chunk_col(cidx);
        const uint32_t tile = xs + (col0 >> 6) * BLOCK_M * 128;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t slot = tile + sw128(r, (cidx & 1) * 4 + i);
            const uint4 x = ld_shared_v4(slot);
            const float4 ba = param4(0, col0, 2 * i), bb = param4(0, col0, 2 * i + 1);
            uint64_t v[4];
            residual_row8_x2(acc + 8 * i, x, ba, bb, v);
            if constexpr (DO_LN) {
                const float4 ga = param4(1, col0, 2 * i), gb = param4(1, col0, 2 * i + 1);
                const float4 ea = param4(2, col0, 2 * i), eb = param4(2, col0, 2 * i + 1);
                v[0] = fma_f32x2(fma_f32x2(v[0], ln_a2, ln_c2), pack_f32x2(ga.x, ga.y), pack_f32x2(ea.x, ea.y));
                v[1] = fma_f32x2(fma_f32x2(v[1], ln_a2, ln_c2), pack_f32x2(ga.z, ga.w), pack_f32x2(ea.z, ea.w));
                v[2] = fma_f32x2(fma_f32x2(v[2], ln_a2, ln_c2), pack_f32x2(gb.x, gb.y), pack_f32x2(eb.x, eb.y));
                v[3] = fma_f32x2(fma_f32x2(v[3], ln_a2, ln_c2), pack_f32x2(gb.z, gb.w), pack_f32x2(eb.z, eb.w));
            }
            uint4 q;
            q.x = pack_bf16_pair(v[0]); q.y = pack_bf16_pair(v[1]); q.z = pack_bf16_pair(v[2]); q.w = pack_bf16_pair(v[3]);
            st_shared_v4(slot, q);
        }
        if (STORE && (cidx & 1)) {   // the warp's slice of this 64-column tile is complete
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
                tma_store_2d(tmap_out, (col0 >> 6) * 64, row0, tile + quad * 32 * 128);   // rows past the matrix are clipped
                bulk_commit();
            }
        }
    };
    {
        uint32_t acc_a[32], acc_b[32];
        tmem_ld_32x32(lane_addr + chunk_col(0), acc_a);
#pragma unroll 1
        for (int cidx = 0; cidx < kColChunks; cidx += 2) {
            tmem_ld_wait();
            tmem_ld_32x32(lane_addr + chunk_col(cidx + 1), acc_b);
            out_chunk(acc_a, cidx);
            tmem_ld_wait();
            if (cidx + 2 < kColChunks) {
                tmem_ld_32x32(lane_addr + chunk_col(cidx + 2), acc_a);
            } else {   // last read of O by this warp
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster_relaxed(lead_o_empty);
            }
            out_chunk(acc_b, cidx + 1);
        }
    }
    return true;
}

template <int HID, bool LN, bool PRE>
__global__ void __launch_bounds__(kThreads, 1)
ffn_fused_tcgen05_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w1,
                         const __grid_constant__ CUtensorMap tmap_w2, const __grid_constant__ CUtensorMap tmap_out,
                         const __grid_constant__ CUtensorMap tmap_wo, const __grid_constant__ CUtensorMap tmap_h, const FfnParams p) {
    using C = Cfg<HID>;
    // Warps that finish rows: the eight epilogue warps as two column groups.  A third group made of the warps that
    // have nothing to issue while rows are finished (X / W1 producer and the three MMA-issuing warps: lane quarters
    // 0, 1, 2, 3; kGroups = 3 at H = 384, every hook below is in place) was measured SLOWER (101 against 96 us per
    // layer at 37 k rows): the passes are paced by the shared-memory pipe, not by the number of warps.
    constexpr int kGroups = 2;
    constexpr int kRowWarps = 4 * kGroups;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* gbase = smem_raw + (base - raw);
    const uint32_t xs = base + C::X_OFF, w1s = base + C::W1_OFF, w2s = base + C::W2_OFF, gs = base + C::G_OFF;
    const uint32_t bars = base + C::BAR_OFF;
    // leader-side barriers that both CTAs' TMA / warps arrive on: x_full[6] (one per k-block tile), w1_full[2], w2_full[2], s_empty[2],
    // g_full[2], o_empty.  Per-CTA barriers (multicast commits / own warps): x_empty, w1_empty[2], w2_empty[2],
    // s_full[2], g_empty[2], o_full.
    const uint32_t x_full = bars, w1_full = x_full + 48, w2_full = w1_full + 16, s_empty = w2_full + 16, g_full = s_empty + 16;
    const uint32_t o_empty = g_full + 16, x_empty = o_empty + 8, w1_empty = x_empty + 8, w2_empty = w1_empty + 16;
    const uint32_t s_full = w2_empty + 16, g_empty = s_full + 16, o_full = g_empty + 16;
    const uint32_t ln_bar = o_full + 8;   // [4] per lane quarter: the two column halves' row sums are in shared memory
    // PRE variant: a_done (per CTA: the projection's products are complete), h_full (per CTA: the residual rows have
    // landed in the X tiles), x_ready (leader: all 16 epilogue warps have written their rows of X)
    const uint32_t a_done = ln_bar + 32, h_full = a_done + 8, x_ready = h_full + 8;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gbase + C::BAR_OFF + 8 * 32);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta_rank = cluster_ctarank();
    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        for (int i = 0; i < C::KB1; ++i) mbar_init(x_full + 8 * i, 1);
        mbar_init(o_empty, 2 * kRowWarps);
        mbar_init(x_empty, 2 + kRowWarps);      // both first-product warps' last commits + this CTA's row-epilogue warps
        mbar_init(o_full, 1);
        for (int i = 0; i < 4; ++i) mbar_init(ln_bar + 8 * i, kGroups);
        mbar_init(a_done, 1); mbar_init(h_full, 1); mbar_init(x_ready, 2 * kRowWarps);
        for (int i = 0; i < 2; ++i) {
            mbar_init(w1_full + 8 * i, 1); mbar_init(w2_full + 8 * i, 1);
            mbar_init(w1_empty + 8 * i, 1); mbar_init(w2_empty + 8 * i, 1);
            mbar_init(s_full + 8 * i, 1); mbar_init(s_empty + 8 * i, 2 * kEpiWarps);
            mbar_init(g_full + 8 * i, 2 * kEpiWarps); mbar_init(g_empty + 8 * i, 1);
        }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmap_x); prefetch_tmap(&tmap_w1); prefetch_tmap(&tmap_w2); prefetch_tmap(&tmap_out);
        if (PRE) { prefetch_tmap(&tmap_wo); prefetch_tmap(&tmap_h); }
    }
    if (warp == 1) {
        tmem_alloc<2>(smem_u32(tmem_slot), C::TMEM_COLS);
        tmem_relinquish<2>();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    pdl_wait();
    int M = p.M;
    if (p.m_ptr != nullptr) M = min(M, __ldg(p.m_ptr));
    const int blocks = (M + kPairRows - 1) / kPairRows;
    const int pairs = gridDim.x / 2, pair0 = blockIdx.x / 2;
    const int n_chunks = p.F / kChunk;

    // ---- row epilogues (the LayerNorm in front with PRE, the block's end), shared by every warp that finishes rows
    const bool epi_warp = warp >= 2 && warp < 2 + kEpiWarps;
    const bool helper_warp = kGroups == 3 && (warp <= 1 || warp == 2 + kEpiWarps || warp == 3 + kEpiWarps);   // lane quarters 0, 1, 2, 3
    RowCtx rc;
    rc.quad = warp & 3;
    rc.lane_addr = tmem + ((uint32_t)(rc.quad * 32) << 16);
    rc.xs = xs; rc.gs = gs; rc.ln_bar = ln_bar; rc.abort_flag = abort_flag; rc.lane = lane;
    rc.r = rc.quad * 32 + lane;
    rc.grp = epi_warp ? (warp - 2) >> 2 : 2;
    rc.wslot = epi_warp ? warp - 2 : kEpiWarps + rc.quad;
    rc.lead_o_empty = map_to_cta(o_empty, 0);
    const uint32_t lead_x_ready = map_to_cta(x_ready, 0);
    // x1 = LayerNorm(ctx Wo^T + bo + h) for the block's rows, written over the residual rows h in the X tiles: the
    // A operand of the first products and the residual of the block's end, never in global memory
    const auto front_rows = [&](uint32_t nb) -> bool {
        if (!mbar_wait(a_done, nb & 1, abort_flag)) return false;
        tc_fence_after();
        if (!mbar_wait(h_full, nb & 1, abort_flag)) return false;
        if (!row_epilogue<HID, true, false, kGroups>(rc, p.bo, p.ln1_gamma, p.ln1_beta, p.ln_eps, 0u, nullptr, 0)) return false;
        fence_proxy_async();     // generic-proxy writes -> visible to the tensor core's reads
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster_release_cta(lead_x_ready);
        return true;
    };
    // out = [LayerNorm](O + b2 + X).  The resident X tiles serve twice more: each thread reads its residual values
    // from them and writes the finished bf16 outputs back to the same 16-byte slots (same rows, same swizzle), and
    // the warp then stores its 32-row slice of a 64-column tile with one TMA store -- the tile's layout in shared
    // memory is the one the TMA load produced, so the store map has the load map's geometry.
    const auto final_rows = [&](uint32_t nb, int blk) -> bool {
        if (!mbar_wait(o_full, nb & 1, abort_flag)) return false;
        tc_fence_after();
        if (!row_epilogue<HID, LN, true, kGroups>(rc, p.b2, p.ln_gamma, p.ln_beta, p.ln_eps, PRE ? 1u : (nb & 1), &tmap_out,
                                                  blk * kPairRows + (int)cta_rank * BLOCK_M + rc.quad * 32)) return false;
        if (lane == 0) {
            bulk_wait_read<0>();      // the stores have read their slices: X may be overwritten
            mbar_arrive(x_empty);
        }
        __syncwarp();
        return true;
    };

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer of X and the W1 chunks (both CTAs)
        // The whole warp runs the loop (lane 0 issues): at H = 384 it also finishes rows as lane quarter 0 of the
        // third column group -- after the first two W1 chunks are on their way (PRE) and after the block's last one.
        {
            bool ok = true;
            uint32_t nb = 0, cc = 0;   // blocks and chunks done so far
            for (int blk = pair0; blk < blocks && ok; blk += pairs, ++nb) {
                if (nb >= 1 && !(ok = mbar_wait_warp(x_empty, (nb - 1) & 1, abort_flag))) break;
                if (lane == 0) {
                    // one barrier per k-block tile: the projection in front starts on tile 0 while the others land
                    const uint32_t lead_x = map_to_cta(x_full, 0);
                    if (cta_rank == 0)
                        for (int kb = 0; kb < C::KB1; ++kb) mbar_expect_tx(x_full + 8 * kb, 2 * BLOCK_M * 128);
                    const int xrow = blk * kPairRows + (int)cta_rank * BLOCK_M;
                    for (int kb = 0; kb < C::KB1; ++kb) tma_load_2d_cg2(xs + kb * BLOCK_M * 128, &tmap_x, kb * BLOCK_K, xrow, lead_x + 8 * kb);
                }
                for (int c = 0; c < n_chunks && ok; ++c, ++cc) {
                    if (PRE && helper_warp && c == 2 && !(ok = front_rows(nb))) break;
                    const uint32_t st = cc & 1, use = cc >> 1;
                    if (use >= 1 && !(ok = mbar_wait_warp(w1_empty + 8 * st, (use - 1) & 1, abort_flag))) break;
                    if (lane == 0) {
                        const uint32_t lead1 = map_to_cta(w1_full + 8 * st, 0);
                        if (cta_rank == 0) mbar_expect_tx(w1_full + 8 * st, 2 * C::W1_STAGE);
                        for (int kb = 0; kb < C::KB1; ++kb)
                            tma_load_2d_cg2(w1s + st * C::W1_STAGE + kb * C::W1_ROWS * 128, &tmap_w1, kb * BLOCK_K,
                                            c * kChunk + (int)cta_rank * C::W1_ROWS, lead1);
                    }
                    __syncwarp();
                }
                if (!ok) break;
                if (PRE && helper_warp && n_chunks <= 2 && !(ok = front_rows(nb))) break;
                if (helper_warp && !(ok = final_rows(nb, blk))) break;
            }
        }
    } else if (warp == 4 + kEpiWarps) {
        // ------------------------------------------------------------ TMA producer of the W2 chunks (both CTAs)
        // A thread of its own: behind the W1 loads in one thread, a W2 slot that frees late (its second
        // product waits for the epilogue warps) would hold back the next chunk's W1 tiles as well.
        // PRE variant: the same ring first carries the k-block tiles of Wo (same shape: H output rows, 64 columns
        // of K), and this thread also reloads the X tiles with the residual rows, tile by tile: the ring slot of Wo's
        // k-block kb is free when the products on ctx tile kb have completed, which is when that tile is dead, so
        // the residual tile follows the wait this thread does anyway before it reuses the slot.
        if (lane == 0) {
            bool ok = true;
            uint32_t u2 = 0, nb = 0;     // uses of the ring so far
            uint32_t blk_u0 = 0;         // ... at the start of the current block
            int blk_row = 0;             // this CTA's first row of the current block
            const auto load_tile = [&](const CUtensorMap* tmap, int kcol) -> bool {
                const uint32_t st = u2 & 1, use = u2 >> 1;
                if (use >= 1 && !mbar_wait(w2_empty + 8 * st, (use - 1) & 1, abort_flag)) return false;
                if (PRE && u2 >= blk_u0 + 2 && u2 - 2 - blk_u0 < (uint32_t)C::KB1) {   // the slot held Wo's k-block kb of this block
                    const int kb = (int)(u2 - 2 - blk_u0);
                    if (kb == 0) mbar_expect_tx(h_full, C::X_BYTES);
                    tma_load_2d(xs + kb * BLOCK_M * 128, &tmap_h, kb * BLOCK_K, blk_row, h_full);
                }
                ++u2;
                const uint32_t lead2 = map_to_cta(w2_full + 8 * st, 0);
                if (cta_rank == 0) mbar_expect_tx(w2_full + 8 * st, 2 * C::W2_STAGE);
                for (int i = 0; i < 2; ++i)   // instruction i covers output columns i*HID/2 .., this CTA feeds its half of them
                    tma_load_2d_cg2(w2s + st * C::W2_STAGE + i * C::W2_ROWS * 128, tmap, kcol,
                                    i * (HID / 2) + (int)cta_rank * C::W2_ROWS, lead2);
                return true;
            };
            for (int blk = pair0; blk < blocks && ok; blk += pairs, ++nb) {
                blk_u0 = u2;
                blk_row = blk * kPairRows + (int)cta_rank * BLOCK_M;
                if (PRE) {
                    for (int kb = 0; kb < C::KB1 && ok; ++kb) ok = load_tile(&tmap_wo, kb * BLOCK_K);
                    if (!ok) break;
                }
                for (int c = 0; c < n_chunks && ok; ++c) ok = load_tile(&tmap_w2, c * kChunk);
            }
        }
    } else if (warp == 1 || warp == 3 + kEpiWarps) {
        // ------------------------------------------------------------ first products S_c = X W1_c^T (leader CTA)
        // Three issuing warps in all: a thread pays ~80-110 cycles per tcgen05.mma and ~230 per barrier round,
        // and a chunk is 24 + 8 instructions, so one thread for everything was the kernel's limiter.  The
        // first products alternate between two warps by chunk parity (warp 1: even chunks into S buffer 0,
        // a second warp: odd chunks into S buffer 1; F is a multiple of 128, so the parity of a chunk is
        // the parity of its ring slot in every block); a third warp issues the second products.  Whole-warp
        // loops, one elected lane issues.
        // In both CTAs these warps are lane quarters 1 and 3 of the third column group of the row epilogues (H = 384).
        {
            constexpr uint32_t id1 = make_idesc(kPairRows, kChunk);
            const uint32_t st = warp == 1 ? 0u : 1u;
            bool ok = true;
            uint32_t nb = 0;
            for (int blk = pair0; blk < blocks && ok; blk += pairs, ++nb) {
                if (PRE && helper_warp && !(ok = front_rows(nb))) break;
                if (cta_rank == 0) {
                    if (PRE) {
                        ok = mbar_wait_warp(x_ready, nb & 1, abort_flag);
                    } else {
                        for (int kb = 0; kb < C::KB1 && ok; ++kb) ok = mbar_wait_warp(x_full + 8 * kb, nb & 1, abort_flag);
                    }
                    if (!ok) break;
                }
                for (int c = st; cta_rank == 0 && c < n_chunks && ok; c += 2) {
                    const uint32_t use = (nb * n_chunks + c) >> 1;
                    if (!(ok = mbar_wait_warp(w1_full + 8 * st, use & 1, abort_flag))) break;
                    if (use >= 1 && !(ok = mbar_wait_warp(s_empty + 8 * st, (use - 1) & 1, abort_flag))) break;
                    tc_fence_after();
                    if (elect_one()) {
                        for (int kb = 0; kb < C::KB1; ++kb) {
                            const uint64_t adesc = make_smem_desc(xs + kb * BLOCK_M * 128);
                            const uint64_t bdesc = make_smem_desc(w1s + st * C::W1_STAGE + kb * C::W1_ROWS * 128);
#pragma unroll
                            for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
                                umma_bf16<2>(tmem + C::COL_S + st * kChunk, adesc + 2 * k, bdesc + 2 * k, id1, (kb | k) != 0 ? 1u : 0u);
                        }
                        umma_commit<2>(w1_empty + 8 * st);
                        umma_commit<2>(s_full + 8 * st);
                        // this warp's last read of X in the block; the barrier counts both first-product warps
                        if (c + 2 >= n_chunks) umma_commit<2>(x_empty);
                    }
                    __syncwarp();
                }
                if (!ok) break;
                if (helper_warp && !(ok = final_rows(nb, blk))) break;
            }
        }
    } else if (warp == 2 + kEpiWarps) {
        // ------------------------------------------------------------ second products O += G_c W2_c^T (leader CTA)
        // In both CTAs this warp is lane quarter 2 of the third column group of the row epilogues (H = 384).
        {
            constexpr uint32_t id2 = make_idesc(kPairRows, HID / 2);
            bool ok = true;
            uint32_t nb = 0, cc = 0, u2 = 0, oe = 0;   // blocks, chunks, W2-ring uses, completions of o_empty waited for
            for (int blk = pair0; blk < blocks && ok; blk += pairs, ++nb) {
                if (PRE && cta_rank == 0) {
                    // the projection in front:  O = ctx Wo^T, the resident tiles as A, Wo's k-block tiles through the ring
                    if (nb >= 1) {   // the previous block's result rows have been read out of O
                        if (!(ok = mbar_wait_warp(o_empty, oe & 1, abort_flag))) break;
                        ++oe;
                    }
                    for (int kb = 0; kb < C::KB1 && ok; ++kb, ++u2) {
                        const uint32_t st2 = u2 & 1;
                        if (!(ok = mbar_wait_warp(x_full + 8 * kb, nb & 1, abort_flag))) break;   // ctx tile kb has landed
                        if (!(ok = mbar_wait_warp(w2_full + 8 * st2, (u2 >> 1) & 1, abort_flag))) break;
                        tc_fence_after();
                        if (elect_one()) {
                            const uint64_t adesc = make_smem_desc(xs + kb * BLOCK_M * 128);
#pragma unroll
                            for (int i = 0; i < 2; ++i) {
                                const uint64_t bdesc = make_smem_desc(w2s + st2 * C::W2_STAGE + i * C::W2_ROWS * 128);
#pragma unroll
                                for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
                                    umma_bf16<2>(tmem + i * (HID / 2), adesc + 2 * k, bdesc + 2 * k, id2, (kb | k) != 0 ? 1u : 0u);
                            }
                            umma_commit<2>(w2_empty + 8 * st2);
                            if (kb == C::KB1 - 1) umma_commit<2>(a_done);
                        }
                        __syncwarp();
                    }
                    if (!ok) break;
                }
                if (PRE && helper_warp && !(ok = front_rows(nb))) break;
                for (int c = 0; cta_rank == 0 && c < n_chunks && ok; ++c, ++cc, ++u2) {
                    const uint32_t st = cc & 1, use = cc >> 1, st2 = u2 & 1;
                    if (!(ok = mbar_wait_warp(w2_full + 8 * st2, (u2 >> 1) & 1, abort_flag))) break;
                    // first accumulation of the block overwrites O: its last readers (the previous block's epilogue, or
                    // with PRE this block's LayerNorm in front) must be done
                    if (c == 0 && (PRE || nb >= 1)) {
                        if (!(ok = mbar_wait_warp(o_empty, oe & 1, abort_flag))) break;
                        ++oe;
                    }
                    if (!(ok = mbar_wait_warp(g_full + 8 * st, use & 1, abort_flag))) break;
                    tc_fence_after();
                    if (elect_one()) {
                        const uint64_t adesc = make_smem_desc(gs + st * C::G_BYTES);
#pragma unroll
                        for (int i = 0; i < 2; ++i) {
                            const uint64_t bdesc = make_smem_desc(w2s + st2 * C::W2_STAGE + i * C::W2_ROWS * 128);
#pragma unroll
                            for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
                                umma_bf16<2>(tmem + i * (HID / 2), adesc + 2 * k, bdesc + 2 * k, id2, (c | k) != 0 ? 1u : 0u);
                        }
                        umma_commit<2>(w2_empty + 8 * st2);
                        umma_commit<2>(g_empty + 8 * st);
                        if (c == n_chunks - 1) umma_commit<2>(o_full);
                    }
                    __syncwarp();
                }
                if (!ok) break;
                if (helper_warp && !(ok = final_rows(nb, blk))) break;
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue warps (both CTAs)
        const int ew = warp - 2, half = ew >> 2;
        const uint32_t lane_addr = rc.lane_addr;
        const int r = rc.r;                                  // this thread's row within the CTA's 128
        const uint32_t b1_slot = base + C::B1_OFF + ew * 128;
        const uint32_t lead_s_empty = map_to_cta(s_empty, 0), lead_g_full = map_to_cta(g_full, 0);
        bool ok = true;
        uint32_t nb = 0, cc = 0;
        for (int blk = pair0; blk < blocks && ok; blk += pairs, ++nb) {
            if (PRE && !(ok = front_rows(nb))) break;
            // Software pipeline over the chunks: the registers hold S_c when an iteration starts; the probe of
            // S_{c+1}'s barrier, the tensor-memory load of S_{c+1} and the probe of the G buffer's barrier are
            // issued between the halves of the GELU arithmetic, so their round trips (150-250 cycles each)
            // overlap it instead of adding to the chain  S ready -> G ready  that paces the whole kernel.
            uint32_t acc[32];
            float b1_next = __ldg(p.b1 + half * 32 + lane);
            {
                const uint32_t st = cc & 1, use = cc >> 1;
                if (!(ok = mbar_wait(s_full + 8 * st, use & 1, abort_flag))) break;
                tc_fence_after();
                tmem_ld_32x32(lane_addr + C::COL_S + st * kChunk + half * 32, acc);
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster_relaxed(lead_s_empty + 8 * st);   // S buffer back to the MMA thread
            }
            for (int c = 0; c < n_chunks && ok; ++c, ++cc) {
                const uint32_t st = cc & 1, use = cc >> 1;
                const bool more = c + 1 < n_chunks;
                const uint32_t nst = st ^ 1, nuse = (cc + 1) >> 1;
                const bool s_ready = more && mbar_test_wait(s_full + 8 * nst, nuse & 1);
                // this warp's 32 bias values: one coalesced load (issued an iteration ahead), then broadcast reads
                // from the warp's slot -- 8 same-address 16-byte global loads per thread cost hundreds of cycles
                st_shared_f32(b1_slot + 4 * lane, b1_next);
                __syncwarp();
                if (more) b1_next = __ldg(p.b1 + (c + 1) * kChunk + half * 32 + lane);
                float v[32];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float4 b = ld_shared_f32x4(b1_slot + 16 * i);
                    v[4 * i + 0] = __uint_as_float(acc[4 * i + 0]) + b.x;
                    v[4 * i + 1] = __uint_as_float(acc[4 * i + 1]) + b.y;
                    v[4 * i + 2] = __uint_as_float(acc[4 * i + 2]) + b.z;
                    v[4 * i + 3] = __uint_as_float(acc[4 * i + 3]) + b.w;
                }
#pragma unroll
                for (int i = 0; i < 16; i += 2) gelu_erf_x2(v[i], v[i + 1]);
                if (more) {
                    if (!s_ready && !(ok = mbar_wait(s_full + 8 * nst, nuse & 1, abort_flag))) break;
                    tc_fence_after();
                    tmem_ld_32x32(lane_addr + C::COL_S + nst * kChunk + half * 32, acc);   // lands during the second half
                }
                // the G buffer is free once the second product of two chunks ago has read it
                const bool g_ready = use < 1 || mbar_test_wait(g_empty + 8 * st, (use - 1) & 1);
#pragma unroll
                for (int i = 16; i < 32; i += 2) gelu_erf_x2(v[i], v[i + 1]);
                uint4 q[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    q[i].x = pack_bf16(v[8 * i + 0], v[8 * i + 1]); q[i].y = pack_bf16(v[8 * i + 2], v[8 * i + 3]);
                    q[i].z = pack_bf16(v[8 * i + 4], v[8 * i + 5]); q[i].w = pack_bf16(v[8 * i + 6], v[8 * i + 7]);
                }
                if (!g_ready && !(ok = mbar_wait(g_empty + 8 * st, (use - 1) & 1, abort_flag))) break;
#pragma unroll
                for (int i = 0; i < 4; ++i) st_shared_v4(gs + st * C::G_BYTES + sw128(r, half * 4 + i), q[i]);
                fence_proxy_async();     // generic-proxy writes -> visible to the tensor core's reads
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster_release_cta(lead_g_full + 8 * st);
                if (more) {
                    tmem_ld_wait();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster_relaxed(lead_s_empty + 8 * nst);
                }
            }
            if (!ok) break;
            // ---- end of the block: out = O + b2 + X ----
            if (!(ok = final_rows(nb, blk))) break;
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
    cluster_sync_all();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc<2>(tmem, C::TMEM_COLS);
    }
}

}  // namespace tcff
}  // namespace rlx
