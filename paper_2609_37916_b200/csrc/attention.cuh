// Key-padding-masked scaled-dot-product attention with online softmax, reading q/k/v as strided
// views of the packed [T, 3H] projection (no split / transpose copies).
//
//  attention_bf16_kernel: bf16 in/out.  One CTA = 128 query rows of one (sequence, head); 8 warps of
//    16 rows each.  K/V stream through shared memory in 64-key blocks (cp.async, 4-stage ring, three
//    blocks in flight), QK^T and PV run on the warp-level tensor-core path (mma.sync m16n8k16, fp32
//    accumulate), the softmax state (running max) lives in registers and is reduced with quad
//    shuffles, the row sums come from an extra ones column of the PV product; the 1/sqrt(d)*log2(e)
//    scale is folded into the exp2 argument.  At head_dim 32 the online-softmax step is 32 keys (half a
//    staged block): 64 registers per thread, four CTAs per SM instead of three (-6 % on the 256 x 256
//    workload; at head_dim 64, and in the mask-kind / rotary modes, the 64-key step is kept).  head_dim 128
//    (mask-kind entry point only) runs one CTA per SM with the 32-key step: 64 output accumulators and
//    32 Q-fragment registers per thread leave no room for more.  Key blocks beyond the
//    last valid key are never loaded; masking runs only in blocks that contain an invalid key.
//  attention_f32_kernel: fp32 in/out CUDA-core kernel, one warp per query row, K/V staged in shared
//    memory 32 keys at a time, warp-shuffle reductions.  Reference-precision mode for testing.
#pragma once
#include "common.cuh"

namespace rlx {

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    const int sz = valid ? 16 : 0;  // src-size 0 -> the 16 destination bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Blackwell packed fp32 arithmetic: one issue slot per register PAIR.  The MMA accumulator quads are
// even-aligned, so (c0,c1) and (c2,c3) pack without a move.
__device__ __forceinline__ uint64_t att_pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void att_unpack2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t att_fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t att_mul2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

constexpr int kAttBlockM = 128;  // query rows per CTA (8 warps x 16 rows)
constexpr int kAttBlockN = 64;   // keys per shared-memory stage (default ring, see AttRing)
constexpr int kAttStages = 4;    // K/V ring depth of the default ring (three blocks in flight ahead of the one being used)
constexpr int kAttThreads = 256;
constexpr int kAttMaxSeq = 512;

// Keys per shared-memory stage and depth of the K/V ring.  The encoder's own shape (head_dim 32, at most 512 keys,
// no window, no rotation: the launcher's choice, kernel parameter WIDE) takes 128-key stages in a two-deep ring: a sequence is one to four stages, so half as
// many CTA-wide barriers are crossed for the same shared memory (-5 % at 256 x 256).  Long sequences (the mask
// kinds, rotary q/k, head_dim 64 / 128) keep 64-key stages four deep: with thousands of keys the prefetch
// distance matters more than the barrier count (the 128 x 2 ring measured 30-50 % slower there).
template <bool WIDE>
struct AttRing {
    static constexpr int BN = WIDE ? 128 : kAttBlockN;
    static constexpr int ST = WIDE ? 2 : kAttStages;
};

template <int D, int BN = kAttBlockN, int ST = kAttStages>
struct AttSmem {
    static constexpr int kStride = D + 8;  // +16 bytes per row: conflict-free ldmatrix
    __nv_bfloat16 q[kAttBlockM * kStride];  // Q tile; reused as the output staging tile at the end
    __nv_bfloat16 k[ST][BN * kStride];
    __nv_bfloat16 v[ST][BN * kStride];
    float bias[kAttMaxSeq];                 // padded mode: 0 for a valid key, -inf for a masked one
    int blk_full[kAttMaxSeq / BN];          // padded mode: 1 when all keys of the block are valid
    int kv_end;
    int q_any;
};

// Positional visibility and rotary embedding (packed mode only; template switches, so the encoder's
// instantiation carries none of it):
//   MK = 1: key k is visible to query i iff  i - window < k <= i  (causal when window >= the sequence
//           length).  Key blocks wholly outside a CTA's rows are never loaded, blocks wholly outside a
//           warp's 16 rows are skipped by that warp, and the element test runs only in blocks that a
//           boundary crosses.
//   kv_group > 1: grouped-query layout, q head j reads k/v head j / kv_group (packed mode only).
//   ROPE:   q and k rows are rotated in shared memory after they land ("rotate-half" pairing of column
//           j with j + D/2 by the angle whose cosine / sine the caller tabulates per position), in fp32,
//           and rounded back to bf16 for the tensor-core products.  Each thread rotates what it copied
//           itself, one key block ahead of the block being multiplied, so no barrier is added.
struct AttKind {
    int window;
    const float* rope_cos;   // [max_len, D/2]
    const float* rope_sin;
    int kv_group;            // q heads per k/v head (1: plain multi-head layout [q | k | v] of width 3H)
};

// Two addressing modes share the kernel:
//   padded: seq_start == nullptr.  Sequence b occupies rows b*S .. b*S+S; `mask` flags valid keys.
//   packed: rows of sequence b are seq_start[b] .. seq_start[b]+seq_len[b], all valid (mask unused).
template <int D, int MK = 0, bool ROPE = false, int KS = (((D == 32 && MK == 0 && !ROPE) || D == 128) ? 32 : 64),
          int MINB = (D == 32 ? (KS == 32 ? 4 : 3) : D == 64 ? 2 : 1), bool WIDE = false>
__global__ void __launch_bounds__(kAttThreads, MINB)
attention_bf16_kernel(const __nv_bfloat16* __restrict__ qkv, const int32_t* __restrict__ mask,
                      const int32_t* __restrict__ seq_start, const int32_t* __restrict__ seq_len,
                      __nv_bfloat16* __restrict__ ctx, int S, int H, float scale_log2e, AttKind kind) {
    constexpr int BN = AttRing<WIDE>::BN, ST = AttRing<WIDE>::ST;
    using SM = AttSmem<D, BN, ST>;
    constexpr int STR = SM::kStride;
    constexpr int KT = D / 16;       // k-tiles of the QK^T product
    constexpr int ND = D / 8;        // n-tiles of the PV product
    constexpr int CH = D / 8;        // 16-byte chunks per row
    extern __shared__ __align__(16) unsigned char att_smem_raw[];
    SM& sm = *reinterpret_cast<SM*>(att_smem_raw);

    pdl_launch_dependents();
    pdl_wait();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int q0 = blockIdx.x * kAttBlockM, head = blockIdx.y, b = blockIdx.z;
    const bool packed = seq_start != nullptr;
    const size_t row0 = packed ? (size_t)__ldg(seq_start + b) : (size_t)b * S;
    const int len = packed ? __ldg(seq_len + b) : S;   // rows of this sequence present in memory
    if (q0 >= len) return;                              // whole CTA outside the sequence (uniform)
    // row layout: H columns of q heads, then H / kv_group of k heads, then as many of v heads
    const int Hkv = H / kind.kv_group;
    const int ld = H + 2 * Hkv;
    const __nv_bfloat16* qbase = qkv + row0 * ld + head * D;
    const __nv_bfloat16* kbase = qkv + row0 * ld + H + (head / kind.kv_group) * D;
    const __nv_bfloat16* vbase = kbase + Hkv;

    int kv_end = len;
    if (!packed) {
        if (tid == 0) { sm.kv_end = 0; sm.q_any = 0; }
        if (tid < kAttMaxSeq / BN) sm.blk_full[tid] = 1;
        __syncthreads();
        int last = 0, any = 0;
        const int spad = (S + BN - 1) / BN * BN;
        for (int k = tid; k < spad; k += kAttThreads) {
            const bool valid = (k < S) && (__ldg(mask + row0 + k) != 0);
            sm.bias[k] = valid ? 0.f : -INFINITY;
            if (valid) {
                last = k + 1;
                any |= (k >= q0 && k < q0 + kAttBlockM);
            } else {
                sm.blk_full[k / BN] = 0;   // benign race: every writer stores 0
            }
        }
        if (last) atomicMax(&sm.kv_end, last);
        if (any) atomicOr(&sm.q_any, 1);
        __syncthreads();
        kv_end = sm.kv_end;
        if (kv_end == 0 || sm.q_any == 0) {
            // nothing observable in this block: write zeros so later stages only ever see finite values
            for (int i = tid; i < kAttBlockM * CH; i += kAttThreads) {
                const int r = i / CH, c = i % CH;
                if (q0 + r < S)
                    *reinterpret_cast<uint4*>(ctx + (row0 + q0 + r) * H + head * D + c * 8) = make_uint4(0, 0, 0, 0);
            }
            return;
        }
    }
    int jb0 = 0, nblk = (kv_end + BN - 1) / BN;   // key blocks jb0 .. nblk-1
    if (MK) {
        const int q_hi = min(q0 + kAttBlockM, len);                // one past this CTA's last real row
        jb0 = max(0, q0 - kind.window + 1) / BN;
        nblk = (q_hi + BN - 1) / BN;
    }

    auto load_rows = [&](const __nv_bfloat16* base, __nv_bfloat16* dst, int first_row, int nrows) {
        for (int i = tid; i < nrows * CH; i += kAttThreads) {
            const int r = i / CH, c = i % CH;
            const bool ok = first_row + r < len;
            const __nv_bfloat16* src = base + (size_t)(ok ? first_row + r : 0) * ld + c * 8;
            cp_async16(smem_u32(dst + r * STR + c * 8), src, ok);
        }
    };
    // Rotary mode: a thread copies BOTH halves of the column pairs it will rotate (chunk c and chunk
    // c + CH/2 of a row), so that once its own copies have completed it can rotate them in place with no
    // CTA barrier in between; the barrier that publishes the tile to the other warps comes afterwards.
    auto load_rows_paired = [&](const __nv_bfloat16* base, __nv_bfloat16* dst, int first_row, int nrows) {
        constexpr int CPR = D / 16;
        for (int i = tid; i < nrows * CPR; i += kAttThreads) {
            const int r = i / CPR, c = i % CPR;
            const bool ok = first_row + r < len;
            const __nv_bfloat16* src = base + (size_t)(ok ? first_row + r : 0) * ld + c * 8;
            cp_async16(smem_u32(dst + r * STR + c * 8), src, ok);
            cp_async16(smem_u32(dst + r * STR + D / 2 + c * 8), src + D / 2, ok);
        }
    };
    auto load_qk = [&](const __nv_bfloat16* base, __nv_bfloat16* dst, int first_row, int nrows) {
        if (ROPE) load_rows_paired(base, dst, first_row, nrows);
        else load_rows(base, dst, first_row, nrows);
    };
    load_qk(qbase, sm.q, q0, kAttBlockM);
#pragma unroll
    for (int j = 0; j < ST - 1; ++j) {
        if (jb0 + j < nblk) {
            load_qk(kbase, sm.k[j], (jb0 + j) * BN, BN);
            load_rows(vbase, sm.v[j], (jb0 + j) * BN, BN);
        }
        cp_async_commit();
    }
    // rotate, in place, the column pairs of a q or k tile that THIS thread copied (same task mapping as
    // load_rows_paired); row r holds position first_pos + r
    auto rope_rows = [&](__nv_bfloat16* tile, int first_pos, int nrows) {
        constexpr int CPR = D / 16;   // tasks per row: 8 (lo, hi) column pairs each
        for (int i = tid; i < nrows * CPR; i += kAttThreads) {
            const int r = i / CPR, c = i % CPR;
            const int pos = first_pos + r;
            if (pos >= len) continue;   // zero-filled row
            uint4* plo = reinterpret_cast<uint4*>(tile + r * STR + c * 8);
            uint4* phi = reinterpret_cast<uint4*>(tile + r * STR + D / 2 + c * 8);
            uint4 lo = *plo, hi = *phi;
            const float4* pc = reinterpret_cast<const float4*>(kind.rope_cos + (size_t)pos * (D / 2) + c * 8);
            const float4* ps = reinterpret_cast<const float4*>(kind.rope_sin + (size_t)pos * (D / 2) + c * 8);
            rope_rotate8(lo, hi, __ldg(pc), __ldg(pc + 1), __ldg(ps), __ldg(ps + 1));
            *plo = lo;
            *phi = hi;
        }
    };

    uint32_t qf[KT][4];
    float o[ND][4];
#pragma unroll
    for (int i = 0; i < ND; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY};   // running max (scaled)
    // Running row sums come out of the tensor cores: P times a column of ones accumulates, in every
    // column of this extra n-tile, the sum of the bf16-rounded probabilities -- the same values the
    // P V product uses, so numerator and denominator of the softmax agree.
    float l_acc[4] = {0.f, 0.f, 0.f, 0.f};
    constexpr uint32_t kOnesBf16x2 = 0x3F803F80u;
    const int g = lane >> 2, t4 = lane & 3;
    const bool warp_active = q0 + warp * 16 < len;   // warps whose 16 rows lie past the sequence only sync

    const int r0 = q0 + warp * 16;   // first query row of this warp (index within the sequence)
    for (int j = jb0; j < nblk; ++j) {
        const int buf = (j - jb0) % ST;
        cp_async_wait<ST - 2>();   // block j (and Q) have landed
        if (ROPE && j == jb0) {            // own copies of Q and the first key block: rotate before publishing
            rope_rows(sm.q, q0, kAttBlockM);
            rope_rows(sm.k[buf], j * BN, BN);
        }
        __syncthreads();                   // ... for every thread; and block j-1's stage is free
        if (j + ST - 1 < nblk) {
            const int nb = (j - jb0 + ST - 1) % ST;
            load_qk(kbase, sm.k[nb], (j + ST - 1) * BN, BN);
            load_rows(vbase, sm.v[nb], (j + ST - 1) * BN, BN);
        }
        cp_async_commit();
        if (ROPE && j + 1 < nblk) {
            // block j+1 is rotated one step ahead by the threads that copied it; nobody reads it before
            // the barrier at the top of the next iteration
            cp_async_wait<ST - 2>();
            rope_rows(sm.k[(j + 1 - jb0) % ST], (j + 1) * BN, BN);
        }
        if (!warp_active) continue;
        if (j == jb0) {
#pragma unroll
            for (int kt = 0; kt < KT; ++kt) {
                const int r = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
                const int c = kt * 16 + (lane >> 4) * 8;
                ldmatrix_x4(smem_u32(sm.q + r * STR + c), qf[kt][0], qf[kt][1], qf[kt][2], qf[kt][3]);
            }
        }
        const int k0 = j * BN;
        if (MK && (k0 > r0 + 15 || k0 + BN - 1 <= r0 - kind.window)) continue;   // nothing visible
        // The online-softmax step covers KS keys (64: the whole staged block; 32: half of it, which halves
        // the score and probability registers and lets a fourth CTA fit on the SM at head_dim 32).
        constexpr int NT = KS / 8;   // score n-tiles per step
#pragma unroll
        for (int hf = 0; hf < BN / KS; ++hf) {
        // packed rows: the sequence's last key block may end before this step's keys begin (uniform in the CTA)
        if (MK == 0 && hf > 0 && packed && k0 + hf * KS >= len) break;
        // ---- S = Q K^T for KS keys: NT n-tiles x 4 accumulators ----
        float s[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
            for (int kp = 0; kp < KT / 2; ++kp) {  // two k-tiles per ldmatrix.x4
                uint32_t b0, b1, b2, b3;
                const int mi = lane >> 3;
                const int r = (hf * NT + nt) * 8 + (lane & 7);
                const int c = kp * 32 + (mi & 1) * 8 + (mi >> 1) * 16;
                ldmatrix_x4(smem_u32(sm.k[buf] + r * STR + c), b0, b1, b2, b3);
                mma_bf16_16816(s[nt], qf[2 * kp][0], qf[2 * kp][1], qf[2 * kp][2], qf[2 * kp][3], b0, b1);
                mma_bf16_16816(s[nt], qf[2 * kp + 1][0], qf[2 * kp + 1][1], qf[2 * kp + 1][2], qf[2 * kp + 1][3], b2, b3);
            }
        }
        // ---- masking only where the block has an invalid key ----
        if (MK) {
            // the block needs the element test unless every key is visible to all 16 rows
            if (k0 + BN > len || k0 + BN - 1 > r0 || k0 <= r0 + 15 - kind.window) {
                const int ia = r0 + g, ib = ia + 8;   // rows of accumulators {0,1} and {2,3}
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const int kk = k0 + (hf * NT + nt) * 8 + 2 * t4;
                    if (!(kk < len && kk <= ia && kk > ia - kind.window)) s[nt][0] = -INFINITY;
                    if (!(kk + 1 < len && kk + 1 <= ia && kk + 1 > ia - kind.window)) s[nt][1] = -INFINITY;
                    if (!(kk < len && kk <= ib && kk > ib - kind.window)) s[nt][2] = -INFINITY;
                    if (!(kk + 1 < len && kk + 1 <= ib && kk + 1 > ib - kind.window)) s[nt][3] = -INFINITY;
                }
            }
        } else {
            const bool need_mask = packed ? (k0 + BN > len) : (sm.blk_full[j] == 0);
            if (need_mask) {
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const int kk = k0 + (hf * NT + nt) * 8 + 2 * t4;
                    const bool v0 = packed ? (kk < len) : (sm.bias[kk] == 0.f);
                    const bool v1 = packed ? (kk + 1 < len) : (sm.bias[kk + 1] == 0.f);
                    if (!v0) { s[nt][0] = -INFINITY; s[nt][2] = -INFINITY; }
                    if (!v1) { s[nt][1] = -INFINITY; s[nt][3] = -INFINITY; }
                }
            }
        }
        // ---- running max on raw scores (the positive scale commutes with max) ----
        float mx[2] = {fmaxf(s[0][0], s[0][1]), fmaxf(s[0][2], s[0][3])};
#pragma unroll
        for (int nt = 1; nt < NT; ++nt) {
            mx[0] = fmax3(mx[0], s[nt][0], s[nt][1]);
            mx[1] = fmax3(mx[1], s[nt][2], s[nt][3]);
        }
        float alpha[2], msub[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
            const float m_new = fmaxf(m_run[r], mx[r] * scale_log2e);
            msub[r] = (m_new == -INFINITY) ? 0.f : m_new;   // all keys so far masked: avoid inf - inf
            alpha[r] = fast_exp2(m_run[r] - msub[r]);        // m_run = -inf -> 0
            m_run[r] = m_new;
        }
        const uint64_t a0 = att_pack2(alpha[0], alpha[0]), a1 = att_pack2(alpha[1], alpha[1]);
#pragma unroll
        for (int nd = 0; nd < ND; ++nd) {
            att_unpack2(att_mul2(att_pack2(o[nd][0], o[nd][1]), a0), o[nd][0], o[nd][1]);
            att_unpack2(att_mul2(att_pack2(o[nd][2], o[nd][3]), a1), o[nd][2], o[nd][3]);
        }
        l_acc[0] *= alpha[0];
        l_acc[2] *= alpha[1];
        // ---- P = exp2(S*c - m), packed to bf16 A fragments ----
        uint32_t pf[NT / 2][4];
        const uint64_t c2 = att_pack2(scale_log2e, scale_log2e);
        const uint64_t nm0 = att_pack2(-msub[0], -msub[0]), nm1 = att_pack2(-msub[1], -msub[1]);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            float x0, x1, x2, x3;
            att_unpack2(att_fma2(att_pack2(s[nt][0], s[nt][1]), c2, nm0), x0, x1);
            att_unpack2(att_fma2(att_pack2(s[nt][2], s[nt][3]), c2, nm1), x2, x3);
            pf[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(fast_exp2(x0), fast_exp2(x1));
            pf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(fast_exp2(x2), fast_exp2(x3));
        }
        // ---- O += P V ----
#pragma unroll
        for (int kk = 0; kk < NT / 2; ++kk) {
            mma_bf16_16816(l_acc, pf[kk][0], pf[kk][1], pf[kk][2], pf[kk][3], kOnesBf16x2, kOnesBf16x2);
#pragma unroll
            for (int np = 0; np < ND / 2; ++np) {  // two n-tiles per ldmatrix.x4.trans
                uint32_t b0, b1, b2, b3;
                const int mi = lane >> 3;
                const int r = (hf * (NT / 2) + kk) * 16 + (mi & 1) * 8 + (lane & 7);
                const int c = np * 16 + (mi >> 1) * 8;
                ldmatrix_x4_trans(smem_u32(sm.v[buf] + r * STR + c), b0, b1, b2, b3);
                mma_bf16_16816(o[2 * np], pf[kk][0], pf[kk][1], pf[kk][2], pf[kk][3], b0, b1);
                mma_bf16_16816(o[2 * np + 1], pf[kk][0], pf[kk][1], pf[kk][2], pf[kk][3], b2, b3);
            }
        }
        }   // hf
    }
    cp_async_wait<0>();
    if (!warp_active) return;

    // ---- normalise, stage this warp's 16 x D tile in its own rows of the Q buffer, store 16 B / lane ----
    float l_run[2] = {l_acc[0], l_acc[2]};   // every column of the ones n-tile holds the full row sum
#pragma unroll
    for (int r = 0; r < 2; ++r) l_run[r] = l_run[r] > 0.f ? 1.0f / l_run[r] : 0.f;
    __nv_bfloat16* stage = sm.q + warp * 16 * STR;   // only this warp ever touched these rows
#pragma unroll
    for (int nd = 0; nd < ND; ++nd) {
        *reinterpret_cast<uint32_t*>(stage + g * STR + nd * 8 + 2 * t4) = pack_bf16(o[nd][0] * l_run[0], o[nd][1] * l_run[0]);
        *reinterpret_cast<uint32_t*>(stage + (g + 8) * STR + nd * 8 + 2 * t4) = pack_bf16(o[nd][2] * l_run[1], o[nd][3] * l_run[1]);
    }
    __syncwarp();
    for (int i = lane; i < 16 * CH; i += 32) {
        const int r = i / CH, c = i % CH;
        const int qr = q0 + warp * 16 + r;
        if (qr < len)
            *reinterpret_cast<uint4*>(ctx + (row0 + qr) * H + head * D + c * 8) =
                *reinterpret_cast<const uint4*>(stage + r * STR + c * 8);
    }
}

// ----------------------------------------------------------------------------------------------
// fp32 reference-precision mode: one warp per query row, 4 warps per CTA sharing the K/V stage.
// ----------------------------------------------------------------------------------------------
constexpr int kAttF32Warps = 4;

template <int D>
__global__ void __launch_bounds__(kAttF32Warps * 32)
attention_f32_kernel(const float* __restrict__ qkv, const int32_t* __restrict__ mask, float* __restrict__ ctx,
                     int S, int H, float scale) {
    constexpr int CPL = D / 32;  // output columns per lane
    __shared__ float sk[32][D + 1];
    __shared__ float sv[32][D + 1];
    __shared__ float sq[kAttF32Warps][D];
    __shared__ int smask[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int head = blockIdx.y, b = blockIdx.z;
    const int qi = blockIdx.x * kAttF32Warps + warp;
    const size_t row0 = (size_t)b * S;
    const int ld = 3 * H;
    const bool active = qi < S;
    if (active)
        for (int c = lane; c < D; c += 32) sq[warp][c] = qkv[(row0 + qi) * ld + head * D + c];
    float m_run = -INFINITY, l_run = 0.f, acc[CPL];
#pragma unroll
    for (int i = 0; i < CPL; ++i) acc[i] = 0.f;

    for (int k0 = 0; k0 < S; k0 += 32) {
        __syncthreads();
        for (int i = threadIdx.x; i < 32 * D; i += kAttF32Warps * 32) {
            const int r = i / D, c = i % D;
            const bool ok = k0 + r < S;
            sk[r][c] = ok ? qkv[(row0 + k0 + r) * ld + H + head * D + c] : 0.f;
            sv[r][c] = ok ? qkv[(row0 + k0 + r) * ld + 2 * H + head * D + c] : 0.f;
        }
        if (threadIdx.x < 32) smask[threadIdx.x] = (k0 + threadIdx.x < S) ? mask[row0 + k0 + threadIdx.x] : 0;
        __syncthreads();
        if (!active) continue;
        // lane = key: score of this lane's key
        float sc = 0.f;
#pragma unroll 8
        for (int c = 0; c < D; ++c) sc += sq[warp][c] * sk[lane][c];
        const bool valid = smask[lane] != 0;
        sc = valid ? sc * scale : -INFINITY;
        const float m_new = fmaxf(m_run, warp_max(sc));
        if (m_new == -INFINITY) continue;  // every key so far is masked
        const float alpha = expf(m_run - m_new);
        const float p = valid ? expf(sc - m_new) : 0.f;
        l_run = l_run * alpha + warp_sum(p);
        m_run = m_new;
#pragma unroll
        for (int i = 0; i < CPL; ++i) acc[i] *= alpha;
        for (int kk = 0; kk < 32; ++kk) {
            const float pk = __shfl_sync(0xffffffffu, p, kk);
#pragma unroll
            for (int i = 0; i < CPL; ++i) acc[i] += pk * sv[kk][lane + 32 * i];
        }
    }
    if (active) {
        const float inv = l_run > 0.f ? 1.0f / l_run : 0.f;
#pragma unroll
        for (int i = 0; i < CPL; ++i) ctx[(row0 + qi) * H + head * D + lane + 32 * i] = acc[i] * inv;
    }
}

}  // namespace rlx
