// Key-padding-masked scaled-dot-product attention with online softmax, reading q/k/v as strided
// views of the packed [T, 3H] projection (no split / transpose copies).
//
//  attention_bf16_kernel: bf16 in/out.  One CTA = 64 query rows of one (sequence, head); 4 warps of
//    16 rows each.  K/V stream through shared memory in 64-key blocks (cp.async double buffer),
//    QK^T and PV run on the warp-level tensor-core path (mma.sync m16n8k16, fp32 accumulate), the
//    softmax state (running max / sum) lives in registers and is reduced with quad shuffles.
//    Key blocks beyond the last valid key are never loaded; masked keys get a -inf bias.
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

constexpr int kAttBlockM = 64;   // query rows per CTA
constexpr int kAttBlockN = 64;   // keys per shared-memory block
constexpr int kAttThreads = 128;

template <int D>
struct AttSmem {
    static constexpr int kStride = D + 8;  // +16 bytes per row: conflict-free ldmatrix
    __nv_bfloat16 q[kAttBlockM * kStride];
    __nv_bfloat16 k[2][kAttBlockN * kStride];
    __nv_bfloat16 v[2][kAttBlockN * kStride];
    float bias[512 + 64];  // 0 for a valid key, -inf for a masked one (seq <= 512 supported here)
    int kv_end;
    int q_any;
};

template <int D>
__global__ void __launch_bounds__(kAttThreads)
attention_bf16_kernel(const __nv_bfloat16* __restrict__ qkv, const int32_t* __restrict__ mask,
                      __nv_bfloat16* __restrict__ ctx, int S, int H, float scale_log2e) {
    using SM = AttSmem<D>;
    constexpr int STR = SM::kStride;
    constexpr int KT = D / 16;       // k-tiles of the QK^T product
    constexpr int ND = D / 8;        // n-tiles of the PV product
    constexpr int CH = D / 8;        // 16-byte chunks per row
    extern __shared__ __align__(16) unsigned char att_smem_raw[];
    SM& sm = *reinterpret_cast<SM*>(att_smem_raw);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int q0 = blockIdx.x * kAttBlockM, head = blockIdx.y, b = blockIdx.z;
    const size_t row0 = (size_t)b * S;
    const int ld = 3 * H;
    const __nv_bfloat16* qbase = qkv + row0 * ld + head * D;
    const __nv_bfloat16* kbase = qbase + H;
    const __nv_bfloat16* vbase = qbase + 2 * H;

    if (tid == 0) { sm.kv_end = 0; sm.q_any = 0; }
    __syncthreads();
    {
        int last = 0, any = 0;
        const int spad = (S + 63) & ~63;
        for (int k = tid; k < spad; k += kAttThreads) {
            const bool valid = (k < S) && (__ldg(mask + row0 + k) != 0);
            sm.bias[k] = valid ? 0.f : -INFINITY;
            if (valid) {
                last = k + 1;
                any |= (k >= q0 && k < q0 + kAttBlockM);
            }
        }
        if (last) atomicMax(&sm.kv_end, last);
        if (any) atomicOr(&sm.q_any, 1);
    }
    __syncthreads();
    const int kv_end = sm.kv_end;
    if (kv_end == 0 || sm.q_any == 0) {
        // nothing observable in this block: write zeros so later stages only ever see finite values
        for (int i = tid; i < kAttBlockM * CH; i += kAttThreads) {
            const int r = i / CH, c = i % CH;
            if (q0 + r < S)
                *reinterpret_cast<uint4*>(ctx + (row0 + q0 + r) * H + head * D + c * 8) = make_uint4(0, 0, 0, 0);
        }
        return;
    }
    const int nblk = (kv_end + kAttBlockN - 1) / kAttBlockN;

    auto load_rows = [&](const __nv_bfloat16* base, __nv_bfloat16* dst, int first_row) {
        for (int i = tid; i < 64 * CH; i += kAttThreads) {
            const int r = i / CH, c = i % CH;
            const bool ok = first_row + r < S;
            const __nv_bfloat16* src = base + (size_t)(ok ? first_row + r : 0) * ld + c * 8;
            cp_async16(smem_u32(dst + r * STR + c * 8), src, ok);
        }
    };
    load_rows(qbase, sm.q, q0);
    load_rows(kbase, sm.k[0], 0);
    load_rows(vbase, sm.v[0], 0);
    cp_async_commit();

    uint32_t qf[KT][4];
    float o[ND][4];
#pragma unroll
    for (int i = 0; i < ND; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    const int g = lane >> 2, t4 = lane & 3;

    for (int j = 0; j < nblk; ++j) {
        const int buf = j & 1;
        if (j + 1 < nblk) {
            load_rows(kbase, sm.k[buf ^ 1], (j + 1) * kAttBlockN);
            load_rows(vbase, sm.v[buf ^ 1], (j + 1) * kAttBlockN);
        }
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();
        if (j == 0) {
#pragma unroll
            for (int kt = 0; kt < KT; ++kt) {
                const int r = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
                const int c = kt * 16 + (lane >> 4) * 8;
                ldmatrix_x4(smem_u32(sm.q + r * STR + c), qf[kt][0], qf[kt][1], qf[kt][2], qf[kt][3]);
            }
        }
        // ---- S = Q K^T for 64 keys: 8 n-tiles x 4 accumulators ----
        float s[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
            for (int kp = 0; kp < KT / 2; ++kp) {  // two k-tiles per ldmatrix.x4
                uint32_t b0, b1, b2, b3;
                const int mi = lane >> 3;
                const int r = nt * 8 + (lane & 7);
                const int c = kp * 32 + (mi & 1) * 8 + (mi >> 1) * 16;
                ldmatrix_x4(smem_u32(sm.k[buf] + r * STR + c), b0, b1, b2, b3);
                mma_bf16_16816(s[nt], qf[2 * kp][0], qf[2 * kp][1], qf[2 * kp][2], qf[2 * kp][3], b0, b1);
                mma_bf16_16816(s[nt], qf[2 * kp + 1][0], qf[2 * kp + 1][1], qf[2 * kp + 1][2], qf[2 * kp + 1][3], b2, b3);
            }
        }
        // ---- scale, mask bias, running max ----
        const float* bias = sm.bias + j * kAttBlockN;
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            const float b0 = bias[nt * 8 + 2 * t4], b1 = bias[nt * 8 + 2 * t4 + 1];
            s[nt][0] = s[nt][0] * scale_log2e + b0;
            s[nt][1] = s[nt][1] * scale_log2e + b1;
            s[nt][2] = s[nt][2] * scale_log2e + b0;
            s[nt][3] = s[nt][3] * scale_log2e + b1;
            mx[0] = fmaxf(mx[0], fmaxf(s[nt][0], s[nt][1]));
            mx[1] = fmaxf(mx[1], fmaxf(s[nt][2], s[nt][3]));
        }
        float alpha[2], msub[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
            mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
            const float m_new = fmaxf(m_run[r], mx[r]);
            msub[r] = (m_new == -INFINITY) ? 0.f : m_new;   // all keys so far masked: avoid inf - inf
            alpha[r] = fast_exp2(m_run[r] - msub[r]);        // m_run = -inf -> 0
            m_run[r] = m_new;
            l_run[r] *= alpha[r];
        }
#pragma unroll
        for (int nd = 0; nd < ND; ++nd) {
            o[nd][0] *= alpha[0]; o[nd][1] *= alpha[0];
            o[nd][2] *= alpha[1]; o[nd][3] *= alpha[1];
        }
        // ---- P = exp2(S - m), row sums, pack to bf16 A fragments ----
        uint32_t pf[4][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            const float p0 = fast_exp2(s[nt][0] - msub[0]);
            const float p1 = fast_exp2(s[nt][1] - msub[0]);
            const float p2 = fast_exp2(s[nt][2] - msub[1]);
            const float p3 = fast_exp2(s[nt][3] - msub[1]);
            l_run[0] += p0 + p1;
            l_run[1] += p2 + p3;
            pf[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p0, p1);
            pf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2, p3);
        }
        // ---- O += P V ----
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
            for (int np = 0; np < ND / 2; ++np) {  // two n-tiles per ldmatrix.x4.trans
                uint32_t b0, b1, b2, b3;
                const int mi = lane >> 3;
                const int r = kk * 16 + (mi & 1) * 8 + (lane & 7);
                const int c = np * 16 + (mi >> 1) * 8;
                ldmatrix_x4_trans(smem_u32(sm.v[buf] + r * STR + c), b0, b1, b2, b3);
                mma_bf16_16816(o[2 * np], pf[kk][0], pf[kk][1], pf[kk][2], pf[kk][3], b0, b1);
                mma_bf16_16816(o[2 * np + 1], pf[kk][0], pf[kk][1], pf[kk][2], pf[kk][3], b2, b3);
            }
        }
        __syncthreads();  // everyone is done with this buffer before the next prefetch overwrites it
    }
    cp_async_wait<0>();

    // ---- normalise and store ----
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
        l_run[r] = l_run[r] > 0.f ? 1.0f / l_run[r] : 0.f;
    }
    const int qr0 = q0 + warp * 16 + g, qr1 = qr0 + 8;
#pragma unroll
    for (int nd = 0; nd < ND; ++nd) {
        const int col = head * D + nd * 8 + 2 * t4;
        if (qr0 < S)
            *reinterpret_cast<uint32_t*>(ctx + (row0 + qr0) * H + col) = pack_bf16(o[nd][0] * l_run[0], o[nd][1] * l_run[0]);
        if (qr1 < S)
            *reinterpret_cast<uint32_t*>(ctx + (row0 + qr1) * H + col) = pack_bf16(o[nd][2] * l_run[1], o[nd][3] * l_run[1]);
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
