// Memory-bound row kernels: embedding gather + LayerNorm, LayerNorm, masked mean-pool + L2 norm.
// One warp owns one row of H = NV * 128 bf16 values; each lane holds NV vectors of 4 values
// (8-byte loads, a warp instruction covers 256 contiguous bytes).  Statistics in fp32, two-pass
// on registers (mean, then centred sum of squares), biased variance, eps inside the square root.
#pragma once
#include "common.cuh"

namespace rlx {

constexpr int kRowWarps = 8;  // rows per CTA

template <int NV>
__device__ __forceinline__ void ln_normalise_store(float (&v)[NV * 4], const float* __restrict__ gamma,
                                                   const float* __restrict__ beta, float eps, int lane,
                                                   __nv_bfloat16* __restrict__ out_row) {
    constexpr int H = NV * 128;
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < NV * 4; ++i) s += v[i];
    const float mean = warp_sum(s) / (float)H;  // true division: a constant row has exactly zero deviation
    float q = 0.f;
#pragma unroll
    for (int i = 0; i < NV * 4; ++i) {
        v[i] -= mean;
        q += v[i] * v[i];
    }
    const float var = warp_sum(q) / (float)H;
    const float rstd = 1.0f / sqrtf(var + eps);
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        const int col = (i * 32 + lane) * 4;
        const float4 g = __ldg(reinterpret_cast<const float4*>(gamma + col));
        const float4 b = __ldg(reinterpret_cast<const float4*>(beta + col));
        uint2 o;
        o.x = pack_bf16(v[i * 4 + 0] * rstd * g.x + b.x, v[i * 4 + 1] * rstd * g.y + b.y);
        o.y = pack_bf16(v[i * 4 + 2] * rstd * g.z + b.z, v[i * 4 + 3] * rstd * g.w + b.w);
        *reinterpret_cast<uint2*>(out_row + col) = o;
    }
}

// gamma / beta of this lane's columns, loaded once and kept in registers by kernels that normalise
// several rows per warp
template <int NV>
struct LnAffine {
    float4 g[NV], b[NV];
    __device__ __forceinline__ void load(const float* __restrict__ gamma, const float* __restrict__ beta, int lane) {
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            g[i] = __ldg(reinterpret_cast<const float4*>(gamma + (i * 32 + lane) * 4));
            b[i] = __ldg(reinterpret_cast<const float4*>(beta + (i * 32 + lane) * 4));
        }
    }
};

template <int NV>
__device__ __forceinline__ void ln_normalise_store(float (&v)[NV * 4], const LnAffine<NV>& af, float eps, int lane,
                                                   __nv_bfloat16* __restrict__ out_row) {
    constexpr int H = NV * 128;
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < NV * 4; ++i) s += v[i];
    const float mean = warp_sum(s) / (float)H;  // true division: a constant row has exactly zero deviation
    float q = 0.f;
#pragma unroll
    for (int i = 0; i < NV * 4; ++i) {
        v[i] -= mean;
        q += v[i] * v[i];
    }
    const float var = warp_sum(q) / (float)H;
    const float rstd = 1.0f / sqrtf(var + eps);
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        const int col = (i * 32 + lane) * 4;
        uint2 o;
        o.x = pack_bf16(v[i * 4 + 0] * rstd * af.g[i].x + af.b[i].x, v[i * 4 + 1] * rstd * af.g[i].y + af.b[i].y);
        o.y = pack_bf16(v[i * 4 + 2] * rstd * af.g[i].z + af.b[i].z, v[i * 4 + 3] * rstd * af.g[i].w + af.b[i].w);
        *reinterpret_cast<uint2*>(out_row + col) = o;
    }
}

// Sequence packing.  Valid tokens (mask != 0) are compacted so that sequence b owns the packed rows
// seq_start[b] .. seq_start[b] + seq_len[b]; every later kernel then works on sum(len) rows instead
// of B*S.  Exact for any 0/1 mask: positions are taken from the original index s, attention only
// ever involves a sequence's valid tokens, pooling averages exactly those rows.
//   seq_len[b]            number of valid positions of sequence b
//   seq_start[0..B]       exclusive prefix sum of seq_len (seq_start[B] = total packed rows)
//   pos_of_rank[b*S + r]  original position s of the r-th valid token of sequence b
// One CTA per sequence; the last CTA to finish (ticket counter, reset for the next launch) scans
// seq_len.  Integer work only.
constexpr int kPackThreads = 128;

__global__ void __launch_bounds__(kPackThreads)
pack_sequences_kernel(const int32_t* __restrict__ mask, int B, int S, int32_t* __restrict__ seq_len,
                      int32_t* __restrict__ seq_start, int32_t* __restrict__ pos_of_rank,
                      unsigned int* __restrict__ ticket, cudaGraphConditionalHandle cond, int cond_min_rows) {
    __shared__ int warp_cnt[kPackThreads / 32];
    __shared__ int is_last;
    pdl_launch_dependents();
    // the tables written here may still be read by the kernels of the previous forward (or sub-batch) on the
    // same workspace when this launch is a programmatic dependent of its last kernel
    pdl_wait();
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int running = 0;
    for (int base = 0; base < S; base += kPackThreads) {
        const int s = base + tid;
        const bool valid = s < S && __ldg(mask + (size_t)b * S + s) != 0;
        const unsigned bal = __ballot_sync(0xffffffffu, valid);
        if (lane == 0) warp_cnt[warp] = __popc(bal);
        __syncthreads();
        int before = 0, chunk = 0;
#pragma unroll
        for (int w = 0; w < kPackThreads / 32; ++w) {
            if (w < warp) before += warp_cnt[w];
            chunk += warp_cnt[w];
        }
        if (valid) pos_of_rank[(size_t)b * S + running + before + __popc(bal & ((1u << lane) - 1u))] = s;
        running += chunk;
        __syncthreads();
    }
    if (tid == 0) {
        seq_len[b] = running;
        __threadfence();
        is_last = (atomicAdd(ticket, 1u) == (unsigned)(B - 1));
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // exclusive scan of seq_len by the last CTA: each warp-sized chunk with shuffles, carried serially
    if (warp == 0) {
        int carry = 0;
        for (int base = 0; base < B; base += 32) {
            const int i = base + lane;
            const int v = i < B ? *((volatile int32_t*)seq_len + i) : 0;
            int incl = v;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int n = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += n;
            }
            if (i < B) seq_start[i] = carry + incl - v;
            carry += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (lane == 0) {
            seq_start[B] = carry;
            *ticket = 0;   // ready for the next launch
            // captured forwards that carry both forms of the layer: the IF / ELSE node behind this kernel takes the
            // one-kernel layer tail when there are enough packed rows for it to pay
            if (cond != 0) cudaGraphSetConditional(cond, carry >= cond_min_rows ? 1u : 0u);
        }
    }
}

// Weight matrices to pull into L2 while the first kernels of a forward run: a small batch starts from
// a cold L2 and would otherwise pay an HBM round trip at the head of every GEMM.  Runs as a side
// branch of the captured graph (nothing on the main chain waits for it).  Pieces are issued in list
// order (layer by layer) as asynchronous bulk prefetches.
constexpr int kMaxPrefetch = 96;
constexpr uint32_t kPrefetchPiece = 32 * 1024;
struct PrefetchList {
    const void* ptr[kMaxPrefetch];
    uint32_t bytes[kMaxPrefetch];        // multiples of 16
    uint32_t first_piece[kMaxPrefetch];  // running count of pieces before this matrix
    int n;
    uint32_t total_pieces;
};

__global__ void __launch_bounds__(32)
prefetch_l2_kernel(const PrefetchList pf) {
    const uint32_t stride = gridDim.x * blockDim.x;
    for (uint32_t piece = blockIdx.x * blockDim.x + threadIdx.x; piece < pf.total_pieces; piece += stride) {
        int m = 0;
        while (m + 1 < pf.n && pf.first_piece[m + 1] <= piece) ++m;
        const uint32_t off = (piece - pf.first_piece[m]) * kPrefetchPiece;
        const uint32_t sz = min(kPrefetchPiece, pf.bytes[m] - off);
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(static_cast<const char*>(pf.ptr[m]) + off), "r"(sz) : "memory");
    }
}

// Largest b with seq_start[b] <= p (seq_start is non-decreasing, seq_start[B] = total > p).
__device__ __forceinline__ int find_sequence(const int32_t* __restrict__ seq_start, int B, int p) {
    int lo = 0, hi = B;   // invariant: seq_start[lo] <= p < seq_start[hi]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(seq_start + mid) <= p) lo = mid; else hi = mid;
    }
    return lo;
}

// Fused QK-RoPE: rotates, in place, the q and k column blocks of packed [rows, ld] projections (v is
// left alone; ld = 3H, or (hq + 2 hkv) D in the grouped-query layout).  grid = (row tiles of kRopeRows, sequences); one task = eight (j, j + D/2) column pairs
// of one head of q or k of one row: 2 x 16 bytes in, 2 x 16 bytes out, consecutive lanes on consecutive
// 16-byte chunks.  A row's position is its index within its sequence.
constexpr int kRopeRows = 16;
constexpr int kRopeThreads = 256;
template <int D>
__global__ void __launch_bounds__(kRopeThreads)
qk_rope_kernel(__nv_bfloat16* __restrict__ qkv, const int32_t* __restrict__ seq_start,
               const int32_t* __restrict__ seq_len, int rot_heads, int ld, const float* __restrict__ rope_cos,
               const float* __restrict__ rope_sin) {
    constexpr int CPR = D / 16;                 // tasks per head
    const int b = blockIdx.y;
    const int len = __ldg(seq_len + b);
    const int p0 = blockIdx.x * kRopeRows;
    if (p0 >= len) return;
    const size_t row0 = (size_t)__ldg(seq_start + b);
    const int per_row = rot_heads * CPR;        // q heads then k heads: one contiguous block of rot_heads * D columns
    const int nrows = min(kRopeRows, len - p0);
    for (int i = threadIdx.x; i < nrows * per_row; i += kRopeThreads) {
        const int r = i / per_row, t = i % per_row;
        const int hd = t / CPR, c = t % CPR;    // hd in [0, rot_heads): a q head, then the k heads
        const int pos = p0 + r;
        __nv_bfloat16* base = qkv + (row0 + pos) * (size_t)ld + hd * D + c * 8;
        uint4 lo = *reinterpret_cast<const uint4*>(base), hi = *reinterpret_cast<const uint4*>(base + D / 2);
        const float4* pc = reinterpret_cast<const float4*>(rope_cos + (size_t)pos * (D / 2) + c * 8);
        const float4* ps = reinterpret_cast<const float4*>(rope_sin + (size_t)pos * (D / 2) + c * 8);
        rope_rotate8(lo, hi, __ldg(pc), __ldg(pc + 1), __ldg(ps), __ldg(ps + 1));
        *reinterpret_cast<uint4*>(base) = lo;
        *reinterpret_cast<uint4*>(base + D / 2) = hi;
    }
}

// cos / sin tables of the rotary embedding: entry [pos, j] = cos / sin(pos * theta^(-2j/D)), j < D/2.
// The angle is formed in fp64 (position times an fp64 power) and the functions are evaluated in fp64,
// so that the fp32 table entries are correctly rounded up to the last bit or so for every position.
__global__ void __launch_bounds__(256)
rope_tables_kernel(float* __restrict__ cos_tab, float* __restrict__ sin_tab, int max_len, int half_dim, double theta) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)max_len * half_dim) return;
    const int pos = (int)(i / half_dim), j = (int)(i % half_dim);
    const double freq = pow(theta, -(double)j / (double)half_dim);   // theta^(-2j/D), D = 2 * half_dim
    const double ang = (double)pos * freq;
    cos_tab[i] = (float)cos(ang);
    sin_tab[i] = (float)sin(ang);
}

// The same search done by a whole warp (p warp-uniform): every round samples 32 evenly spaced entries
// of the remaining range and a ballot picks the sub-range, so 256 sequences take two dependent loads
// instead of eight.
__device__ __forceinline__ int find_sequence_warp(const int32_t* __restrict__ seq_start, int B, int p, int lane) {
    int lo = 0, n = B;   // invariant: the answer lies in [lo, lo + n) and seq_start[lo] <= p
    while (n > 1) {
        const int step = (n + 31) >> 5;
        const int idx = lo + lane * step;
        const bool le = idx < lo + n && __ldg(seq_start + idx) <= p;   // true for a prefix of the lanes
        const int k = 31 - __clz(__ballot_sync(0xffffffffu, le));       // lane 0 is always true
        lo += k * step;
        n = min(step, n - k * step);
    }
    return lo;
}

// x[row] = LN(word[id] + pos[s] + type[0]).  Ids outside [0, V) are clamped and flagged.
// Padded mode (seq_start == nullptr): row = token t = b*S + s for all T tokens.
// Packed mode: row p < seq_start[B] belongs to sequence b = find_sequence(p) at position
// s = pos_of_rank[b*S + (p - seq_start[b])].
template <int NV>
__global__ void __launch_bounds__(kRowWarps * 32)
embed_ln_kernel(const int32_t* __restrict__ ids, const __nv_bfloat16* __restrict__ word,
                const __nv_bfloat16* __restrict__ pos, const __nv_bfloat16* __restrict__ type,
                const float* __restrict__ gamma, const float* __restrict__ beta,
                __nv_bfloat16* __restrict__ out, int T, int S, int V, float eps, int32_t* status,
                const int32_t* __restrict__ seq_start, const int32_t* __restrict__ pos_of_rank, int B) {
    constexpr int H = NV * 128;
    pdl_launch_dependents();
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * kRowWarps + (threadIdx.x >> 5);
    if (t >= T) return;
    int tok = t, s = t % S;
    if (seq_start != nullptr) {
        if (t >= __ldg(seq_start + B)) return;
        const int b = find_sequence_warp(seq_start, B, t, lane);
        s = __ldg(pos_of_rank + (size_t)b * S + (t - __ldg(seq_start + b)));
        tok = b * S + s;
    }
    int id = __ldg(ids + tok);
    if (id < 0 || id >= V) {
        if (lane == 0 && status) atomicOr(status, RLX_DEVSTAT_TOKEN_RANGE_BIT);
        id = id < 0 ? 0 : V - 1;
    }
    const __nv_bfloat16* wrow = word + (size_t)id * H;
    const __nv_bfloat16* prow = pos + (size_t)s * H;
    float v[NV * 4];
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        const int col = (i * 32 + lane) * 4;
        const uint2 a = __ldg(reinterpret_cast<const uint2*>(wrow + col));
        const uint2 b = __ldg(reinterpret_cast<const uint2*>(prow + col));
        const uint2 c = __ldg(reinterpret_cast<const uint2*>(type + col));
        v[i * 4 + 0] = bf16lo(a.x) + bf16lo(b.x) + bf16lo(c.x);
        v[i * 4 + 1] = bf16hi(a.x) + bf16hi(b.x) + bf16hi(c.x);
        v[i * 4 + 2] = bf16lo(a.y) + bf16lo(b.y) + bf16lo(c.y);
        v[i * 4 + 3] = bf16hi(a.y) + bf16hi(b.y) + bf16hi(c.y);
    }
    ln_normalise_store<NV>(v, gamma, beta, eps, lane, out + (size_t)t * H);
}

// out = LN(x) row by row (the residual sum was already formed by the producing GEMM's epilogue).
// Each warp handles kLnRowsPerWarp rows with all of their loads issued before the first reduction,
// so with 4 rows per warp a warp keeps 3 KB (H=384) in flight and the grid is 4x smaller; small
// problems use 1 row per warp so that every SM still gets CTAs.
template <int NV, int kLnRowsPerWarp>
__global__ void __launch_bounds__(kRowWarps * 32)
layernorm_kernel(const __nv_bfloat16* __restrict__ x, const float* __restrict__ gamma,
                 const float* __restrict__ beta, __nv_bfloat16* __restrict__ out, int T, float eps,
                 const int32_t* __restrict__ rows_ptr) {
    constexpr int H = NV * 128;
    pdl_launch_dependents();
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const int t0 = (blockIdx.x * kRowWarps + (threadIdx.x >> 5)) * kLnRowsPerWarp;
    int rows = T;
    if (rows_ptr != nullptr) rows = min(rows, __ldg(rows_ptr));   // rows_ptr: packed row count
    if (t0 >= rows) return;
    uint2 raw[kLnRowsPerWarp][NV];
#pragma unroll
    for (int r = 0; r < kLnRowsPerWarp; ++r) {
        const int t = min(t0 + r, rows - 1);   // clamp: tail rows are loaded twice, stored once
        const __nv_bfloat16* row = x + (size_t)t * H;
#pragma unroll
        for (int i = 0; i < NV; ++i) raw[r][i] = __ldg(reinterpret_cast<const uint2*>(row + (i * 32 + lane) * 4));
    }
    LnAffine<NV> af;
    if (kLnRowsPerWarp > 1) af.load(gamma, beta, lane);   // once per warp instead of once per row
#pragma unroll
    for (int r = 0; r < kLnRowsPerWarp; ++r) {
        if (t0 + r >= rows) break;
        float v[NV * 4];
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            v[i * 4 + 0] = bf16lo(raw[r][i].x);
            v[i * 4 + 1] = bf16hi(raw[r][i].x);
            v[i * 4 + 2] = bf16lo(raw[r][i].y);
            v[i * 4 + 3] = bf16hi(raw[r][i].y);
        }
        if (kLnRowsPerWarp > 1) ln_normalise_store<NV>(v, af, eps, lane, out + (size_t)(t0 + r) * H);
        else ln_normalise_store<NV>(v, gamma, beta, eps, lane, out + (size_t)(t0 + r) * H);
    }
}

// Masked mean-pool + L2 normalisation.  One CTA per sequence.  Thread (g, c) owns the 8-column
// vector c of the row and walks rows g, g+G, ... skipping rows with mask 0; the G partial sums per
// column vector are combined through shared memory in a fixed order (no atomics: deterministic).
constexpr int kPoolThreads = 384;

__global__ void __launch_bounds__(kPoolThreads)
pool_l2norm_kernel(const __nv_bfloat16* __restrict__ x, const int32_t* __restrict__ mask,
                   float* __restrict__ out, int S, int H, const int32_t* __restrict__ seq_start,
                   const int32_t* __restrict__ seq_len) {
    extern __shared__ float pool_smem[];  // [G][H] partial sums, then [kPoolThreads/32] reductions
    pdl_launch_dependents();
    pdl_wait();
    const int b = blockIdx.x;
    const int vecs = H / 8;               // 16-byte vectors per row
    const int G = kPoolThreads / vecs;    // row groups (>= 1 since H <= 1024 -> vecs <= 128)
    const int g = threadIdx.x / vecs, c = threadIdx.x % vecs;
    // packed mode (seq_start != nullptr): the sequence's rows are contiguous and all valid
    const bool packed = seq_start != nullptr;
    const __nv_bfloat16* xb = x + (packed ? (size_t)__ldg(seq_start + b) : (size_t)b * S) * H;
    const int32_t* mb = mask + (size_t)b * S;
    const int nrows = packed ? __ldg(seq_len + b) : S;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    int count = 0;
    if (g < G) {
        auto add_row = [&](const uint4& a) {
            acc[0] += bf16lo(a.x); acc[1] += bf16hi(a.x);
            acc[2] += bf16lo(a.y); acc[3] += bf16hi(a.y);
            acc[4] += bf16lo(a.z); acc[5] += bf16hi(a.z);
            acc[6] += bf16lo(a.w); acc[7] += bf16hi(a.w);
        };
        if (packed) {
            // all rows valid: eight, then four, independent 16-byte loads in flight per thread
            int s = g;
            for (; s + 7 * G < nrows; s += 8 * G) {
                uint4 a[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) a[u] = __ldg(reinterpret_cast<const uint4*>(xb + (size_t)(s + u * G) * H + c * 8));
#pragma unroll
                for (int u = 0; u < 8; ++u) add_row(a[u]);
                count += 8;
            }
            for (; s + 3 * G < nrows; s += 4 * G) {
                uint4 a[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) a[u] = __ldg(reinterpret_cast<const uint4*>(xb + (size_t)(s + u * G) * H + c * 8));
#pragma unroll
                for (int u = 0; u < 4; ++u) add_row(a[u]);
                count += 4;
            }
            for (; s < nrows; s += G) {
                add_row(__ldg(reinterpret_cast<const uint4*>(xb + (size_t)s * H + c * 8)));
                ++count;
            }
        } else {
            for (int s = g; s < nrows; s += G) {
                if (__ldg(mb + s) == 0) continue;
                ++count;
                add_row(__ldg(reinterpret_cast<const uint4*>(xb + (size_t)s * H + c * 8)));
            }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) pool_smem[g * H + c * 8 + i] = acc[i];
    }
    // number of pooled rows: every group counted its own (integer sums: any order gives the same value)
    __shared__ int s_count[kPoolThreads / 32];
    {
        int cnt = (g < G && c == 0) ? count : 0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
        if ((threadIdx.x & 31) == 0) s_count[threadIdx.x >> 5] = cnt;
    }
    __syncthreads();
    // column sums: thread j < H owns column j
    int n_rows = 0;
#pragma unroll
    for (int i = 0; i < kPoolThreads / 32; ++i) n_rows += s_count[i];
    const float n_valid = (float)n_rows;
    float colsum[3] = {0.f, 0.f, 0.f};  // H <= 1024 -> at most ceil(1024/384) = 3 columns per thread
    float sq = 0.f;
    const float inv_n = 1.0f / fmaxf(n_valid, 1e-9f);
#pragma unroll
    for (int r = 0; r < 3; ++r) {
        const int j = threadIdx.x + r * kPoolThreads;
        if (j < H) {
            float t = 0.f;
            for (int gg = 0; gg < G; ++gg) t += pool_smem[gg * H + j];
            t *= inv_n;
            colsum[r] = t;
            sq += t * t;
        }
    }
    __syncthreads();
    float* red = pool_smem;  // reuse
    sq = warp_sum(sq);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = sq;
    __syncthreads();
    float tot = 0.f;
    for (int i = 0; i < kPoolThreads / 32; ++i) tot += red[i];
    const float inv_norm = 1.0f / fmaxf(sqrtf(tot), 1e-12f);
#pragma unroll
    for (int r = 0; r < 3; ++r) {
        const int j = threadIdx.x + r * kPoolThreads;
        if (j < H) out[(size_t)b * H + j] = colsum[r] * inv_norm;
    }
}

// ----------------------------------------------------------------------------------------------
// LayerNorm folding (post-LN encoders without LayerNorm kernels).
//
// LN(y) W^T + b = rstd * (y (gamma o W)^T - mu * c) + d  with  c_n = sum_k gamma_k W_nk,
// d_n = sum_k beta_k W_nk + b_n: the GEMM that consumes a LayerNorm output can run on the RAW
// activation y with gamma-scaled weights and fix the result up per row in its epilogue.  This kernel
// prepares W' = bf16(gamma o W) (c is summed over the ROUNDED W', so the identity holds exactly for the
// weights the tensor cores see), c and d for a list of matrices in one launch: one warp per output row.
constexpr int kFoldMaxJobs = 24;
constexpr int kFoldWarps = 8;
struct FoldList {
    const __nv_bfloat16* w[kFoldMaxJobs];
    const float* gamma[kFoldMaxJobs];
    const float* beta[kFoldMaxJobs];
    const float* bias[kFoldMaxJobs];
    __nv_bfloat16* wf[kFoldMaxJobs];
    float* c[kFoldMaxJobs];
    float* d[kFoldMaxJobs];
    int first_row[kFoldMaxJobs + 1];   // prefix sums of the jobs' row counts
    int n;
    int K;                              // row length (the LayerNorm width), K % 256 == 0 not required: K % 8 == 0
};

__global__ void __launch_bounds__(kFoldWarps * 32)
ln_fold_weights_kernel(const __grid_constant__ FoldList fl) {
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * kFoldWarps + (threadIdx.x >> 5);
    if (row >= fl.first_row[fl.n]) return;
    int j = 0;
    while (row >= fl.first_row[j + 1]) ++j;
    const int n = row - fl.first_row[j];
    const int K = fl.K;
    const __nv_bfloat16* wr = fl.w[j] + (size_t)n * K;
    __nv_bfloat16* wo = fl.wf[j] + (size_t)n * K;
    float cs = 0.f, ds = 0.f;
    for (int k = lane * 8; k < K; k += 256) {
        const uint4 q = __ldg(reinterpret_cast<const uint4*>(wr + k));
        const float4 g0 = __ldg(reinterpret_cast<const float4*>(fl.gamma[j] + k)), g1 = __ldg(reinterpret_cast<const float4*>(fl.gamma[j] + k) + 1);
        const float4 b0 = __ldg(reinterpret_cast<const float4*>(fl.beta[j] + k)), b1 = __ldg(reinterpret_cast<const float4*>(fl.beta[j] + k) + 1);
        const float wv[8] = {bf16lo(q.x), bf16hi(q.x), bf16lo(q.y), bf16hi(q.y), bf16lo(q.z), bf16hi(q.z), bf16lo(q.w), bf16hi(q.w)};
        const float gv[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
        const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
        uint32_t o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            o[i] = pack_bf16(wv[2 * i] * gv[2 * i], wv[2 * i + 1] * gv[2 * i + 1]);
            cs += bf16lo(o[i]) + bf16hi(o[i]);
            ds = fmaf(bv[2 * i], wv[2 * i], fmaf(bv[2 * i + 1], wv[2 * i + 1], ds));
        }
        *reinterpret_cast<uint4*>(wo + k) = make_uint4(o[0], o[1], o[2], o[3]);
    }
    cs = warp_sum(cs);
    ds = warp_sum(ds);
    if (lane == 0) {
        fl.c[j][n] = cs;
        fl.d[j][n] = ds + __ldg(fl.bias[j] + n);
    }
}

// Masked mean-pool + L2 normalisation of LN(z), z being the RAW last activation and its row statistics
// arriving as per-32-column partials (the form the folding GEMM epilogues write).  One CTA per
// sequence: first every row's (rstd, -rstd*mu) goes to shared memory, then thread (g, c) accumulates
// z * rstd over its rows for its 8 columns; sum_r LN(z)_rc = gamma_c * (sum_r z_rc rstd_r + sum_r b_r)
// + n * beta_c.  Fixed-order reductions (deterministic).
constexpr int kPoolMaxRows = 512;
__global__ void __launch_bounds__(kPoolThreads)
pool_ln_l2norm_kernel(const __nv_bfloat16* __restrict__ z, const int32_t* __restrict__ mask, float* __restrict__ out, int S,
                      int H, const int32_t* __restrict__ seq_start, const int32_t* __restrict__ seq_len,
                      const float2* __restrict__ stats, int P, const float* __restrict__ gamma,
                      const float* __restrict__ beta, float eps) {
    extern __shared__ float pool_smem[];   // [G][H] partial sums
    __shared__ float s_a[kPoolMaxRows], s_b[kPoolThreads / 32];
    __shared__ float s_red[kPoolThreads / 32];
    __shared__ int s_cnt[kPoolThreads / 32];
    pdl_launch_dependents();
    pdl_wait();
    const int b = blockIdx.x;
    const int vecs = H / 8, G = kPoolThreads / vecs;
    const int g = threadIdx.x / vecs, c = threadIdx.x % vecs;
    const bool packed = seq_start != nullptr;
    const size_t row0 = packed ? (size_t)__ldg(seq_start + b) : (size_t)b * S;
    const int nrows = packed ? __ldg(seq_len + b) : S;
    const int32_t* mb = mask + (size_t)b * S;
    // phase 0: row statistics -> (a, b) per row; a = 0 marks a row that is not pooled
    float bsum = 0.f;
    int cnt = 0;
    for (int r = threadIdx.x; r < nrows; r += kPoolThreads) {
        float a = 0.f, bb = 0.f;
        if (packed || __ldg(mb + r) != 0) {
            float mu, rstd;
            // inline Chan combination of the row's partials
            const float2* sp = stats + (row0 + r) * (size_t)P;
            float sm = 0.f;
            for (int i = 0; i < P; ++i) sm += __ldg(&sp[i]).x;
            mu = sm / (float)P;
            float m2 = 0.f;
            for (int i = 0; i < P; ++i) {
                const float2 q = __ldg(&sp[i]);
                const float dl = q.x - mu;
                m2 += q.y + 32.f * dl * dl;
            }
            rstd = 1.0f / sqrtf(m2 / (32.f * (float)P) + eps);
            a = rstd;
            bb = -rstd * mu;
            ++cnt;
        }
        s_a[r] = a;
        bsum += bb;
    }
    // sum of the b terms and the row count: warp butterflies, then the warps' values in index order
    // (a fixed order, so every thread and every run gets the same bits)
    {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
            bsum += __shfl_xor_sync(0xffffffffu, bsum, o);
        }
        if ((threadIdx.x & 31) == 0) {
            s_cnt[threadIdx.x >> 5] = cnt;
            s_b[threadIdx.x >> 5] = bsum;
        }
    }
    __syncthreads();
    bsum = 0.f;
#pragma unroll
    for (int i = 0; i < kPoolThreads / 32; ++i) bsum += s_b[i];
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (g < G) {
        const __nv_bfloat16* zb = z + row0 * H + c * 8;
        for (int r = g; r < nrows; r += G) {
            const float a = s_a[r];
            if (a == 0.f) continue;
            const uint4 q = __ldg(reinterpret_cast<const uint4*>(zb + (size_t)r * H));
            acc[0] = fmaf(bf16lo(q.x), a, acc[0]); acc[1] = fmaf(bf16hi(q.x), a, acc[1]);
            acc[2] = fmaf(bf16lo(q.y), a, acc[2]); acc[3] = fmaf(bf16hi(q.y), a, acc[3]);
            acc[4] = fmaf(bf16lo(q.z), a, acc[4]); acc[5] = fmaf(bf16hi(q.z), a, acc[5]);
            acc[6] = fmaf(bf16lo(q.w), a, acc[6]); acc[7] = fmaf(bf16hi(q.w), a, acc[7]);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) pool_smem[g * H + c * 8 + i] = acc[i];
    }
    __syncthreads();
    int n_rows = 0;
#pragma unroll
    for (int i = 0; i < kPoolThreads / 32; ++i) n_rows += s_cnt[i];
    const float n_valid = (float)n_rows;
    const float inv_n = 1.0f / fmaxf(n_valid, 1e-9f);
    float colsum[3] = {0.f, 0.f, 0.f};
    float sq = 0.f;
#pragma unroll
    for (int rr = 0; rr < 3; ++rr) {
        const int j = threadIdx.x + rr * kPoolThreads;
        if (j < H) {
            float t = 0.f;
            for (int gg = 0; gg < G; ++gg) t += pool_smem[gg * H + j];
            t = (__ldg(gamma + j) * (t + bsum) + n_valid * __ldg(beta + j)) * inv_n;
            colsum[rr] = t;
            sq += t * t;
        }
    }
    sq = warp_sum(sq);
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = sq;
    __syncthreads();
    float tot = 0.f;
    for (int i = 0; i < kPoolThreads / 32; ++i) tot += s_red[i];
    const float inv_norm = 1.0f / fmaxf(sqrtf(tot), 1e-12f);
#pragma unroll
    for (int rr = 0; rr < 3; ++rr) {
        const int j = threadIdx.x + rr * kPoolThreads;
        if (j < H) out[(size_t)b * H + j] = colsum[rr] * inv_norm;
    }
}

}  // namespace rlx
