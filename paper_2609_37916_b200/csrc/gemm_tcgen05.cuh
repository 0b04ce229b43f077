// bf16 "Linear" GEMM for sm_100a: out[M,N] = epilogue(A[M,K] * W[N,K]^T + bias).
//
// Structure (one persistent CTA per SM, 320 to 576 threads):
//   warp 0      TMA producer: streams 128x64 A tiles and BLOCK_N x 64 W tiles (128-byte swizzle)
//               through a STAGES-deep shared-memory ring guarded by full/empty mbarriers; a stage
//               holds one or two 64-wide k-blocks behind one barrier pair
//   warp 1      allocates tensor memory; one elected lane issues tcgen05.mma (M=128, N=BLOCK_N,
//               K=16 per instruction) into one of two fp32 accumulator buffers in TMEM and
//               commits stage releases / accumulator-ready signals to mbarriers
//               (both warps run their loops warp-uniformly; elect.sync picks the issuing lane)
//   warps 2..   epilogue (8 to 16 warps): each warp owns one TMEM lane quadrant (32 rows) and one 64-column
//               slab of the tile; it tcgen05.ld's its slab into registers and hands the accumulator back
//               at once, then per 32-column chunk adds bias, applies GELU or adds the residual in fp32,
//               rounds to bf16, writes the chunk into its swizzled staging buffer and issues a TMA store
//               for it (which drains while the next chunk is computed).
//               The second accumulator buffer lets tile i's epilogue overlap tile i+1's main loop.
// Epilogue modes (template EPI): 0 bias; 1 bias + GELU; 2 bias + residual; and the LayerNorm-folding
// modes that let a post-LN encoder drop its LayerNorm kernels:
//   3 / 4  the A operand is a RAW pre-LayerNorm activation y and W was pre-multiplied by gamma:
//          out = rstd_m * (acc - mu_m * c_n) + d_n  (then GELU for 4), with c_n = sum_k W'[n,k],
//          d_n = sum_k beta_k W[n,k] + bias_n, and (mu_m, rstd_m) rebuilt per row from per-32-column
//          partial (mean, M2) pairs written by the GEMM that produced y  ==  LN(y) W^T + bias;
//   5      bias + residual (already normalised), and the partial statistics of the result are written;
//   6      bias + LN(raw residual) rebuilt on the fly from the residual's partial statistics, gamma
//          and beta, and the partial statistics of the result are written.
// Two instantiations per tile shape: CG = 1 (one CTA per 128 x BLOCK_N tile) and CG = 2, where a
// cluster of two CTAs on neighbouring SMs computes a 256 x BLOCK_N tile with tcgen05.mma.cta_group::2:
// each CTA loads its own 128 rows of A and only HALF of the W tile, the leader CTA issues the MMAs
// for both, and each CTA finds its 128 accumulator rows in its own TMEM.  This halves the W bytes
// every SM has to pull from L2 (the operand feed, not the tensor pipe, is what limits these GEMMs)
// without any multicast load.  Completion is signalled to both CTAs with a multicast tcgen05.commit.
// Every mbarrier wait is bounded by a wall-clock budget; on expiry the CTA raises an abort flag,
// records RLX_DEVSTAT_TIMEOUT, drains, frees its tensor memory and returns.
#pragma once
#include <cuda.h>
#include "common.cuh"
#include "epilogue.cuh"

namespace rlx {
namespace tc {

constexpr int BLOCK_M = 128;
constexpr int BLOCK_K = 64;   // 64 bf16 = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;
constexpr int kStageBufBytes = 32 * 32 * 2;          // one 32-row x 32-column bf16 chunk
constexpr uint64_t kWaitBudgetNs = 2000000000ull;  // 2 s per wait

template <int BLOCK_N, int CG = 1>
struct Cfg {
    static constexpr int A_BYTES = BLOCK_M * BLOCK_K * 2;
    static constexpr int B_ROWS = BLOCK_N / CG;                  // W rows this CTA loads per k-block
    static constexpr int B_BYTES = B_ROWS * BLOCK_K * 2;
    static constexpr int KB_BYTES = A_BYTES + B_BYTES;           // operands of one 64-wide k-block
    // epilogue: EPI_SPLIT warps share each 32-row TMEM quadrant, each taking a 64-column slab (32 for the
    // narrowest tile): at most 64 accumulator registers per thread leave the compiler room to interleave
    // many independent GELU evaluations (with 128 of them live the special-function and FP32 pipes idled
    // on dependent chains), and four warps per scheduler hide what is left.  One staging buffer per warp:
    // the TMA store of a chunk drains while the next chunk is being computed.
    static constexpr int EPI_SPLIT = BLOCK_N >= 128 ? BLOCK_N / 64 : 2;
    static constexpr int EPI_WARPS = 4 * EPI_SPLIT;
    static constexpr int THREADS = 64 + 32 * EPI_WARPS;
    static constexpr int SLAB = BLOCK_N / EPI_SPLIT;
    static constexpr int STAGING_BYTES = EPI_WARPS * kStageBufBytes;
    static constexpr int BAR_BYTES = 256;
    static constexpr int RING_BUDGET = 227 * 1024 - 1024 - BAR_BYTES - STAGING_BYTES;
    // A stage holds KPS k-blocks behind ONE full / empty barrier pair.  A barrier round costs the issuing
    // thread a couple of hundred cycles whether or not the barrier is already complete (measured: 4 MMAs
    // + wait + commit take ~430 cycles of the thread, 8 MMAs ~620), so with one k-block per round the
    // single MMA thread, not the tensor pipe, paces every tile narrower than 256 columns (384 tensor
    // cycles per k-block at N = 192).  Such tiles take two k-blocks per stage when four stages still
    // fit; 256-wide tiles (512 tensor cycles per k-block) keep one, which buys ring depth: what the
    // ring can hide is (STAGES - 1) stages of tensor time, and the operands come from L2 or HBM.
#ifndef RLX_KPS_MIN_STAGES
#define RLX_KPS_MIN_STAGES 4
#endif
#ifndef RLX_KPS_MAX_BN
#define RLX_KPS_MAX_BN 192
#endif
    static constexpr int KPS = (BLOCK_N <= RLX_KPS_MAX_BN && RLX_KPS_MIN_STAGES * 2 * KB_BYTES <= RING_BUDGET) ? 2 : 1;
    static constexpr int STAGE_BYTES = KPS * KB_BYTES;
    static constexpr int STAGES = (RING_BUDGET / STAGE_BYTES) > 8 ? 8 : (RING_BUDGET / STAGE_BYTES);
    static constexpr int TMEM_COLS = (2 * BLOCK_N <= 32) ? 32 : (2 * BLOCK_N <= 64) ? 64 : (2 * BLOCK_N <= 128) ? 128
                                     : (2 * BLOCK_N <= 256) ? 256 : 512;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + STAGING_BYTES + BAR_BYTES + 1024;  // +1024: manual alignment
    static_assert(BLOCK_N % 16 == 0 && BLOCK_N >= 16 && BLOCK_N <= 256, "UMMA N for M=128 / M=256");
    static_assert(CG == 1 || CG == 2, "cta_group");
    static_assert(B_BYTES % 1024 == 0, "stage tiles must stay 1024-byte aligned");
    static_assert(STAGES >= 2, "ring too shallow");
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory");
    static_assert(16 * STAGES + 48 <= BAR_BYTES, "barrier block");
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Non-blocking probe (try_wait may suspend the thread for a while; this one never does): issued early,
// its result is consumed after independent work, which hides the round trip to the barrier.
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when the budget ran out or another role already aborted.
__device__ __forceinline__ bool mbar_wait_budget(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint64_t budget_ns) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 0xff) == 0) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > budget_ns) {
                *abort_flag = 1;
                return false;
            }
        }
    }
    return true;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    return mbar_wait_budget(bar, parity, abort_flag, kWaitBudgetNs);
}
// The same wait executed by all 32 lanes of a converged warp, with one outcome for the whole warp
// (a lane that gave up takes the others with it), so that the warp stays converged afterwards.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    return __all_sync(0xffffffffu, mbar_wait_budget(bar, parity, abort_flag, kWaitBudgetNs)) != 0;
}

// Self-test of the bounded wait: one thread waits, with a caller-chosen budget, on an mbarrier that
// nothing ever arrives on; the wait must give up, raise the abort flag and leave the time-out bit in the
// status word exactly as the GEMM / attention pipelines do when a wait of theirs expires.
__global__ void bounded_wait_selftest_kernel(int32_t* status, unsigned long long budget_ns, unsigned long long* waited_ns) {
    __shared__ __align__(8) unsigned long long bar_storage;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        const uint32_t bar = smem_u32(&bar_storage);
        abort_flag = 0;
        mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const uint64_t t0 = global_timer_ns();
        const bool ok = mbar_wait_budget(bar, 0, &abort_flag, budget_ns);
        const uint64_t t1 = global_timer_ns();
        if (waited_ns) *waited_ns = t1 - t0;
        if (!ok && abort_flag) atomicOr(status, RLX_DEVSTAT_TIMEOUT_BIT);
    }
}
// ---- cluster helpers (CG = 2) ----
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cluster address of `smem_addr` (a shared::cta address) in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Arrivals that publish no memory writes of the arriving thread (handing a TMEM accumulator back after
// tcgen05.wait::ld: the data is in registers, the tcgen05 fence orders the tensor-memory reads).  A
// release-arrive would first wait for every earlier global store of the thread to become visible at
// the barrier's scope -- at cluster scope that held the accumulator for thousands of cycles.
__device__ __forceinline__ void mbar_arrive_relaxed(uint32_t bar) {
    asm volatile("mbarrier.arrive.relaxed.cta.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster_relaxed(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Arrival on another CTA's barrier that publishes only shared-memory stores of the arriving warp which a
// fence.proxy.async has already made visible to the async proxy (an operand tile written from registers
// for the tensor core of this same SM).  Release at CTA scope: the cluster-scope form also waits for the
// thread's global traffic and costs over a thousand cycles per arrival.
__device__ __forceinline__ void mbar_arrive_cluster_release_cta(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cta.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tma_load_2d(uint32_t smem_dst, const CUtensorMap* tmap, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(bar) : "memory");
}
// TMA store of one staged chunk (shared -> global), tracked by the issuing thread's bulk async-group
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tmap, int x, int y, uint32_t smem_src) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(smem_src) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait() { asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ uint4 ld_shared_v4(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
// Global accesses of the epilogue with L1 policies: the streamed output rows must not push the few
// lines every warp re-reads (bias, gamma, beta) out of the small L1 that is left next to ~220 KB of
// shared memory.  (Residual rows keep the default policy: a thread reads its 64-byte piece with four
// 16-byte loads, and only L1 allocation keeps the last three from going back to L2.)
__device__ __forceinline__ void st_global_stream_v4(void* ptr, uint4 v) {
    asm volatile("st.global.L1::no_allocate.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(ptr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ float4 ld_global_keep_f4(const float* ptr) {
    float4 v;   // not volatile: a read of read-only data, free to be scheduled early and together with its neighbours
    asm("ld.global.nc.L1::evict_last.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(ptr));
    return v;
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint4 v) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
// 3-D forms: operand viewed as [k-block][row][64 columns]; the box covers several k-blocks, which land
// one after the other as complete 128-byte-swizzled tiles
__device__ __forceinline__ void tma_load_3d(uint32_t smem_dst, const CUtensorMap* tmap, int x, int y, int z, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(smem_dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_3d_cg2(uint32_t smem_dst, const CUtensorMap* tmap, int x, int y, int z, uint32_t bar_cluster) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(smem_dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(z), "r"(bar_cluster) : "memory");
}
// CG = 2 form: the mbarrier may live in the peer CTA (cluster address); the data lands in this CTA
__device__ __forceinline__ void tma_load_2d_cg2(uint32_t smem_dst, const CUtensorMap* tmap, int x, int y, uint32_t bar_cluster) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(bar_cluster) : "memory");
}
// L2 prefetch of one box of a tiled tensor (no shared-memory destination, no barrier)
__device__ __forceinline__ void tma_prefetch_2d(const CUtensorMap* tmap, int x, int y) {
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global [%0, {%1, %2}];"
                 ::"l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_prefetch_3d(const CUtensorMap* tmap, int x, int y, int z) {
    asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global [%0, {%1, %2, %3}];"
                 ::"l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(z) : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* tmap) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(tmap)) : "memory");
}
template <int CG>
__device__ __forceinline__ void tmem_alloc(uint32_t smem_slot, uint32_t ncols) {
    if constexpr (CG == 1)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_slot), "r"(ncols) : "memory");
    else
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_slot), "r"(ncols) : "memory");
}
template <int CG>
__device__ __forceinline__ void tmem_relinquish() {
    if constexpr (CG == 1)
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    else
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
template <int CG>
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    if constexpr (CG == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
    else
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// True in exactly one lane of a fully converged warp.  The producer and MMA warps run their loops with
// all 32 lanes (warp-uniform control flow and addresses) and let the elected lane issue the TMA /
// tcgen05 instructions: measured on the MMA loop, a loop executed by a single lane under a divergent
// branch costs the issuing thread ~110-120 cycles per tcgen05.mma, the warp-uniform form ~80.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n"
        ".reg .pred P;\n"
        "elect.sync _|P, 0xFFFFFFFF;\n"
        "selp.u32 %0, 1, 0, P;\n"
        "}\n"
        : "=r"(pred));
    return pred != 0;
}
template <int CG>
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    if constexpr (CG == 1)
        asm volatile(
            "{\n"
            ".reg .pred p;\n"
            "setp.ne.b32 p, %4, 0;\n"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
            "}\n" ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
    else
        asm volatile(
            "{\n"
            ".reg .pred p;\n"
            "setp.ne.b32 p, %4, 0;\n"
            "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n"
            "}\n" ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// mbarrier arrives once all tcgen05.mma issued so far by this thread have completed.  CG = 2: the
// arrive is multicast to the barrier at the same offset in both CTAs of the pair.
template <int CG>
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    if constexpr (CG == 1) {
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
    } else {
        const uint16_t mask = 3;
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                     ::"r"(bar), "h"(mask) : "memory");
    }
}
// 32 lanes x 32 consecutive 32-bit columns -> 32 registers per thread (thread = lane = row)
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major tile of 128-byte rows written by TMA with the 128-byte
// swizzle; 8-row groups are 1024 bytes apart (stride byte offset); the leading byte offset is not
// used by swizzled K-major layouts (encoded 1); descriptor version 1; swizzle mode 2 = 128 B.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptor for kind::f16: fp32 accumulate, bf16 A and B, both K-major, M x N tile.
__host__ __device__ constexpr uint32_t make_idesc(int m, int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

struct Params {
    const float* bias;               // [N]
    const __nv_bfloat16* residual;   // [M,N] or null
    __nv_bfloat16* out;              // [M,N]
    int M, N, K;
    int32_t* status;                 // device status word (may be null)
    const int32_t* m_ptr;            // optional device row count: rows >= *m_ptr are not computed
    int kblock_maps;                 // the operand tensor maps are 3-D views [K/64][rows][64]: one TMA load brings a
                                     // whole stage's k-blocks of an operand (needs K % 64 == 0); else 2-D, one per k-block
#ifdef RLX_EXPERIMENTS
    int debug;                       // ablation switches of the experiments build (kDbg* bits)
    unsigned long long* trace;       // experiments build: 64 timestamp slots per CTA (or null)
#endif
    // LayerNorm folding (EPI 3..6); unused fields stay null
    const float* cvec;               // [N] EPI 3/4: column sums of the gamma-scaled weights
    const float* dvec;               // [N] EPI 3/4: beta . W + bias
    const float2* stats_in;          // [M, stats_in_p] partial (mean, M2) per 32 columns: of A's rows (3/4) or the residual's (6)
    int stats_in_p;
    const float* ln_gamma;           // [N] EPI 6
    const float* ln_beta;            // [N] EPI 6
    float2* stats_out;               // [M, N/32] EPI 5/6
    float ln_eps;
};

// (mu, rstd) of one row from its per-32-column partials (equal counts: Chan's combination)
// One pass over 16-byte loads (two partials each, all in flight together): sum of the means, of the M2
// terms and of the squared means; the between-chunk part  32 * (sum mean_i^2 - P mu^2)  is a difference
// of small numbers of one sign-definite kind (clamped at zero), accurate unless |mu| exceeds the row's
// standard deviation by three orders of magnitude.
__device__ __forceinline__ void row_stats_from_partials(const float2* __restrict__ sp, int P, float eps, float& mu, float& rstd) {
    float sm = 0.f, sq = 0.f, m2 = 0.f;
    const float4* sp4 = reinterpret_cast<const float4*>(sp);
    for (int i = 0; i < P / 2; ++i) {
        const float4 q = __ldg(sp4 + i);
        sm += q.x + q.z;
        sq = fmaf(q.x, q.x, fmaf(q.z, q.z, sq));
        m2 += q.y + q.w;
    }
    if (P & 1) {
        const float2 q = __ldg(sp + P - 1);
        sm += q.x;
        sq = fmaf(q.x, q.x, sq);
        m2 += q.y;
    }
    mu = sm / (float)P;
    const float between = fmaxf(sq - (float)P * mu * mu, 0.f);
    rstd = 1.0f / sqrtf((m2 + 32.f * between) / (32.f * (float)P) + eps);
}

#ifdef RLX_EXPERIMENTS
constexpr int kDbgNoEpilogue = 1;   // epilogue warps hand the accumulator back without reading it
constexpr int kDbgNoStore = 2;      // everything but the global stores
constexpr int kDbgNoMma = 4;        // the MMA thread only commits (operand feed alone)
constexpr int kDbgNoLoad = 8;       // the producer only arrives (tensor pipe alone)
#define RLX_DBG(p, bit) (((p).debug & (bit)) != 0)
#define RLX_TRACE(p, slot) do { if ((p).trace) (p).trace[blockIdx.x * 64 + (slot)] = global_timer_ns(); } while (0)
#define RLX_TRACE_CLK(p, slot) do { if ((p).trace) (p).trace[blockIdx.x * 64 + (slot)] = (unsigned long long)clock64(); } while (0)
#define RLX_CLK_DECL(name) long long name = 0
#define RLX_CLK_ADD(name, expr) do { const long long _c0 = clock64(); expr; name += clock64() - _c0; } while (0)
#define RLX_TRACE_VAL(p, slot, v) do { if ((p).trace) (p).trace[blockIdx.x * 64 + (slot)] = (unsigned long long)(v); } while (0)
#else
#define RLX_DBG(p, bit) false
#define RLX_TRACE(p, slot) do { } while (0)
#define RLX_TRACE_CLK(p, slot) do { } while (0)
#define RLX_CLK_DECL(name) do { } while (0)
#define RLX_CLK_ADD(name, expr) do { expr; } while (0)
#define RLX_TRACE_VAL(p, slot, v) do { } while (0)
#endif

// One epilogue warp's share of one output tile: 32 rows (a TMEM lane quadrant, thread = row) x NC
// chunks of 32 columns.  prefetch() issues the loads that do not depend on the accumulator (residual
// rows, LayerNorm row statistics) so that their latency hides behind the main loop; drain() reads the
// warp's accumulator slab into registers, hands the buffer back to the MMA thread, then chunk by chunk
// applies the epilogue in fp32, rounds to bf16, writes the chunk into the warp's swizzled staging
// buffer (thread = row, 64 bytes) and lets one lane hand it to the TMA engine as a 32 x 32
// box.  The load/store pipe of the SM is what the epilogue runs out of first (reading the accumulator
// and the bias already costs 64 shared-pipe wavefronts per chunk), so the stores do not go through it:
// TMA reads the staged tile itself and writes whole lines.  Rows at or beyond the matrix's row count
// are clipped by the tensor map; rows between a smaller device-side row count (packed batches) and the
// end of the last tile are written with values nobody reads.
template <int EPI, int NC>
struct EpilogueTile {
    static constexpr bool kRes = EPI == 2 || EPI == 5 || EPI == 6;     // a residual tile is added
    static constexpr bool kFold = EPI == 3 || EPI == 4;                // LayerNorm folded into this GEMM's input
    static constexpr bool kStatsIn = kFold || EPI == 6;
    static constexpr bool kStatsOut = EPI == 5 || EPI == 6;
    uint4 res[kRes ? NC : 1][4];
    float ln_a = 1.f, ln_b = 0.f;   // x_norm = x * ln_a + ln_b  (ln_a = rstd, ln_b = -rstd * mu)

    // The bias values of a slab (one 128-byte line per chunk) are pulled into L1 a tile ahead of their
    // use by every lane, so that no chunk starts with an L2 round trip.
    static __device__ __forceinline__ void prefetch_bias(const Params& p, int n0) {
        if (p.bias != nullptr && (threadIdx.x & 31) < NC) asm volatile("prefetch.global.L1 [%0];" ::"l"(p.bias + n0 + (threadIdx.x & 31) * 32));
    }

    __device__ __forceinline__ void prefetch(const Params& p, int M, int m, int n0) {
        if (kRes && m < M) {
            const __nv_bfloat16* rpre = p.residual + (size_t)m * p.N + n0;
#pragma unroll
            for (int c = 0; c < NC; ++c)
#pragma unroll
                for (int i = 0; i < 4; ++i) res[c][i] = __ldg(reinterpret_cast<const uint4*>(rpre + c * 32) + i);
        }
        if (kStatsIn && m < M) {
            float mu, rstd;
            row_stats_from_partials(p.stats_in + (size_t)m * p.stats_in_p, p.stats_in_p, p.ln_eps, mu, rstd);
            ln_a = rstd;
            ln_b = -rstd * mu;
        }
    }

    template <int CG>
    __device__ __forceinline__ void release(uint32_t tempty, uint32_t cta_rank, int lane) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
            if (CG == 1) mbar_arrive_relaxed(tempty);
            else mbar_arrive_cluster_relaxed(map_to_cta(tempty, 0));   // the leader's barrier collects both CTAs' warps
        }
    }

    template <int CG>
    __device__ __forceinline__ void drain(const Params& p, const CUtensorMap* tmap_out, int M, int m_row0, int n0,
                                          uint32_t taddr, uint32_t stg, int lane, uint32_t tempty, uint32_t cta_rank,
                                          int trace_slot = -1) {
        const int m = m_row0 + lane;
        const bool row_ok = m < M;
        const uint32_t row_off = lane * 64;                 // 64-byte rows in the staging chunk
        const uint32_t swz = (uint32_t)((lane >> 1) & 3);   // 64-byte swizzle: 16-byte chunk index ^ (row/2 % 4)
        const float* brow = p.bias + n0;
        if (RLX_DBG(p, kDbgNoEpilogue)) {
            release<CG>(tempty, cta_rank, lane);
            return;
        }
        if (trace_slot >= 0) RLX_TRACE_CLK(p, 56 + (trace_slot - 40) / 8);
        // Without a residual the warp's whole slab goes to registers first, so that the accumulator
        // buffer returns to the MMA thread after one TMEM round trip, before any of the epilogue's memory
        // traffic.  With a residual tile held in registers there is no room for that: chunks are read one
        // ahead and the accumulator goes back once the last one has landed.
        constexpr bool kAllFirst = !kRes;
        uint32_t r[kAllFirst ? NC : 2][32];
        if constexpr (kAllFirst) {
#pragma unroll
            for (int c = 0; c < NC; ++c) tmem_ld_32x32(taddr + c * 32, r[c]);
            tmem_ld_wait();
            release<CG>(tempty, cta_rank, lane);
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                if (trace_slot >= 0 && c < 2) RLX_TRACE_CLK(p, trace_slot + 4 * c);
                uint4 q[4];
                compute_chunk(p, r[c], n0 + c * 32, c, m, row_ok, brow + c * 32, q);
                if (trace_slot >= 0 && c < 2) RLX_TRACE_CLK(p, trace_slot + 4 * c + 1);
                store_chunk(p, tmap_out, q, n0 + c * 32, m_row0, stg, lane, row_off, swz);
                if (trace_slot >= 0 && c < 2) RLX_TRACE_CLK(p, trace_slot + 4 * c + 3);
            }
        } else {
            tmem_ld_32x32(taddr, r[0]);
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                tmem_ld_wait();
                if (c + 1 < NC) tmem_ld_32x32(taddr + (c + 1) * 32, r[(c + 1) & 1]);
                else release<CG>(tempty, cta_rank, lane);
                if (trace_slot >= 0 && c < 2) RLX_TRACE_CLK(p, trace_slot + 4 * c);
                uint4 q[4];
                compute_chunk(p, r[c & 1], n0 + c * 32, c, m, row_ok, brow + c * 32, q);
                if (trace_slot >= 0 && c < 2) RLX_TRACE_CLK(p, trace_slot + 4 * c + 1);
                store_chunk(p, tmap_out, q, n0 + c * 32, m_row0, stg, lane, row_off, swz);
                if (trace_slot >= 0 && c < 2) RLX_TRACE_CLK(p, trace_slot + 4 * c + 3);
            }
        }
    }

    // Epilogue arithmetic of one 32-column chunk of this thread's row: acc -> bf16 pairs (16 words).
    __device__ __forceinline__ void compute_chunk(const Params& p, const uint32_t (&acc)[32], int ncol, int c, int m,
                                                  bool row_ok, const float* bias32, uint4 (&q)[4]) {
        float v[32];
        if constexpr (kFold) {
            const float* crow = p.cvec + ncol;
            const float* drow = p.dvec + ncol;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float4 c4 = __ldg(reinterpret_cast<const float4*>(crow) + i);
                const float4 d4 = __ldg(reinterpret_cast<const float4*>(drow) + i);
                v[4 * i + 0] = fmaf(ln_a, __uint_as_float(acc[4 * i + 0]), fmaf(ln_b, c4.x, d4.x));
                v[4 * i + 1] = fmaf(ln_a, __uint_as_float(acc[4 * i + 1]), fmaf(ln_b, c4.y, d4.y));
                v[4 * i + 2] = fmaf(ln_a, __uint_as_float(acc[4 * i + 2]), fmaf(ln_b, c4.z, d4.z));
                v[4 * i + 3] = fmaf(ln_a, __uint_as_float(acc[4 * i + 3]), fmaf(ln_b, c4.w, d4.w));
            }
        } else {
            float4 b4[8];
            if (p.bias != nullptr) {   // uniform; the encoder's GEMMs always carry a bias
#pragma unroll
                for (int i = 0; i < 8; ++i) b4[i] = ld_global_keep_f4(bias32 + 4 * i);
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) b4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                v[4 * i + 0] = __uint_as_float(acc[4 * i + 0]) + b4[i].x;
                v[4 * i + 1] = __uint_as_float(acc[4 * i + 1]) + b4[i].y;
                v[4 * i + 2] = __uint_as_float(acc[4 * i + 2]) + b4[i].z;
                v[4 * i + 3] = __uint_as_float(acc[4 * i + 3]) + b4[i].w;
            }
        }
        if (EPI == 1 || EPI == 4) {
#pragma unroll
            for (int i = 0; i < 32; i += 2) gelu_erf_x2(v[i], v[i + 1]);
        }
        if ((EPI == 2 || EPI == 5) && row_ok) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint4 w = res[kRes ? c : 0][i];
                v[8 * i + 0] += bf16lo(w.x); v[8 * i + 1] += bf16hi(w.x);
                v[8 * i + 2] += bf16lo(w.y); v[8 * i + 3] += bf16hi(w.y);
                v[8 * i + 4] += bf16lo(w.z); v[8 * i + 5] += bf16hi(w.z);
                v[8 * i + 6] += bf16lo(w.w); v[8 * i + 7] += bf16hi(w.w);
            }
        }
        if (EPI == 6 && row_ok) {
            // residual = LN(raw residual row): (x * rstd - rstd * mu) * gamma_n + beta_n
            const float* grow = p.ln_gamma + ncol;
            const float* berow = p.ln_beta + ncol;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint4 w = res[kRes ? c : 0][i];
                const float4 g0 = __ldg(reinterpret_cast<const float4*>(grow) + 2 * i);
                const float4 g1 = __ldg(reinterpret_cast<const float4*>(grow) + 2 * i + 1);
                const float4 e0 = __ldg(reinterpret_cast<const float4*>(berow) + 2 * i);
                const float4 e1 = __ldg(reinterpret_cast<const float4*>(berow) + 2 * i + 1);
                v[8 * i + 0] += fmaf(fmaf(bf16lo(w.x), ln_a, ln_b), g0.x, e0.x);
                v[8 * i + 1] += fmaf(fmaf(bf16hi(w.x), ln_a, ln_b), g0.y, e0.y);
                v[8 * i + 2] += fmaf(fmaf(bf16lo(w.y), ln_a, ln_b), g0.z, e0.z);
                v[8 * i + 3] += fmaf(fmaf(bf16hi(w.y), ln_a, ln_b), g0.w, e0.w);
                v[8 * i + 4] += fmaf(fmaf(bf16lo(w.z), ln_a, ln_b), g1.x, e1.x);
                v[8 * i + 5] += fmaf(fmaf(bf16hi(w.z), ln_a, ln_b), g1.y, e1.y);
                v[8 * i + 6] += fmaf(fmaf(bf16lo(w.w), ln_a, ln_b), g1.z, e1.z);
                v[8 * i + 7] += fmaf(fmaf(bf16hi(w.w), ln_a, ln_b), g1.w, e1.w);
            }
        }
        if (kStatsOut && row_ok) {
            // partial statistics of this row's 32 results (two-pass inside the chunk)
            float sm = 0.f;
#pragma unroll
            for (int i = 0; i < 32; ++i) sm += v[i];
            const float mean = sm * (1.0f / 32.0f);
            float m2 = 0.f;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const float dl = v[i] - mean;
                m2 = fmaf(dl, dl, m2);
            }
            p.stats_out[(size_t)m * (p.N / 32) + ncol / 32] = make_float2(mean, m2);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            q[i].x = pack_bf16(v[8 * i + 0], v[8 * i + 1]);
            q[i].y = pack_bf16(v[8 * i + 2], v[8 * i + 3]);
            q[i].z = pack_bf16(v[8 * i + 4], v[8 * i + 5]);
            q[i].w = pack_bf16(v[8 * i + 6], v[8 * i + 7]);
        }
    }

    // Stage one chunk in the warp's buffer (the TMA store of the previous chunk, issued a chunk's worth
    // of arithmetic ago, must be done reading it) and hand it to the TMA engine.
    static __device__ __forceinline__ void store_chunk(const Params& p, const CUtensorMap* tmap_out, const uint4 (&q)[4],
                                                       int ncol, int m_row0, uint32_t stg, int lane, uint32_t row_off,
                                                       uint32_t swz) {
        if (lane == 0) bulk_wait_read<0>();
        __syncwarp();
#pragma unroll
        for (int i = 0; i < 4; ++i) st_shared_v4(stg + row_off + (((uint32_t)i ^ swz) << 4), q[i]);
        fence_proxy_async();   // the writes above become visible to the TMA engine
        __syncwarp();
        if (lane == 0 && !RLX_DBG(p, kDbgNoStore)) {
            tma_store_2d(tmap_out, ncol, m_row0, stg);
            bulk_commit();
        }
    }

    // Before the warp leaves the kernel: its TMA stores must have completed (they read shared memory).
    static __device__ __forceinline__ void finish(int lane) {
        if (lane == 0) bulk_wait<0>();
        __syncwarp();
    }
};

template <int BLOCK_N, int EPI, int CG>
__global__ void __launch_bounds__((Cfg<BLOCK_N, CG>::THREADS), 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                    const __grid_constant__ CUtensorMap tmap_out, const Params p) {
    using C = Cfg<BLOCK_N, CG>;
    constexpr int TILE_M = BLOCK_M * CG;   // rows of one output tile (per CTA pair when CG = 2)
    extern __shared__ unsigned char smem_raw[];
    // manual 1024-byte alignment (required by the 128-byte swizzle atoms)
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* gbase = smem_raw + (base - raw);
    const uint32_t staging = base + C::STAGES * C::STAGE_BYTES;
    const uint32_t bars = staging + C::STAGING_BYTES;
    // barrier block: full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2], tmem slot, abort flag
    const uint32_t full_bar = bars, empty_bar = bars + 8 * C::STAGES;
    const uint32_t tfull_bar = bars + 16 * C::STAGES, tempty_bar = tfull_bar + 16;
    uint32_t* tmem_slot =
        reinterpret_cast<uint32_t*>(gbase + C::STAGES * C::STAGE_BYTES + C::STAGING_BYTES + 16 * C::STAGES + 32);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta_rank = (CG == 2) ? cluster_ctarank() : 0u;   // rank 0 leads the pair
    pdl_launch_dependents();
    if (threadIdx.x == 0) RLX_TRACE(p, 0);

    if (threadIdx.x == 0) {
        for (int i = 0; i < C::STAGES; ++i) {
            mbar_init(full_bar + 8 * i, 1);
            mbar_init(empty_bar + 8 * i, 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(tfull_bar + 8 * i, 1);
            mbar_init(tempty_bar + 8 * i, C::EPI_WARPS * CG);   // the leader's barrier collects both CTAs' warps
        }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmap_a);
        prefetch_tmap(&tmap_b);
        prefetch_tmap(&tmap_out);
    }
    if (warp == 1) {
        tmem_alloc<CG>(smem_u32(tmem_slot), C::TMEM_COLS);
        tmem_relinquish<CG>();
    }
    tc_fence_before();
    __syncthreads();
    if constexpr (CG == 2) cluster_sync_all();   // the peer's barriers are initialised before any remote use
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // everything above is independent of the previous kernel; its outputs are read only from here on
    if (threadIdx.x == 0) RLX_TRACE(p, 1);
    pdl_wait();
    if (threadIdx.x == 0) RLX_TRACE(p, 2);
    int M = p.M;
    if (p.m_ptr != nullptr) M = min(M, __ldg(p.m_ptr));   // packed activations: only sum(len) rows exist
    const int n_tiles = p.N / BLOCK_N;
    const int m_tiles = (M + TILE_M - 1) / TILE_M;
    const int num_tiles = n_tiles * m_tiles;
    const int num_kb = (p.K + BLOCK_K - 1) / BLOCK_K;
    const int tile0 = blockIdx.x / CG, tile_step = gridDim.x / CG;   // both CTAs of a pair walk the same tiles

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (whole warp, one lane issues)
        {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            int pit = 0;
            for (int tile = tile0; tile < num_tiles && ok; tile += tile_step, ++pit) {
                const int m_blk = tile / n_tiles, n_blk = tile % n_tiles;
                for (int kb = 0; kb < num_kb; kb += C::KPS) {
                    const int cnt = min(C::KPS, num_kb - kb);   // k-blocks in this stage
                    if (pit == 2 && kb == 0 && lane == 0) RLX_TRACE_CLK(p, 58);   // about to wait for a free stage
                    if (!mbar_wait_warp(empty_bar + 8 * stage, phase ^ 1, abort_flag)) { ok = false; break; }
                    if (pit == 2 && kb == 0 && lane == 0) RLX_TRACE_CLK(p, 59);   // stage free: loads issued now
                    const uint32_t st0 = base + stage * C::STAGE_BYTES;   // [A k-blocks][W k-blocks]
                    const uint32_t sb0 = st0 + C::KPS * C::A_BYTES;
                    if (elect_one()) {
                        // 3-D maps: one load per operand brings all KPS k-blocks (a k-block past the end of K
                        // arrives as zeros and still counts its bytes)
                        const bool k3 = p.kblock_maps != 0;
                        const int nbytes = k3 ? C::KPS * C::KB_BYTES : cnt * C::KB_BYTES;
                        if (RLX_DBG(p, kDbgNoLoad)) {
                            if (cta_rank == 0) mbar_arrive(full_bar + 8 * stage);
                        } else if constexpr (CG == 1) {
                            mbar_expect_tx(full_bar + 8 * stage, nbytes);
                            if (k3) {
                                tma_load_3d(st0, &tmap_a, 0, m_blk * BLOCK_M, kb, full_bar + 8 * stage);
                                tma_load_3d(sb0, &tmap_b, 0, n_blk * BLOCK_N, kb, full_bar + 8 * stage);
                            } else {
                                for (int i = 0; i < cnt; ++i) {
                                    tma_load_2d(st0 + i * C::A_BYTES, &tmap_a, (kb + i) * BLOCK_K, m_blk * BLOCK_M, full_bar + 8 * stage);
                                    tma_load_2d(sb0 + i * C::B_BYTES, &tmap_b, (kb + i) * BLOCK_K, n_blk * BLOCK_N, full_bar + 8 * stage);
                                }
                            }
                        } else {
                            // both CTAs' copies complete on the LEADER's full barrier, which expects all bytes
                            const uint32_t lead_full = map_to_cta(full_bar + 8 * stage, 0);
                            if (cta_rank == 0) mbar_expect_tx(full_bar + 8 * stage, 2 * nbytes);
                            const int arow = m_blk * TILE_M + (int)cta_rank * BLOCK_M, brow = n_blk * BLOCK_N + (int)cta_rank * C::B_ROWS;
                            if (k3) {
                                tma_load_3d_cg2(st0, &tmap_a, 0, arow, kb, lead_full);
                                tma_load_3d_cg2(sb0, &tmap_b, 0, brow, kb, lead_full);
                            } else {
                                for (int i = 0; i < cnt; ++i) {
                                    tma_load_2d_cg2(st0 + i * C::A_BYTES, &tmap_a, (kb + i) * BLOCK_K, arow, lead_full);
                                    tma_load_2d_cg2(sb0 + i * C::B_BYTES, &tmap_b, (kb + i) * BLOCK_K, brow, lead_full);
                                }
                            }
                        }
                        if (tile == tile0 && kb == 0) RLX_TRACE(p, 3);
                    }
                    __syncwarp();
                    if (++stage == C::STAGES) { stage = 0; phase ^= 1; }
                }
            }
            if (lane == 0) RLX_TRACE(p, 4);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (whole warp, one lane issues)
        if (cta_rank == 0) {
            constexpr uint32_t idesc = make_idesc(TILE_M, BLOCK_N);
            int stage = 0;
            uint32_t phase = 0;
            int it = 0;
            bool ok = true;
            if (lane == 0) { RLX_TRACE(p, 9); RLX_TRACE_CLK(p, 14); }
            RLX_CLK_DECL(clk_full);
            RLX_CLK_DECL(clk_tempty);
            for (int tile = tile0; tile < num_tiles && ok; tile += tile_step, ++it) {
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
                    if (it == 2 && kb == 0 && lane == 0) RLX_TRACE_CLK(p, 60);            // MMA thread starts waiting for that stage
                    RLX_CLK_ADD(clk_full, got_ops = mbar_wait_warp(full_bar + 8 * stage, phase, abort_flag));
                    if (!got_ops) { ok = false; break; }
                    if (it == 2 && kb == 0 && lane == 0) RLX_TRACE_CLK(p, 61);            // operands landed
                    tc_fence_after();
                    const uint32_t st0 = base + stage * C::STAGE_BYTES;
                    if (elect_one()) {
                        if (it == 0 && kb == 0) RLX_TRACE(p, 5);
                        if (!RLX_DBG(p, kDbgNoMma)) {
                            for (int i = 0; i < cnt; ++i) {
                                const uint64_t adesc = make_smem_desc(st0 + i * C::A_BYTES);
                                const uint64_t bdesc = make_smem_desc(st0 + C::KPS * C::A_BYTES + i * C::B_BYTES);
#pragma unroll
                                for (int k = 0; k < BLOCK_K / UMMA_K; ++k) {
                                    // advancing 16 bf16 = 32 bytes along K inside the swizzle row: +2 in 16-byte units
                                    umma_bf16<CG>(tmem_d, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | i | k) != 0 ? 1u : 0u);
                                }
                            }
                        }
                        umma_commit<CG>(empty_bar + 8 * stage);  // stage reusable once these MMAs have read it
                    }
                    __syncwarp();
                    if (++stage == C::STAGES) { stage = 0; phase ^= 1; }
                }
                if (ok && elect_one()) {
                    umma_commit<CG>(tfull_bar + 8 * as);  // accumulator complete
                    if (it == 0) RLX_TRACE(p, 6);
                }
                __syncwarp();
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
        const int half = ew >> 2;             // which column slab of the tile
        const uint32_t stg = staging + ew * kStageBufBytes;
        int it = 0;
        bool ok = true;
        if (tile0 < num_tiles) EpilogueTile<EPI, C::SLAB / 32>::prefetch_bias(p, (tile0 % n_tiles) * BLOCK_N + half * C::SLAB);
        for (int tile = tile0; tile < num_tiles && ok; tile += tile_step, ++it) {
            const int m_blk = tile / n_tiles, n_blk = tile % n_tiles;
            if (tile + tile_step < num_tiles)
                EpilogueTile<EPI, C::SLAB / 32>::prefetch_bias(p, ((tile + tile_step) % n_tiles) * BLOCK_N + half * C::SLAB);
            const int as = it & 1;
            const uint32_t aphase = (it >> 1) & 1;
            const int m_row0 = m_blk * TILE_M + (int)cta_rank * BLOCK_M + quad * 32;
            const int n0 = n_blk * BLOCK_N + half * C::SLAB;
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + as * BLOCK_N + half * C::SLAB;
            EpilogueTile<EPI, C::SLAB / 32> et;
            et.prefetch(p, M, m_row0 + lane, n0);   // residual / row statistics: issued before the accumulator wait
            if (!mbar_wait(tfull_bar + 8 * as, aphase, abort_flag)) { ok = false; break; }
            tc_fence_after();
            if (ew == 0 && lane == 0 && it < 12) RLX_TRACE(p, 16 + it);
            et.template drain<CG>(p, &tmap_out, M, m_row0, n0, taddr, stg, lane, tempty_bar + 8 * as, cta_rank,
                                  (ew == 0 && lane == 0 && (it == 1 || it == 5)) ? 40 + 2 * (it - 1) : -1);
            if (ew == 0 && lane == 0 && it < 12) RLX_TRACE(p, 28 + it);
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
    if constexpr (CG == 2) cluster_sync_all();   // neither CTA leaves while the pair still uses its memory
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc<CG>(tmem_base, C::TMEM_COLS);
        if (lane == 0) RLX_TRACE(p, 13);
    }
}

}  // namespace tc
}  // namespace rlx
