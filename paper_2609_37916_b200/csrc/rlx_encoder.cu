// C-ABI library of the sm_100a encoder forward: host runtime (validation, workspace arena,
// tensor-map construction, CUDA-graph cache) and the launchers of every kernel.
// Single translation unit: all kernels are included below.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <vector>

#include "../../include/rlx_encoder.h"
#include "attention.cuh"
#include "attention_tc.cuh"
#include "gemm_mx_tcgen05.cuh"
#include "gemm_ffn_tcgen05.cuh"
#include "dequant.cuh"
#include "gemm_simt.cuh"
#include "gemm_tcgen05.cuh"
#include "gemm_ares_tcgen05.cuh"
#include "gemm_ln_tcgen05.cuh"
#include "gemm_cln_tcgen05.cuh"
#include "rowwise.cuh"

namespace {

using bf16 = __nv_bfloat16;

#define RLX_CUDA_TRY(expr)                      \
    do {                                        \
        cudaError_t _e = (expr);                \
        if (_e != cudaSuccess) {                \
            g_last_cuda_error = _e;             \
            (void)cudaGetLastError();           \
            return RLX_ERR_CUDA;                \
        }                                       \
    } while (0)

thread_local cudaError_t g_last_cuda_error = cudaSuccess;

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// ------------------------------------------------------------------ tensor maps
typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

encode_tiled_fn get_encode_fn() {
    static encode_tiled_fn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<encode_tiled_fn>(p);
    });
    return fn;
}

// bf16 row-major [rows, cols] matrix, box = box_rows x box_cols; operand tiles use 64 columns with the
// 128-byte swizzle, output chunks 32 columns with the 64-byte swizzle; zero OOB fill on loads,
// out-of-range rows dropped on stores.
bool make_tmap(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows,
               uint32_t box_cols = rlx::tc::BLOCK_K, CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_128B) {
    encode_tiled_fn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * sizeof(bf16)};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// Row-major matrix of BYTES (8-bit element codes), 128-byte swizzle, box = box_rows x 128 bytes.
bool make_tmap_u8(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    encode_tiled_fn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols};
    cuuint32_t box[2] = {128, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// The same matrix viewed as [k-block][row][64 columns] (cols % 64 == 0): a box of `kps` k-blocks x
// box_rows rows lands in shared memory as kps complete 128-byte-swizzled operand tiles, one after the
// other, so one TMA instruction feeds a whole multi-k-block pipeline stage.
bool make_tmap_kblocks(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows, uint32_t kps) {
    encode_tiled_fn fn = get_encode_fn();
    if (!fn || cols % rlx::tc::BLOCK_K != 0) return false;
    cuuint64_t dims[3] = {(cuuint64_t)rlx::tc::BLOCK_K, rows, cols / rlx::tc::BLOCK_K};
    cuuint64_t strides[2] = {cols * sizeof(bf16), rlx::tc::BLOCK_K * sizeof(bf16)};
    cuuint32_t box[3] = {(cuuint32_t)rlx::tc::BLOCK_K, box_rows, kps};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// Operand maps of a GEMM whose pipeline stages hold `kps` k-blocks: the k-block view when it exists
// (K % 64 == 0, kps > 1), else the plain 2-D maps with one load per k-block.  Returns the kblock_maps flag.
int make_operand_tmaps(CUtensorMap* ta, CUtensorMap* tb, const void* A, const void* W, uint64_t M, uint64_t N, uint64_t K,
                       uint32_t a_rows, uint32_t b_rows, int kps) {
    if (kps > 1 && K % rlx::tc::BLOCK_K == 0 && make_tmap_kblocks(ta, A, M, K, a_rows, (uint32_t)kps) &&
        make_tmap_kblocks(tb, W, N, K, b_rows, (uint32_t)kps))
        return 1;
    if (!make_tmap(ta, A, M, K, a_rows) || !make_tmap(tb, W, N, K, b_rows)) return -1;
    return 0;
}

// ------------------------------------------------------------------ one-time kernel attributes
template <int BN, int EPI, int CG>
cudaError_t set_gemm_attr() {
    return cudaFuncSetAttribute(rlx::tc::gemm_tcgen05_kernel<BN, EPI, CG>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                rlx::tc::Cfg<BN, CG>::SMEM_BYTES);
}
template <int BN, int CG = 1>
cudaError_t set_gemm_attr_all() {
    cudaError_t e;
    if ((e = set_gemm_attr<BN, 0, CG>()) != cudaSuccess) return e;
    if ((e = set_gemm_attr<BN, 1, CG>()) != cudaSuccess) return e;
    if ((e = set_gemm_attr<BN, 2, CG>()) != cudaSuccess) return e;
    if ((e = set_gemm_attr<BN, 3, CG>()) != cudaSuccess) return e;
    if ((e = set_gemm_attr<BN, 4, CG>()) != cudaSuccess) return e;
    if ((e = set_gemm_attr<BN, 5, CG>()) != cudaSuccess) return e;
    return set_gemm_attr<BN, 6, CG>();
}

// Number of CTA pairs that can be resident at once (pairs must sit in one GPC), per device.
int g_max_pairs[64] = {};
int g_max_pairs_resident[64] = {};   // the same for the A-resident kernel (its own shared-memory footprint)

// Multiprocessor count of the current device (grids of the persistent kernels are sized from it).
constexpr int kNominalSMs = 148;   // B200; used only when no device can be queried (host-only callers)
int sm_count_of(int dev) {
    static int cached[64] = {};
    if (dev < 0 || dev >= 64) return kNominalSMs;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
            (void)cudaGetLastError();
            return kNominalSMs;
        }
        cached[dev] = n;
    }
    return cached[dev];
}
int sm_count() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return kNominalSMs;
    }
    return sm_count_of(dev);
}

cudaError_t init_kernels_for_current_device() {
    static std::mutex mu;
    static bool done[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lk(mu);
    if (dev < 64 && done[dev]) return cudaSuccess;
    if ((e = set_gemm_attr_all<64>()) != cudaSuccess) return e;
    if ((e = set_gemm_attr_all<128>()) != cudaSuccess) return e;
    if ((e = set_gemm_attr_all<192>()) != cudaSuccess) return e;
    if ((e = set_gemm_attr_all<256>()) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(rlx::tcln::gemm_ln_tcgen05_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  rlx::tcln::Cfg<128>::SMEM_BYTES)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(rlx::tcln::gemm_ln_tcgen05_kernel<192>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  rlx::tcln::Cfg<192>::SMEM_BYTES)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(rlx::tcln::gemm_ln_tcgen05_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  rlx::tcln::Cfg<256>::SMEM_BYTES)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(rlx::tccl::gemm_cln_tcgen05_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  rlx::tccl::Cfg<64>::SMEM_BYTES)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(rlx::tccl::gemm_cln_tcgen05_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  rlx::tccl::Cfg<128>::SMEM_BYTES)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(rlx::tccl::gemm_cln_tcgen05_kernel<192>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  rlx::tccl::Cfg<192>::SMEM_BYTES)) != cudaSuccess) return e;
    if ((e = (set_gemm_attr_all<128, 2>())) != cudaSuccess) return e;
    if ((e = (set_gemm_attr_all<192, 2>())) != cudaSuccess) return e;
    if ((e = (set_gemm_attr_all<256, 2>())) != cudaSuccess) return e;
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2 * sm_count());
        cfg.blockDim = dim3(rlx::tc::Cfg<256, 2>::THREADS);
        cfg.dynamicSmemBytes = rlx::tc::Cfg<256, 2>::SMEM_BYTES;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int n = 0;
        if ((e = cudaOccupancyMaxActiveClusters(&n, rlx::tc::gemm_tcgen05_kernel<256, 0, 2>, &cfg)) != cudaSuccess) return e;
        if (dev < 64) g_max_pairs[dev] = n;
    }
#define RLX_ARES_ATTR(BN, EPI)                                                                                  \
    if ((e = cudaFuncSetAttribute(rlx::tcar::gemm_ares_tcgen05_kernel<BN, EPI>,                                \
                                  cudaFuncAttributeMaxDynamicSharedMemorySize, rlx::tcar::Cfg<BN>::SMEM_BYTES)) != \
        cudaSuccess)                                                                                           \
        return e;
    RLX_ARES_ATTR(128, 0) RLX_ARES_ATTR(128, 1) RLX_ARES_ATTR(128, 2)
    RLX_ARES_ATTR(192, 0) RLX_ARES_ATTR(192, 1) RLX_ARES_ATTR(192, 2)
    RLX_ARES_ATTR(256, 0) RLX_ARES_ATTR(256, 1) RLX_ARES_ATTR(256, 2)
#undef RLX_ARES_ATTR
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2 * sm_count());
        cfg.blockDim = dim3(rlx::tcar::Cfg<256>::THREADS);
        cfg.dynamicSmemBytes = rlx::tcar::Cfg<256>::SMEM_BYTES;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int n = 0;
        if ((e = cudaOccupancyMaxActiveClusters(&n, rlx::tcar::gemm_ares_tcgen05_kernel<256, 0>, &cfg)) != cudaSuccess) return e;
        if (dev < 64) g_max_pairs_resident[dev] = n;
    }
    {
        const void* ffn_kernels[] = {(const void*)rlx::tcff::ffn_fused_tcgen05_kernel<384, false, false>, (const void*)rlx::tcff::ffn_fused_tcgen05_kernel<384, true, false>,
                                     (const void*)rlx::tcff::ffn_fused_tcgen05_kernel<384, true, true>,   (const void*)rlx::tcff::ffn_fused_tcgen05_kernel<256, false, false>,
                                     (const void*)rlx::tcff::ffn_fused_tcgen05_kernel<256, true, false>,  (const void*)rlx::tcff::ffn_fused_tcgen05_kernel<256, true, true>};
        for (int i = 0; i < 6; ++i)
            if ((e = cudaFuncSetAttribute(ffn_kernels[i], cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          i < 3 ? rlx::tcff::Cfg<384>::SMEM_BYTES : rlx::tcff::Cfg<256>::SMEM_BYTES)) != cudaSuccess) return e;
    }
    if ((e = cudaFuncSetAttribute(rlx::tcmx::gemm_mx_tcgen05_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  rlx::tcmx::kSmemBytes)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(rlx::tcmx::wide::gemm_mx192_tcgen05_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  rlx::tcmx::wide::kSmemBytesW)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(rlx::tca::attention_tc_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  rlx::tca::Smem<32>::BYTES)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(rlx::tca::attention_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  rlx::tca::Smem<64>::BYTES)) != cudaSuccess) return e;
#define RLX_ATT_SMEM_ATTR(D, MK, ROPE)                                                                       \
    if ((e = cudaFuncSetAttribute(rlx::attention_bf16_kernel<D, MK, ROPE>,                                  \
                                  cudaFuncAttributeMaxDynamicSharedMemorySize,                 \
                                  (int)sizeof(rlx::AttSmem<D>))) != \
        cudaSuccess)                                                                                        \
        return e;
    RLX_ATT_SMEM_ATTR(32, 0, false) RLX_ATT_SMEM_ATTR(64, 0, false)
    if ((e = cudaFuncSetAttribute(rlx::attention_bf16_kernel<32, 0, false, 32, 4, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  (int)sizeof(rlx::AttSmem<32, rlx::AttRing<true>::BN, rlx::AttRing<true>::ST>))) != cudaSuccess)
        return e;
    RLX_ATT_SMEM_ATTR(32, 0, true) RLX_ATT_SMEM_ATTR(64, 0, true)
    RLX_ATT_SMEM_ATTR(32, 1, false) RLX_ATT_SMEM_ATTR(64, 1, false)
    RLX_ATT_SMEM_ATTR(32, 1, true) RLX_ATT_SMEM_ATTR(64, 1, true)
    RLX_ATT_SMEM_ATTR(128, 0, false) RLX_ATT_SMEM_ATTR(128, 0, true) RLX_ATT_SMEM_ATTR(128, 1, false) RLX_ATT_SMEM_ATTR(128, 1, true)
#undef RLX_ATT_SMEM_ATTR
    if (dev < 64) done[dev] = true;
    return cudaSuccess;
}

// ------------------------------------------------------------------ launchers
// When set, kernels are launched with the programmatic-stream-serialization attribute so that each
// kernel's prologue overlaps its predecessor's tail (the kernels call griddepcontrol.wait before
// they read anything a predecessor wrote).  Set by enqueue_forward around its launches.
thread_local bool g_pdl_launch = false;

thread_local int g_cluster_x = 1;   // set by the CTA-pair GEMM launcher around its launch

template <typename... KArgs, typename... Args>
cudaError_t launch_ex(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    unsigned n = 0;
    if (g_pdl_launch) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    if (g_cluster_x > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = (unsigned)g_cluster_x;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

struct Packing {   // device arrays written by pack_sequences_kernel; all null in padded mode
    const int32_t* seq_len = nullptr;
    const int32_t* seq_start = nullptr;    // [B+1]; seq_start[B] = number of packed rows
    const int32_t* pos_of_rank = nullptr;
    int B = 0;
    const int32_t* total() const { return seq_start ? seq_start + B : nullptr; }
};

rlx_status_t launch_pack(const int32_t* mask, int B, int S, int32_t* seq_len, int32_t* seq_start,
                         int32_t* pos_of_rank, unsigned int* ticket, cudaStream_t st,
                         cudaGraphConditionalHandle cond = 0, int cond_min_rows = 0) {
    rlx::pack_sequences_kernel<<<B, rlx::kPackThreads, 0, st>>>(mask, B, S, seq_len, seq_start, pos_of_rank, ticket, cond,
                                                                cond_min_rows);
    RLX_CUDA_TRY(cudaGetLastError());
    return RLX_OK;
}

rlx_status_t launch_embed_ln(const int32_t* ids, const bf16* word, const bf16* pos, const bf16* type,
                             const float* g, const float* b, int T, int S, int H, int V, float eps, bf16* out,
                             int32_t* status, cudaStream_t st, const Packing& pk = Packing()) {
    const int grid = (T + rlx::kRowWarps - 1) / rlx::kRowWarps, thr = rlx::kRowWarps * 32;
    switch (H / 128) {
#define RLX_CASE(NV) case NV: RLX_CUDA_TRY(launch_ex(rlx::embed_ln_kernel<NV>, grid, thr, 0, st, ids, word, pos, type, g, b, out, T, S, V, eps, status, pk.seq_start, pk.pos_of_rank, pk.B)); break;
        RLX_CASE(1) RLX_CASE(2) RLX_CASE(3) RLX_CASE(4) RLX_CASE(5) RLX_CASE(6) RLX_CASE(7) RLX_CASE(8)
#undef RLX_CASE
        default: return RLX_ERR_UNSUPPORTED;
    }
    RLX_CUDA_TRY(cudaGetLastError());
    return RLX_OK;
}

rlx_status_t launch_layernorm(const bf16* x, const float* g, const float* b, int T, int H, float eps, bf16* out,
                              cudaStream_t st, const int32_t* rows_ptr = nullptr) {
    // rows per warp: as many as still leave ~4 CTAs for every SM (static row bound T), so that large
    // problems run as about one full wave of fat CTAs and small ones still cover all SMs
    const int want_ctas = 4 * sm_count();
    const int rpw = (T >= want_ctas * rlx::kRowWarps * 4) ? 4 : 1;   // 8 rows per warp measured slower
    const int rows_per_cta = rlx::kRowWarps * rpw;
    const int grid = (T + rows_per_cta - 1) / rows_per_cta, thr = rlx::kRowWarps * 32;
    switch (H / 128) {
#define RLX_CASE(NV) case NV: if (rpw == 4) RLX_CUDA_TRY(launch_ex(rlx::layernorm_kernel<NV, 4>, grid, thr, 0, st, x, g, b, out, T, eps, rows_ptr)); \
                     else RLX_CUDA_TRY(launch_ex(rlx::layernorm_kernel<NV, 1>, grid, thr, 0, st, x, g, b, out, T, eps, rows_ptr)); break;
        RLX_CASE(1) RLX_CASE(2) RLX_CASE(3) RLX_CASE(4) RLX_CASE(5) RLX_CASE(6) RLX_CASE(7) RLX_CASE(8)
#undef RLX_CASE
        default: return RLX_ERR_UNSUPPORTED;
    }
    RLX_CUDA_TRY(cudaGetLastError());
    return RLX_OK;
}

rlx_status_t launch_pool(const bf16* x, const int32_t* mask, int B, int S, int H, float* out, cudaStream_t st,
                         const Packing& pk = Packing()) {
    const int vecs = H / 8, G = rlx::kPoolThreads / vecs;
    const size_t smem = (size_t)G * H * sizeof(float);
    RLX_CUDA_TRY(launch_ex(rlx::pool_l2norm_kernel, B, rlx::kPoolThreads, smem, st, x, mask, out, S, H, pk.seq_start, pk.seq_len));
    RLX_CUDA_TRY(cudaGetLastError());
    return RLX_OK;
}

rlx_status_t launch_pool_ln(const bf16* z, const int32_t* mask, int B, int S, int H, float* out, cudaStream_t st,
                            const Packing& pk, const float2* stats, const float* gamma, const float* beta, float eps) {
    if (S > rlx::kPoolMaxRows) return RLX_ERR_UNSUPPORTED;
    const int vecs = H / 8, G = rlx::kPoolThreads / vecs;
    const size_t smem = (size_t)G * H * sizeof(float);
    RLX_CUDA_TRY(launch_ex(rlx::pool_ln_l2norm_kernel, B, rlx::kPoolThreads, smem, st, z, mask, out, S, H, pk.seq_start,
                           pk.seq_len, stats, H / 32, gamma, beta, eps));
    RLX_CUDA_TRY(cudaGetLastError());
    return RLX_OK;
}

// positional = false: every key of the sequence is visible (the encoder's attention); true: the window
// rule of the kernel's MK = 1 mode (packed rows only).  rope_cos == nullptr: no rotary embedding.
rlx_status_t launch_attention_bf16(const bf16* qkv, const int32_t* mask, const int32_t* seq_start,
                                   const int32_t* seq_len, int B, int S, int h, int d, bf16* ctx, cudaStream_t st,
                                   bool positional = false, int window = 0, const float* rope_cos = nullptr,
                                   const float* rope_sin = nullptr, int kv_group = 1) {
    const int H = h * d;
    const float scale_log2e = 1.4426950408889634f / sqrtf((float)d);
    dim3 grid((S + rlx::kAttBlockM - 1) / rlx::kAttBlockM, h, B);
    const rlx::AttKind kind{window, rope_cos, rope_sin, kv_group};
    const bool rope = rope_cos != nullptr;
    if (d != 32 && d != 64 && d != 128) return RLX_ERR_UNSUPPORTED;
#define RLX_ATT_LAUNCH(D, MK, ROPE)                                                                              \
    RLX_CUDA_TRY(launch_ex(rlx::attention_bf16_kernel<D, MK, ROPE>, grid, rlx::kAttThreads,                      \
                           sizeof(rlx::AttSmem<D>),                                                                 \
                           st, qkv, mask, seq_start, seq_len, ctx, S, H, scale_log2e, kind))
    if (d == 32) {
        if (!positional && !rope && S <= rlx::kAttMaxSeq)   // the encoder's shape: 128-key stages, two deep
            RLX_CUDA_TRY(launch_ex(rlx::attention_bf16_kernel<32, 0, false, 32, 4, true>, grid, rlx::kAttThreads,
                                   sizeof(rlx::AttSmem<32, rlx::AttRing<true>::BN, rlx::AttRing<true>::ST>), st, qkv, mask, seq_start,
                                   seq_len, ctx, S, H, scale_log2e, kind));
        else if (!positional && !rope) RLX_ATT_LAUNCH(32, 0, false);
        else if (!positional) RLX_ATT_LAUNCH(32, 0, true);
        else if (!rope) RLX_ATT_LAUNCH(32, 1, false);
        else RLX_ATT_LAUNCH(32, 1, true);
    } else if (d == 64) {
        if (!positional && !rope) RLX_ATT_LAUNCH(64, 0, false);
        else if (!positional) RLX_ATT_LAUNCH(64, 0, true);
        else if (!rope) RLX_ATT_LAUNCH(64, 1, false);
        else RLX_ATT_LAUNCH(64, 1, true);
    } else {
        if (!positional && !rope) RLX_ATT_LAUNCH(128, 0, false);
        else if (!positional) RLX_ATT_LAUNCH(128, 0, true);
        else if (!rope) RLX_ATT_LAUNCH(128, 1, false);
        else RLX_ATT_LAUNCH(128, 1, true);
    }
#undef RLX_ATT_LAUNCH
    RLX_CUDA_TRY(cudaGetLastError());
    return RLX_OK;
}

__device__ unsigned int g_attn_ticket_standalone;   // work-item counter of rlx_attention_packed_bf16's own launches

// Packed-sequence attention on tcgen05 (the product path): qkv is the packed [rows, 3H] projection.
rlx_status_t launch_attention_tc(const bf16* qkv, int rows, const int32_t* seq_start, const int32_t* seq_len, int B,
                                 int S, int h, int d, bf16* ctx, unsigned int* ticket, int32_t* status, cudaStream_t st) {
    const int H = h * d;
    const float scale_log2e = 1.4426950408889634f / sqrtf((float)d);
    CUtensorMap tq;
    if (!make_tmap(&tq, qkv, (uint64_t)rows, (uint64_t)3 * H, rlx::tca::kBlockN, (uint32_t)d,
                   d == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B))
        return RLX_ERR_CUDA;
    // persistent: two CTAs per SM walk the (sequence, query tile, head) list with a fixed stride
    const int qtiles = (S + rlx::tca::kBlockM - 1) / rlx::tca::kBlockM;
    const long long n_cand = (long long)B * qtiles * h;
#ifdef RLX_ATTN_ONE_PER_SM
    const int grid = (int)std::min<long long>(n_cand, 1LL * sm_count());
#else
    const int grid = (int)std::min<long long>(n_cand, 2LL * sm_count());
#endif
    if (d == 32)
        RLX_CUDA_TRY(launch_ex(rlx::tca::attention_tc_kernel<32>, dim3(grid), rlx::tca::kThreads, rlx::tca::Smem<32>::BYTES, st,
                               tq, seq_start, seq_len, ctx, H, scale_log2e, B, qtiles, ticket, status));
    else if (d == 64)
        RLX_CUDA_TRY(launch_ex(rlx::tca::attention_tc_kernel<64>, dim3(grid), rlx::tca::kThreads, rlx::tca::Smem<64>::BYTES, st,
                               tq, seq_start, seq_len, ctx, H, scale_log2e, B, qtiles, ticket, status));
    else
        return RLX_ERR_UNSUPPORTED;
    RLX_CUDA_TRY(cudaGetLastError());
    return RLX_OK;
}

// Feed-forward block in one kernel (hidden 256 or 384, F % 64 == 0): out = gelu(x W1^T + b1) W2^T + b2 + x.
bool ffn_fused_supported(int H, int F) { return (H == 256 || H == 384) && F % 128 == 0 && F >= 128; }
// One launcher for the three forms of the row-block kernel:
//   pre == nullptr:  out = [LayerNorm2](gelu(x W1^T + b1) W2^T + b2 + x)
//   pre != nullptr:  x1 = LayerNorm1(ctx Wo^T + bo + h) first (x = ctx), then the same with x1 in place of x
struct FfnPre {
    const bf16* h;      // residual rows of the projection in front
    const bf16* wo;     // [H, H]
    const float* bo;
    const float* ln1_gamma;
    const float* ln1_beta;
};
rlx_status_t launch_ffn_fused(const bf16* x, const bf16* w1, const float* b1, const bf16* w2, const float* b2, int M, int H,
                              int F, bf16* out, int32_t* status, cudaStream_t st, const int32_t* rows_ptr,
                              const float* ln_gamma = nullptr, const float* ln_beta = nullptr, float ln_eps = 0.f,
                              const FfnPre* pre = nullptr) {
    if (!ffn_fused_supported(H, F)) return RLX_ERR_UNSUPPORTED;
    if (pre && !ln_gamma) return RLX_ERR_INVALID_ARG;
    const uint32_t w2_rows = H == 384 ? rlx::tcff::Cfg<384>::W2_ROWS : rlx::tcff::Cfg<256>::W2_ROWS;
    CUtensorMap tx, t1, t2, to, two, th;
    if (!make_tmap(&tx, x, (uint64_t)M, (uint64_t)H, rlx::tc::BLOCK_M) || !make_tmap(&to, out, (uint64_t)M, (uint64_t)H, 32) ||
        !make_tmap(&t1, w1, (uint64_t)F, (uint64_t)H, H == 384 ? rlx::tcff::Cfg<384>::W1_ROWS : rlx::tcff::Cfg<256>::W1_ROWS) ||
        !make_tmap(&t2, w2, (uint64_t)H, (uint64_t)F, w2_rows))
        return RLX_ERR_CUDA;
    two = t2; th = tx;
    if (pre && (!make_tmap(&two, pre->wo, (uint64_t)H, (uint64_t)H, w2_rows) || !make_tmap(&th, pre->h, (uint64_t)M, (uint64_t)H, rlx::tc::BLOCK_M)))
        return RLX_ERR_CUDA;
    rlx::tcff::FfnParams p;
    p.b1 = b1; p.b2 = b2; p.out = out; p.M = M; p.F = F; p.m_ptr = rows_ptr; p.status = status;
    p.ln_gamma = ln_gamma; p.ln_beta = ln_beta; p.ln_eps = ln_eps;
    p.bo = pre ? pre->bo : nullptr; p.ln1_gamma = pre ? pre->ln1_gamma : nullptr; p.ln1_beta = pre ? pre->ln1_beta : nullptr;
    const int form = pre ? 2 : ln_gamma ? 1 : 0;
    int dev = 0;
    cudaGetDevice(&dev);
    const int pairs_max = (dev >= 0 && dev < 64 && g_max_pairs_resident[dev] > 0) ? g_max_pairs_resident[dev] : sm_count() / 2;
    const int blocks = (M + rlx::tcff::kPairRows - 1) / rlx::tcff::kPairRows;
    const int grid = 2 * std::min(blocks, pairs_max);
    struct ClusterScope {
        ClusterScope() { g_cluster_x = 2; }
        ~ClusterScope() { g_cluster_x = 1; }
    } scope;
#define RLX_FFN_LAUNCH(HID, LN, PRE)                                                                                   \
    RLX_CUDA_TRY(launch_ex(rlx::tcff::ffn_fused_tcgen05_kernel<HID, LN, PRE>, grid, rlx::tcff::kThreads,               \
                           rlx::tcff::Cfg<HID>::SMEM_BYTES, st, tx, t1, t2, to, two, th, p))
    if (H == 384) {
        if (form == 2) RLX_FFN_LAUNCH(384, true, true); else if (form == 1) RLX_FFN_LAUNCH(384, true, false); else RLX_FFN_LAUNCH(384, false, false);
    } else {
        if (form == 2) RLX_FFN_LAUNCH(256, true, true); else if (form == 1) RLX_FFN_LAUNCH(256, true, false); else RLX_FFN_LAUNCH(256, false, false);
    }
#undef RLX_FFN_LAUNCH
    RLX_CUDA_TRY(cudaGetLastError());
    return RLX_OK;
}

struct TileChoice { int bn; int cg; };

// Tuning overrides: compiled in only with -DRLX_EXPERIMENTS (rlx_experiment_set); constants otherwise.
#ifdef RLX_EXPERIMENTS
int g_exp_cg = 0, g_exp_bn = 0, g_exp_debug = 0, g_exp_resident = 0;
unsigned long long* g_exp_trace = nullptr;
#else
constexpr int g_exp_cg = 0, g_exp_resident = 0;
#endif

// Tile shape for an [M, N] output.  CTA pairs (cg = 2, 256-row tiles, each CTA loading half of the
// W tile) are used when there are enough tiles to keep every pair busy for a few rounds; smaller
// problems keep one CTA per 128-row tile and shrink BLOCK_N until every SM has work.
TileChoice pick_tile(int M, int N, int K, int want_cg = 0) {
    const int force_cg = want_cg ? want_cg : g_exp_cg;
    int dev = 0;
    cudaGetDevice(&dev);
    const int pairs = (dev >= 0 && dev < 64) ? g_max_pairs[dev] : 0;
#ifdef RLX_EXPERIMENTS
    if (g_exp_bn && N % g_exp_bn == 0 && (g_exp_bn == 64 || g_exp_bn == 128 || g_exp_bn == 192 || g_exp_bn == 256))
        return {g_exp_bn, (force_cg == 2 && g_exp_bn >= 128) ? 2 : 1};
#endif
    // pairs pay off once a tile's main loop is long enough to amortise the cross-CTA handshakes
    // (K >= 1536, or K >= 768 with a wide output) and every pair gets at least two tiles
    if (force_cg != 1 && pairs > 0 && (force_cg == 2 || K >= 1536 || (K >= 768 && N >= 1536))) {
        const int m_tiles2 = (M + 255) / 256;
        const int cand2[3] = {256, 192, 128};
        for (int i = 0; i < 3; ++i)
            if (N % cand2[i] == 0 && (force_cg == 2 || m_tiles2 * (N / cand2[i]) >= 2 * pairs)) return {cand2[i], 2};
    }
    // long contraction, too few tiles for the rule above: a pair per 256 x 128 tile still beats 128 x 64 tiles
    // on single CTAs once half of the pairs have work (measured at 4096 rows, K = 1536: 10.6 vs 15.3 us)
    if (force_cg != 1 && pairs > 0 && K >= 1536 && N % 128 == 0 && ((M + 255) / 256) * (N / 128) >= pairs / 2)
        return {128, 2};
    const int m_tiles = (M + rlx::tc::BLOCK_M - 1) / rlx::tc::BLOCK_M;
    // short contractions run a little faster on 192-wide tiles than on 256-wide ones when both fill the SMs
    const int cand[4] = {K <= 384 ? 192 : 256, K <= 384 ? 256 : 192, 128, 64};
    // first tile in that order that still gives every SM work; otherwise the smallest that divides N
    for (int i = 0; i < 4; ++i)
        if (N % cand[i] == 0 && m_tiles * (N / cand[i]) >= sm_count()) return {cand[i], 1};
    const int small[4] = {64, 128, 192, 256};
    for (int i = 0; i < 4; ++i)
        if (N % small[i] == 0) return {small[i], 1};
    return {0, 1};
}

template <int BN, int CG>
rlx_status_t launch_gemm_tc_bn(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& to,
                               const rlx::tc::Params& p, int epi, cudaStream_t st) {
    const int tile_m = rlx::tc::BLOCK_M * CG;
    const int tiles = ((p.M + tile_m - 1) / tile_m) * (p.N / BN);
    int dev = 0;
    cudaGetDevice(&dev);
    const int slots = CG == 1 ? sm_count() : ((dev >= 0 && dev < 64) ? g_max_pairs[dev] : 1);
    const int grid = CG * (tiles < slots ? tiles : slots);
    const int smem = rlx::tc::Cfg<BN, CG>::SMEM_BYTES;
    struct ClusterScope {
        explicit ClusterScope(int x) { g_cluster_x = x; }
        ~ClusterScope() { g_cluster_x = 1; }
    } scope(CG);
    switch (epi) {
        case 0: RLX_CUDA_TRY(launch_ex(rlx::tc::gemm_tcgen05_kernel<BN, 0, CG>, grid, rlx::tc::Cfg<BN, CG>::THREADS, smem, st, ta, tb, to, p)); break;
        case 1: RLX_CUDA_TRY(launch_ex(rlx::tc::gemm_tcgen05_kernel<BN, 1, CG>, grid, rlx::tc::Cfg<BN, CG>::THREADS, smem, st, ta, tb, to, p)); break;
        case 2: RLX_CUDA_TRY(launch_ex(rlx::tc::gemm_tcgen05_kernel<BN, 2, CG>, grid, rlx::tc::Cfg<BN, CG>::THREADS, smem, st, ta, tb, to, p)); break;
        case 3: RLX_CUDA_TRY(launch_ex(rlx::tc::gemm_tcgen05_kernel<BN, 3, CG>, grid, rlx::tc::Cfg<BN, CG>::THREADS, smem, st, ta, tb, to, p)); break;
        case 4: RLX_CUDA_TRY(launch_ex(rlx::tc::gemm_tcgen05_kernel<BN, 4, CG>, grid, rlx::tc::Cfg<BN, CG>::THREADS, smem, st, ta, tb, to, p)); break;
        case 5: RLX_CUDA_TRY(launch_ex(rlx::tc::gemm_tcgen05_kernel<BN, 5, CG>, grid, rlx::tc::Cfg<BN, CG>::THREADS, smem, st, ta, tb, to, p)); break;
        case 6: RLX_CUDA_TRY(launch_ex(rlx::tc::gemm_tcgen05_kernel<BN, 6, CG>, grid, rlx::tc::Cfg<BN, CG>::THREADS, smem, st, ta, tb, to, p)); break;
        default: return RLX_ERR_INVALID_ARG;
    }
    RLX_CUDA_TRY(cudaGetLastError());
    return RLX_OK;
}

// A-resident CTA-pair GEMM (short contractions): grid = 2 x min(work units, resident pairs).
template <int BN>
rlx_status_t launch_gemm_resident_bn(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& to,
                                     const rlx::tc::Params& p, int epi, cudaStream_t st) {
    int dev = 0;
    cudaGetDevice(&dev);
    const int pairs = (dev >= 0 && dev < 64) ? g_max_pairs_resident[dev] : 0;
    if (pairs <= 0) return RLX_ERR_UNSUPPORTED;
    const int m_blocks = (p.M + rlx::tcar::kPairRows - 1) / rlx::tcar::kPairRows;
    const int units = m_blocks * (p.N / BN);   // the finest split the kernel may choose
    const int grid = 2 * (units < pairs ? units : pairs);
    const int smem = rlx::tcar::Cfg<BN>::SMEM_BYTES, thr = rlx::tcar::Cfg<BN>::THREADS;
    struct ClusterScope {
        explicit ClusterScope(int x) { g_cluster_x = x; }
        ~ClusterScope() { g_cluster_x = 1; }
    } scope(2);
    switch (epi) {
        case 0: RLX_CUDA_TRY(launch_ex(rlx::tcar::gemm_ares_tcgen05_kernel<BN, 0>, grid, thr, smem, st, ta, tb, to, p)); break;
        case 1: RLX_CUDA_TRY(launch_ex(rlx::tcar::gemm_ares_tcgen05_kernel<BN, 1>, grid, thr, smem, st, ta, tb, to, p)); break;
        case 2: RLX_CUDA_TRY(launch_ex(rlx::tcar::gemm_ares_tcgen05_kernel<BN, 2>, grid, thr, smem, st, ta, tb, to, p)); break;
        default: return RLX_ERR_INVALID_ARG;
    }
    RLX_CUDA_TRY(cudaGetLastError());
    return RLX_OK;
}

// Tile width of the A-resident kernel for an [M, N] x K problem, or 0 when it does not apply: K must
// fit the resident block, N must split into 256-, 192- or 128-wide tiles, and (unless forced) there must
// be enough 256-row blocks to give every CTA pair one -- smaller problems keep 128-row tiles per CTA.
int pick_resident_bn(int M, int N, int K, int epi, bool forced) {
    if (epi > 2 || K > rlx::tcar::kMaxKB * rlx::tc::BLOCK_K) return 0;
    int dev = 0;
    cudaGetDevice(&dev);
    const int pairs = (dev >= 0 && dev < 64) ? g_max_pairs_resident[dev] : 0;
    if (pairs <= 0) return 0;
    if (!forced && (M + rlx::tcar::kPairRows - 1) / rlx::tcar::kPairRows < pairs) return 0;
    const int cand[3] = {256, 192, 128};
    for (int i = 0; i < 3; ++i)
        if (N % cand[i] == 0) return cand[i];
    return 0;
}

// Extra operands of the LayerNorm-folding epilogues (EPI 3..6 of the tcgen05 GEMM).
struct LnFold {
    const float* cvec = nullptr;
    const float* dvec = nullptr;
    const float2* stats_in = nullptr;
    int stats_in_p = 0;
    const float* gamma = nullptr;
    const float* beta = nullptr;
    float2* stats_out = nullptr;
    float eps = 0.f;
};

rlx_status_t launch_gemm(const bf16* A, const bf16* W, const float* bias, const bf16* residual, int epi, int M, int N,
                         int K, bf16* out, bool simt, int32_t* status, cudaStream_t st,
                         const int32_t* m_ptr = nullptr, int want_cg = 0, const LnFold* lf = nullptr) {
    if (simt) {
        if (epi >= 3) return RLX_ERR_UNSUPPORTED;
        dim3 grid((N + rlx::kSimtTile - 1) / rlx::kSimtTile, (M + rlx::kSimtTile - 1) / rlx::kSimtTile);
        switch (epi) {
            case 0: rlx::gemm_simt_kernel<0><<<grid, 256, 0, st>>>(A, W, bias, residual, out, M, N, K); break;
            case 1: rlx::gemm_simt_kernel<1><<<grid, 256, 0, st>>>(A, W, bias, residual, out, M, N, K); break;
            case 2: rlx::gemm_simt_kernel<2><<<grid, 256, 0, st>>>(A, W, bias, residual, out, M, N, K); break;
            default: return RLX_ERR_INVALID_ARG;
        }
        RLX_CUDA_TRY(cudaGetLastError());
        return RLX_OK;
    }
    if (K % 8 != 0) return RLX_ERR_UNSUPPORTED;
    rlx::tc::Params p{};
    p.bias = bias; p.residual = residual; p.out = out; p.M = M; p.N = N; p.K = K; p.status = status; p.m_ptr = m_ptr;
#ifdef RLX_EXPERIMENTS
    p.debug = g_exp_debug;
    p.trace = g_exp_trace;
#endif
    CUtensorMap ta, tb, to;
    // output chunks: 32 x 32 bf16 boxes with the 64-byte swizzle of the epilogue's staging buffers
    if (!make_tmap(&to, out, (uint64_t)M, (uint64_t)N, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B)) return RLX_ERR_CUDA;
    // want_cg == 3: the A-resident CTA-pair kernel, forced; 0: chosen when the problem is large enough
    if (want_cg == 3 || (want_cg == 0 && g_exp_resident >= 0)) {
        const int rbn = pick_resident_bn(M, N, K, epi, want_cg == 3 || g_exp_resident > 0);
        if (rbn == 0 && want_cg == 3) return RLX_ERR_UNSUPPORTED;
        if (rbn != 0) {
            p.kblock_maps = make_operand_tmaps(&ta, &tb, A, W, (uint64_t)M, (uint64_t)N, (uint64_t)K, rlx::tc::BLOCK_M,
                                               (uint32_t)(rbn / 2), rlx::tcar::Cfg<128>::KPS);
            if (p.kblock_maps < 0) return RLX_ERR_CUDA;
            switch (rbn) {
                case 128: return launch_gemm_resident_bn<128>(ta, tb, to, p, epi, st);
                case 192: return launch_gemm_resident_bn<192>(ta, tb, to, p, epi, st);
                case 256: return launch_gemm_resident_bn<256>(ta, tb, to, p, epi, st);
            }
        }
    }
    const TileChoice tc = pick_tile(M, N, K, want_cg);
    const int bn = tc.bn;
    if (bn == 0) return RLX_ERR_UNSUPPORTED;
    int kps = 1;
    switch (bn * 10 + tc.cg) {
        case 641: kps = rlx::tc::Cfg<64, 1>::KPS; break;
        case 1281: kps = rlx::tc::Cfg<128, 1>::KPS; break;
        case 1921: kps = rlx::tc::Cfg<192, 1>::KPS; break;
        case 2561: kps = rlx::tc::Cfg<256, 1>::KPS; break;
        case 1282: kps = rlx::tc::Cfg<128, 2>::KPS; break;
        case 1922: kps = rlx::tc::Cfg<192, 2>::KPS; break;
        case 2562: kps = rlx::tc::Cfg<256, 2>::KPS; break;
    }
    p.kblock_maps = make_operand_tmaps(&ta, &tb, A, W, (uint64_t)M, (uint64_t)N, (uint64_t)K, rlx::tc::BLOCK_M,
                                       (uint32_t)(bn / tc.cg), kps);
    if (p.kblock_maps < 0) return RLX_ERR_CUDA;
    if (epi >= 3) {
        if (!lf || N % 32 != 0) return RLX_ERR_INVALID_ARG;
        p.cvec = lf->cvec; p.dvec = lf->dvec; p.stats_in = lf->stats_in; p.stats_in_p = lf->stats_in_p;
        p.ln_gamma = lf->gamma; p.ln_beta = lf->beta; p.stats_out = lf->stats_out; p.ln_eps = lf->eps;
    }
    if (tc.cg == 2) {
        switch (bn) {
            case 128: return launch_gemm_tc_bn<128, 2>(ta, tb, to, p, epi, st);
            case 192: return launch_gemm_tc_bn<192, 2>(ta, tb, to, p, epi, st);
            case 256: return launch_gemm_tc_bn<256, 2>(ta, tb, to, p, epi, st);
        }
        return RLX_ERR_UNSUPPORTED;
    }
    switch (bn) {
        case 64: return launch_gemm_tc_bn<64, 1>(ta, tb, to, p, epi, st);
        case 128: return launch_gemm_tc_bn<128, 1>(ta, tb, to, p, epi, st);
        case 192: return launch_gemm_tc_bn<192, 1>(ta, tb, to, p, epi, st);
        case 256: return launch_gemm_tc_bn<256, 1>(ta, tb, to, p, epi, st);
    }
    return RLX_ERR_UNSUPPORTED;
}

// out = LN(A W^T + bias + residual): whole rows per CTA (N = 256, 384 or 512).
rlx_status_t launch_gemm_ln(const bf16* A, const bf16* W, const float* bias, const bf16* residual, const float* gamma,
                            const float* beta, float eps, int M, int N, int K, bf16* out, int32_t* status,
                            cudaStream_t st, const int32_t* m_ptr = nullptr) {
    if ((N != 256 && N != 384 && N != 512) || K % 8 != 0) return RLX_ERR_UNSUPPORTED;
    const int nh = N / 2;
    CUtensorMap ta, tb;
    if (!make_tmap(&ta, A, (uint64_t)M, (uint64_t)K, rlx::tc::BLOCK_M)) return RLX_ERR_CUDA;
    if (!make_tmap(&tb, W, (uint64_t)N, (uint64_t)K, (uint32_t)nh)) return RLX_ERR_CUDA;
    rlx::tcln::Params p{bias, residual, gamma, beta, out, eps, M, K, status, m_ptr};
    const int tiles = (M + rlx::tc::BLOCK_M - 1) / rlx::tc::BLOCK_M;
    const int grid = tiles < sm_count() ? tiles : sm_count();
    switch (nh) {
        case 128: RLX_CUDA_TRY(launch_ex(rlx::tcln::gemm_ln_tcgen05_kernel<128>, grid, rlx::tcln::kThreads, rlx::tcln::Cfg<128>::SMEM_BYTES, st, ta, tb, p)); break;
        case 192: RLX_CUDA_TRY(launch_ex(rlx::tcln::gemm_ln_tcgen05_kernel<192>, grid, rlx::tcln::kThreads, rlx::tcln::Cfg<192>::SMEM_BYTES, st, ta, tb, p)); break;
        case 256: RLX_CUDA_TRY(launch_ex(rlx::tcln::gemm_ln_tcgen05_kernel<256>, grid, rlx::tcln::kThreads, rlx::tcln::Cfg<256>::SMEM_BYTES, st, ta, tb, p)); break;
    }
    RLX_CUDA_TRY(cudaGetLastError());
    return RLX_OK;
}

// out = LN(A W^T + bias + residual) with cluster-wide row statistics: N / BLOCK_N CTAs per cluster.
template <int BN>
rlx_status_t launch_gemm_cln_bn(const bf16* A, const bf16* W, const rlx::tccl::Params& p, cudaStream_t st) {
    const int nranks = p.N / BN;
    CUtensorMap ta, tb;
    if (!make_tmap(&ta, A, (uint64_t)p.M, (uint64_t)p.K, rlx::tc::BLOCK_M)) return RLX_ERR_CUDA;
    if (!make_tmap(&tb, W, (uint64_t)p.N, (uint64_t)p.K, (uint32_t)BN)) return RLX_ERR_CUDA;
    const int m_tiles = (p.M + rlx::tc::BLOCK_M - 1) / rlx::tc::BLOCK_M;
    // clusters that can be resident at once for this cluster size (cached per device and size)
    static int max_clusters[64][rlx::tccl::kMaxCluster + 1] = {};
    int dev = 0;
    RLX_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return RLX_ERR_UNSUPPORTED;
    if (max_clusters[dev][nranks] == 0) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(nranks * sm_count());
        cfg.blockDim = dim3(rlx::tccl::Cfg<BN>::THREADS);
        cfg.dynamicSmemBytes = rlx::tccl::Cfg<BN>::SMEM_BYTES;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)nranks;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int n = 0;
        RLX_CUDA_TRY(cudaOccupancyMaxActiveClusters(&n, rlx::tccl::gemm_cln_tcgen05_kernel<BN>, &cfg));
        if (n <= 0) return RLX_ERR_UNSUPPORTED;
        max_clusters[dev][nranks] = n;
    }
    const int clusters = m_tiles < max_clusters[dev][nranks] ? m_tiles : max_clusters[dev][nranks];
    struct ClusterScope {
        explicit ClusterScope(int x) { g_cluster_x = x; }
        ~ClusterScope() { g_cluster_x = 1; }
    } scope(nranks);
    RLX_CUDA_TRY(launch_ex(rlx::tccl::gemm_cln_tcgen05_kernel<BN>, nranks * clusters, rlx::tccl::Cfg<BN>::THREADS,
                           rlx::tccl::Cfg<BN>::SMEM_BYTES, st, ta, tb, p));
    RLX_CUDA_TRY(cudaGetLastError());
    return RLX_OK;
}

// Slab width for the clustered LayerNorm GEMM: the widest slab (fewest operand re-reads) that still
// gives every SM a CTA, among those with N / BLOCK_N <= 8 CTAs per cluster; 0 if none fits.
int pick_cln_block_n(int M, int N) {
    const int m_tiles = (M + rlx::tc::BLOCK_M - 1) / rlx::tc::BLOCK_M;
    const int cand[3] = {192, 128, 64};
    int fallback = 0;
    for (int i = 0; i < 3; ++i) {
        if (N % cand[i] != 0 || N / cand[i] > rlx::tccl::kMaxCluster) continue;
        if (m_tiles * (N / cand[i]) >= sm_count()) return cand[i];
        fallback = cand[i];   // keeps the narrowest admissible slab
    }
    return fallback;
}

rlx_status_t launch_gemm_cln(const bf16* A, const bf16* W, const float* bias, const bf16* residual, const float* gamma,
                             const float* beta, float eps, int M, int N, int K, bf16* out, int32_t* status,
                             cudaStream_t st, const int32_t* m_ptr = nullptr) {
    const int bn = pick_cln_block_n(M, N);
    if (bn == 0 || K % 8 != 0) return RLX_ERR_UNSUPPORTED;
    rlx::tccl::Params p{bias, residual, gamma, beta, out, eps, M, N, K, status, m_ptr};
    switch (bn) {
        case 64: return launch_gemm_cln_bn<64>(A, W, p, st);
        case 128: return launch_gemm_cln_bn<128>(A, W, p, st);
        case 192: return launch_gemm_cln_bn<192>(A, W, p, st);
    }
    return RLX_ERR_UNSUPPORTED;
}

// ------------------------------------------------------------------ workspace arena
struct Arena {
    size_t status, ids, mask, out, seq_len, seq_start, pos_of_rank, x, qkv, ctx, y, x1, g, total;
    // RLX_FLAG_FOLD_LN: partial row statistics of y and z, and per layer the gamma-scaled weights with
    // their c / d vectors (fold_layer bytes per layer: Wqkv' | W1' | cqkv | dqkv | c1 | d1)
    size_t stats_y, stats_z, fold, fold_layer, f_wqkv, f_w1, f_cqkv, f_dqkv, f_c1, f_d1;
};
constexpr size_t kTicketOffset = 64;   // packing ticket counter inside the 256-byte status block
constexpr size_t kAttnTicketOffset = 128;   // work-item counter of the attention kernel, same block

Arena plan_arena(int B, int S, int H, int F, int L = 0, bool fold = false) {
    const size_t T = (size_t)B * S;
    Arena a{};
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t o = off;
        off += round_up(bytes, 256);
        return o;
    };
    a.status = take(256);
    a.ids = take(T * 4);
    a.mask = take(T * 4);
    a.out = take((size_t)B * H * 4);
    a.seq_len = take((size_t)B * 4);
    a.seq_start = take((size_t)(B + 1) * 4);
    a.pos_of_rank = take(T * 4);
    a.x = take(T * H * 2);
    a.qkv = take(T * 3 * H * 2);
    a.ctx = take(T * H * 2);
    a.y = take(T * H * 2);
    a.x1 = take(T * H * 2);
    a.g = take(T * F * 2);
    if (fold) {
        a.stats_y = take(T * (size_t)(H / 32) * sizeof(float2));
        a.stats_z = take(T * (size_t)(H / 32) * sizeof(float2));
        size_t lo = 0;
        auto sub = [&](size_t bytes) { size_t o = lo; lo += round_up(bytes, 256); return o; };
        a.f_wqkv = sub((size_t)3 * H * H * 2);
        a.f_w1 = sub((size_t)F * H * 2);
        a.f_cqkv = sub((size_t)3 * H * 4);
        a.f_dqkv = sub((size_t)3 * H * 4);
        a.f_c1 = sub((size_t)F * 4);
        a.f_d1 = sub((size_t)F * 4);
        a.fold_layer = lo;
        a.fold = take(lo * (size_t)L);
    }
    a.total = off;
    return a;
}

// With RLX_FLAG_FUSED_LN the out-projection and FFN-down GEMMs absorb the residual LayerNorm when a
// whole row fits in tensor memory and there are enough 128-row tiles to give every SM one (whole-row
// tiles cannot be split across SMs, so small batches keep the separate GEMM + LayerNorm kernels).
// Opt-in: measured on the 256x256 batch it is on par with the separate kernels, not ahead of them.
bool uses_fused_ln(const rlx_encoder_config_t& c, int B, int S) {
    if ((c.flags & RLX_FLAG_GEMM_SIMT) || !(c.flags & RLX_FLAG_FUSED_LN)) return false;
    if (c.hidden != 256 && c.hidden != 384 && c.hidden != 512) return false;
    return (long long)B * S >= 128ll * sm_count_of(c.device);
}

// Everything of a layer behind the attention in one kernel (out-projection, residual, LayerNorm, FFN-up, GELU,
// FFN-down, residual, LayerNorm): a layer is QKV GEMM, attention and this.  The kernel works in blocks of 256
// rows, one per CTA pair, so it needs about a wave of blocks to beat the separate kernels: forced by
// RLX_FLAG_FUSED_FFN at any size, chosen by itself from 32768 padded tokens on, never with
// RLX_FLAG_NO_FUSED_FFN.  The number of VALID tokens is known only on the device: the form pays from about 9000
// valid rows on (8972 valid: -1 %, 37 k: -15 %) and loses up to 20 % on a heavily padded batch (20480 padded,
// 2729 valid: 393 against 330 us), so the padded threshold is set where a half-empty batch still breaks even.
constexpr long long kAutoFusedFfnMinTokens = 32768;
// Sub-batches of a chunked call take the kernel choice of the whole call (its padded token count), so that
// chunking never changes which kernels compute a row.
thread_local long long g_whole_call_tokens = 0;
// Bodies of the IF / ELSE node of a captured forward are recorded with the choice forced (1: layer tail, 0: separate
// kernels; -1: the host's rule).
thread_local int g_force_layer_tail = -1;
// RLX_FLAG_DEVICE_CHOICE: captured forwards from this size on carry BOTH forms of the layer behind an IF / ELSE node
// that the packing kernel sets from the packed row count: the host knows only the padded size, and the layer tail
// loses up to 20 % on a heavily padded batch (measured: it pays from about 9000 valid rows on).  The node costs
// 15-20 us per forward (no programmatic launch across it), which is why the host's rule is the default.
constexpr long long kDeviceChoiceMinTokens = 12288;   // padded tokens; below, the separate kernels always win
constexpr int kDeviceChoiceMinRows = 9216;            // packed rows from which the layer tail is taken
bool ffn_fused_supported(int H, int F);
bool uses_fold_ln(const rlx_encoder_config_t& c, int B, int S);
bool uses_fused_ffn(const rlx_encoder_config_t& c, int B, int S) {
    if (g_force_layer_tail >= 0) return g_force_layer_tail == 1;
    if (c.flags & (RLX_FLAG_GEMM_SIMT | RLX_FLAG_FUSED_LN | RLX_FLAG_CLUSTER_LN | RLX_FLAG_NO_FUSED_FFN)) return false;
    const long long tokens = g_whole_call_tokens > 0 ? g_whole_call_tokens : (long long)B * S;
    if (!(c.flags & RLX_FLAG_FUSED_FFN) && tokens < kAutoFusedFfnMinTokens) return false;
    return ffn_fused_supported(c.hidden, c.ffn) && !uses_fold_ln(c, B, S);
}

bool uses_device_choice(const rlx_encoder_config_t& c, int B, int S) {
    if (c.flags & (RLX_FLAG_GEMM_SIMT | RLX_FLAG_FUSED_LN | RLX_FLAG_CLUSTER_LN | RLX_FLAG_NO_FUSED_FFN | RLX_FLAG_FUSED_FFN |
                   RLX_FLAG_KERNEL_EVENTS | RLX_FLAG_CHUNKED | RLX_FLAG_NO_PACK | RLX_FLAG_NO_GRAPH | RLX_FLAG_FOLD_LN))
        return false;
    return (c.flags & RLX_FLAG_DEVICE_CHOICE) && g_force_layer_tail < 0 && g_whole_call_tokens == 0 &&
           (long long)B * S >= kDeviceChoiceMinTokens &&
           ffn_fused_supported(c.hidden, c.ffn) && !uses_fold_ln(c, B, S);
}

// RLX_FLAG_CLUSTER_LN: LayerNorm folded into the out-proj / FFN-down GEMMs with cluster-wide row
// statistics.  Opt-in: the two exchanges per tile cost about what the separate LayerNorm kernel costs.
bool uses_cluster_ln(const rlx_encoder_config_t& c) {
    if ((c.flags & RLX_FLAG_GEMM_SIMT) || !(c.flags & RLX_FLAG_CLUSTER_LN)) return false;
    return pick_cln_block_n(128, c.hidden) != 0;
}

// RLX_FLAG_FOLD_LN: LayerNorm folded algebraically into the consuming GEMMs (hidden % 32 == 0, seq <= 512).
// LayerNorm folded into the GEMMs: asked for by flag, or chosen automatically for small batches, where a
// forward is a chain of launch latencies and 5 kernels per layer beat 7 (measured: 1 x 16 tokens 0.043 vs
// 0.046 ms, 1 x 128 0.186 vs 0.199, 32 x 128 with 2.1 k valid tokens 0.254 vs 0.262; the break-even is
// near 3 k VALID tokens -- 32 x 128 with every position valid loses 4 % -- but only the padded size is
// known on the host; at 256 x 256 the folded form loses 10 %).
constexpr int kAutoFoldMaxTokens = 4096;
// Set for the duration of a call that runs out of the built-in arena: the folded form needs room for a
// gamma-scaled copy of every Linear weight (12 MB at H = 384), which that arena does not have.
thread_local bool g_no_auto_fold = false;
bool uses_fold_ln(const rlx_encoder_config_t& c, int B, int S) {
    const bool can = !(c.flags & RLX_FLAG_GEMM_SIMT) && c.hidden % 32 == 0 && c.max_seq <= rlx::kPoolMaxRows;
    if (!can) return false;
    if (c.flags & RLX_FLAG_FOLD_LN) return true;
    const bool other_fusion = (c.flags & (RLX_FLAG_FUSED_LN | RLX_FLAG_CLUSTER_LN)) != 0;
    return !g_no_auto_fold && !(c.flags & RLX_FLAG_NO_AUTO_FOLD) && !other_fusion && (long long)B * S <= kAutoFoldMaxTokens;
}

int kernels_in_forward(const rlx_encoder_config_t& c, int B, int S) {
    const bool pack = !(c.flags & RLX_FLAG_NO_PACK) && !(c.flags & RLX_FLAG_GEMM_SIMT);
    const bool fused = uses_fold_ln(c, B, S) || uses_fused_ln(c, B, S) || uses_cluster_ln(c);
    return 2 + ((fused ? 5 : 7) - (uses_fused_ffn(c, B, S) ? 4 : 0)) * c.num_layers + (pack ? 1 : 0);
}
bool uses_chunks(const rlx_encoder_config_t& c, int B, int S);
int chunk_batch(int B, int S);

struct GraphEntry {
    int B, S;
    const void *ids, *mask, *out, *ws;
    cudaGraphExec_t exec;
};

}  // namespace

struct rlx_encoder {
    rlx_encoder_config_t cfg;
    int head_dim;
    std::vector<rlx_layer_weights_t> layers;  // last weight set seen (graph-cache key)
    rlx_encoder_weights_t weights;
    bool have_weights = false;
    std::vector<GraphEntry> graphs;
    int last_kernels = 0;                   // kernels of the most recent forward (for kernel_times)
    std::vector<cudaEvent_t> events;        // RLX_FLAG_KERNEL_EVENTS: one before the first kernel, one after each
    cudaStream_t side_stream = nullptr;     // side branch of the captured graph (weight prefetch)
    cudaStream_t body_stream = nullptr;     // the two bodies of a captured forward's IF / ELSE node are recorded here
    cudaEvent_t fork_event = nullptr, join_event = nullptr, fold_event = nullptr;
    cudaStream_t capture_stream = nullptr;  // graphs are recorded here (the caller's stream may be the
                                            // legacy default stream, which cannot be captured)
};

namespace {

bool same_weights(const rlx_encoder* e, const rlx_encoder_weights_t* w) {
    if (!e->have_weights) return false;
    if (w->word_emb != e->weights.word_emb || w->pos_emb != e->weights.pos_emb || w->type_emb != e->weights.type_emb ||
        w->emb_ln_g != e->weights.emb_ln_g || w->emb_ln_b != e->weights.emb_ln_b)
        return false;
    return std::memcmp(w->layers, e->layers.data(), sizeof(rlx_layer_weights_t) * e->layers.size()) == 0;
}

void drop_graphs(rlx_encoder* e) {
    for (auto& g : e->graphs) cudaGraphExecDestroy(g.exec);
    e->graphs.clear();
}

// The kernel sequence of one forward, enqueued on `st` (eagerly or under stream capture).
rlx_status_t enqueue_forward(const rlx_encoder* e, const int32_t* ids, const int32_t* mask, int B, int S,
                             const rlx_encoder_weights_t* w, float* out, unsigned char* ws, cudaStream_t st,
                             bool capturing, bool with_events = true, bool body_only = false) {
    const rlx_encoder_config_t& c = e->cfg;
    const int H = c.hidden, F = c.ffn, T = B * S, h = c.num_heads, d = e->head_dim;
    const bool simt = (c.flags & RLX_FLAG_GEMM_SIMT) != 0;
    // valid tokens are packed unless the caller asked for the padded layout (the bring-up GEMM has
    // no dynamic row count, so it implies the padded layout too)
    const bool pack = !(c.flags & RLX_FLAG_NO_PACK) && !simt;
    const bool fold = uses_fold_ln(c, B, S);
    const Arena a = plan_arena(B, S, H, F, c.num_layers, fold);
    int32_t* status = reinterpret_cast<int32_t*>(ws + a.status);
    bf16* x = reinterpret_cast<bf16*>(ws + a.x);
    bf16* qkv = reinterpret_cast<bf16*>(ws + a.qkv);
    bf16* ctx = reinterpret_cast<bf16*>(ws + a.ctx);
    bf16* y = reinterpret_cast<bf16*>(ws + a.y);
    bf16* x1 = reinterpret_cast<bf16*>(ws + a.x1);
    bf16* g = reinterpret_cast<bf16*>(ws + a.g);
    rlx_status_t s;
    size_t ev = 0;
    // With RLX_FLAG_KERNEL_EVENTS an event is recorded between consecutive kernels; under stream
    // capture the records become event-record nodes of the graph, so replays time each kernel on
    // the device without any host launch gap.
    const bool timing = with_events && !e->events.empty();
    auto mark = [&]() -> rlx_status_t {
        if (!timing) return RLX_OK;
        RLX_CUDA_TRY(cudaEventRecordWithFlags(e->events[ev++], st,
                                              capturing ? cudaEventRecordExternal : cudaEventRecordDefault));
        return RLX_OK;
    };
#define RLX_TRY(call) do { s = (call); if (s != RLX_OK) return s; s = mark(); if (s != RLX_OK) return s; } while (0)
    s = mark();
    if (s != RLX_OK) return s;
    // programmatic dependent launch between consecutive kernels; not combined with per-kernel events
    struct PdlScope {
        explicit PdlScope(bool on) { g_pdl_launch = on; }
        ~PdlScope() { g_pdl_launch = false; }
    } pdl_scope(!(c.flags & RLX_FLAG_NO_PDL) && !timing);
    // side branch (captured graphs only): prefetch the Linear weights into L2 when they all fit
    bool forked = false;
    if (capturing && !body_only && e->side_stream && !(c.flags & RLX_FLAG_NO_PREFETCH) && !fold) {   // the fold pass reads the weights anyway
        const size_t per_layer = ((size_t)3 * H * H + (size_t)H * H + (size_t)2 * H * F) * sizeof(bf16);
        if (per_layer * c.num_layers <= ((size_t)48 << 20) && 4 * c.num_layers <= rlx::kMaxPrefetch) {
            rlx::PrefetchList pf = {};
            for (int l = 0; l < c.num_layers; ++l) {
                const rlx_layer_weights_t& lw = w->layers[l];
                const void* ptrs[4] = {lw.wqkv, lw.wo, lw.w1, lw.w2};
                const size_t bytes[4] = {(size_t)3 * H * H * 2, (size_t)H * H * 2, (size_t)F * H * 2, (size_t)H * F * 2};
                for (int i = 0; i < 4; ++i) {
                    pf.ptr[pf.n] = ptrs[i];
                    pf.bytes[pf.n] = (uint32_t)bytes[i];
                    pf.first_piece[pf.n] = pf.total_pieces;
                    pf.total_pieces += (uint32_t)((bytes[i] + rlx::kPrefetchPiece - 1) / rlx::kPrefetchPiece);
                    ++pf.n;
                }
            }
            RLX_CUDA_TRY(cudaEventRecord(e->fork_event, st));
            RLX_CUDA_TRY(cudaStreamWaitEvent(e->side_stream, e->fork_event, 0));
            rlx::prefetch_l2_kernel<<<sm_count(), 32, 0, e->side_stream>>>(pf);
            RLX_CUDA_TRY(cudaGetLastError());
            RLX_CUDA_TRY(cudaEventRecord(e->join_event, e->side_stream));
            forked = true;
        }
    }
    Packing pk;
    if (pack) {
        int32_t* seq_len = reinterpret_cast<int32_t*>(ws + a.seq_len);
        int32_t* seq_start = reinterpret_cast<int32_t*>(ws + a.seq_start);
        int32_t* pos_of_rank = reinterpret_cast<int32_t*>(ws + a.pos_of_rank);
        pk.seq_len = seq_len; pk.seq_start = seq_start; pk.pos_of_rank = pos_of_rank; pk.B = B;
        // The tickets live in the status block, which the caller zeroes once before the first call; each
        // kernel leaves its own at zero again, so no memset node sits in front of the first kernel.
        unsigned int* ticket = reinterpret_cast<unsigned int*>(ws + a.status + kTicketOffset);
        if (capturing && !body_only && e->body_stream && uses_device_choice(c, B, S)) {
            // Both forms of everything behind the packing kernel, as the two bodies of an IF / ELSE node whose
            // condition that kernel sets from the packed row count.
            cudaStreamCaptureStatus cstat;
            cudaGraph_t gcap = nullptr;
            const cudaGraphNode_t* deps = nullptr;
            size_t ndeps = 0;
            RLX_CUDA_TRY(cudaStreamGetCaptureInfo_v2(st, &cstat, nullptr, &gcap, &deps, &ndeps));
            if (cstat != cudaStreamCaptureStatusActive || gcap == nullptr) return RLX_ERR_CUDA;
            cudaGraphConditionalHandle cond;
            RLX_CUDA_TRY(cudaGraphConditionalHandleCreate(&cond, gcap, 0, cudaGraphCondAssignDefault));
            RLX_TRY(launch_pack(mask, B, S, seq_len, seq_start, pos_of_rank, ticket, st, cond, kDeviceChoiceMinRows));
            RLX_CUDA_TRY(cudaStreamGetCaptureInfo_v2(st, &cstat, nullptr, &gcap, &deps, &ndeps));
            cudaGraphNodeParams np = {};
            np.type = cudaGraphNodeTypeConditional;
            np.conditional.handle = cond;
            np.conditional.type = cudaGraphCondTypeIf;
            np.conditional.size = 2;
            cudaGraphNode_t cnode = nullptr;
            RLX_CUDA_TRY(cudaGraphAddNode(&cnode, gcap, deps, ndeps, &np));
            for (int body = 0; body < 2; ++body) {
                RLX_CUDA_TRY(cudaStreamBeginCaptureToGraph(e->body_stream, np.conditional.phGraph_out[body], nullptr, nullptr, 0,
                                                           cudaStreamCaptureModeThreadLocal));
                g_force_layer_tail = body == 0 ? 1 : 0;
                const rlx_status_t bs = enqueue_forward(e, ids, mask, B, S, w, out, ws, e->body_stream, true, false, true);
                g_force_layer_tail = -1;
                g_pdl_launch = !(c.flags & RLX_FLAG_NO_PDL) && !timing;   // the nested call's scope switched it off
                cudaGraph_t ended = nullptr;
                const cudaError_t ce = cudaStreamEndCapture(e->body_stream, &ended);
                if (bs != RLX_OK) return bs;
                RLX_CUDA_TRY(ce);
            }
            RLX_CUDA_TRY(cudaStreamUpdateCaptureDependencies(st, &cnode, 1, cudaStreamSetCaptureDependencies));
            if (forked) RLX_CUDA_TRY(cudaStreamWaitEvent(st, e->join_event, 0));   // join the side branch
            return RLX_OK;
        }
        if (!body_only) RLX_TRY(launch_pack(mask, B, S, seq_len, seq_start, pos_of_rank, ticket, st));
    }
    const int32_t* rows = pk.total();
    const bool fuse_ln = !fold && uses_fused_ln(c, B, S);
    const bool fuse_cln = !fold && !fuse_ln && uses_cluster_ln(c);
    const bool fuse_ffn = uses_fused_ffn(c, B, S);
    if (fold) {
        // ---- LayerNorm folded into the GEMMs: 5 kernels per layer, no LayerNorm kernel ----
        // gamma-scaled weights and their c / d vectors, rebuilt inside every forward (weights may change
        // behind the same pointers).  Under capture the fold runs on the side branch and is joined before
        // the first GEMM that needs it; eager launches run it first on the main stream.
        rlx::FoldList fl = {};
        fl.K = H;
        auto add_job = [&](const void* wm, const float* gm, const float* bt, const float* bias, size_t wf_off, size_t c_off,
                           size_t d_off, int l, int nrows) {
            unsigned char* base = ws + a.fold + (size_t)l * a.fold_layer;
            fl.w[fl.n] = (const bf16*)wm; fl.gamma[fl.n] = gm; fl.beta[fl.n] = bt; fl.bias[fl.n] = bias;
            fl.wf[fl.n] = (bf16*)(base + wf_off); fl.c[fl.n] = (float*)(base + c_off); fl.d[fl.n] = (float*)(base + d_off);
            fl.first_row[fl.n + 1] = fl.first_row[fl.n] + nrows;
            ++fl.n;
        };
        const bool fold_on_side = capturing && e->side_stream != nullptr;
        cudaStream_t fold_st = fold_on_side ? e->side_stream : st;
        if (fold_on_side && !forked) {
            RLX_CUDA_TRY(cudaEventRecord(e->fork_event, st));
            RLX_CUDA_TRY(cudaStreamWaitEvent(e->side_stream, e->fork_event, 0));
            forked = true;
        }
        auto flush_jobs = [&]() -> rlx_status_t {
            if (fl.n == 0) return RLX_OK;
            const int total_rows = fl.first_row[fl.n];
            rlx::ln_fold_weights_kernel<<<(total_rows + rlx::kFoldWarps - 1) / rlx::kFoldWarps, rlx::kFoldWarps * 32, 0, fold_st>>>(fl);
            RLX_CUDA_TRY(cudaGetLastError());
            fl.n = 0;
            fl.first_row[0] = 0;
            return RLX_OK;
        };
        for (int l = 0; l < c.num_layers; ++l) {
            const rlx_layer_weights_t& lw = w->layers[l];
            if (l > 0) {   // the QKV projection of layer l consumes LN2 of layer l-1
                const rlx_layer_weights_t& pw = w->layers[l - 1];
                add_job(lw.wqkv, pw.ln2_g, pw.ln2_b, lw.bqkv, a.f_wqkv, a.f_cqkv, a.f_dqkv, l, 3 * H);
                if (fl.n == rlx::kFoldMaxJobs) { s = flush_jobs(); if (s != RLX_OK) return s; }
            }
            add_job(lw.w1, lw.ln1_g, lw.ln1_b, lw.b1, a.f_w1, a.f_c1, a.f_d1, l, F);
            if (fl.n == rlx::kFoldMaxJobs) { s = flush_jobs(); if (s != RLX_OK) return s; }
        }
        s = flush_jobs();
        if (s != RLX_OK) return s;
        if (fold_on_side) RLX_CUDA_TRY(cudaEventRecord(e->fold_event, e->side_stream));
        if (forked) RLX_CUDA_TRY(cudaEventRecord(e->join_event, e->side_stream));

        float2* stats_y = reinterpret_cast<float2*>(ws + a.stats_y);
        float2* stats_z = reinterpret_cast<float2*>(ws + a.stats_z);
        bf16* z = x1;   // raw output of the FFN-down projection (pre-LayerNorm), reused across layers
        const int P = H / 32;
        RLX_TRY(launch_embed_ln(ids, (const bf16*)w->word_emb, (const bf16*)w->pos_emb, (const bf16*)w->type_emb,
                                w->emb_ln_g, w->emb_ln_b, T, S, H, c.vocab, c.ln_eps, x, status, st, pk));
        for (int l = 0; l < c.num_layers; ++l) {
            const rlx_layer_weights_t& lw = w->layers[l];
            unsigned char* fb = ws + a.fold + (size_t)l * a.fold_layer;
            LnFold lf;
            lf.eps = c.ln_eps;
            if (l == 0) {
                RLX_TRY(launch_gemm(x, (const bf16*)lw.wqkv, lw.bqkv, nullptr, RLX_EPI_BIAS, T, 3 * H, H, qkv, false, status, st, rows));
            } else {
                lf.cvec = (const float*)(fb + a.f_cqkv); lf.dvec = (const float*)(fb + a.f_dqkv);
                lf.stats_in = stats_z; lf.stats_in_p = P;
                RLX_TRY(launch_gemm(z, (const bf16*)(fb + a.f_wqkv), lw.bqkv, nullptr, 3, T, 3 * H, H, qkv, false, status, st, rows, 0, &lf));
            }
            if (pack && (c.flags & RLX_FLAG_ATTN_TCGEN05))
                RLX_TRY(launch_attention_tc(qkv, T, pk.seq_start, pk.seq_len, B, S, h, d, ctx,
                                            reinterpret_cast<unsigned int*>(ws + a.status + kAttnTicketOffset), status, st));
            else
                RLX_TRY(launch_attention_bf16(qkv, mask, pk.seq_start, pk.seq_len, B, S, h, d, ctx, st));
            // y = ctx Wo^T + bo + (l == 0 ? x : LN2_{l-1}(z)); partial statistics of y
            lf = LnFold();
            lf.eps = c.ln_eps;
            lf.stats_out = stats_y;
            if (l == 0) {
                RLX_TRY(launch_gemm(ctx, (const bf16*)lw.wo, lw.bo, x, 5, T, H, H, y, false, status, st, rows, 0, &lf));
            } else {
                const rlx_layer_weights_t& pw = w->layers[l - 1];
                lf.stats_in = stats_z; lf.stats_in_p = P; lf.gamma = pw.ln2_g; lf.beta = pw.ln2_b;
                RLX_TRY(launch_gemm(ctx, (const bf16*)lw.wo, lw.bo, z, 6, T, H, H, y, false, status, st, rows, 0, &lf));
            }
            // g = gelu(LN1(y) W1^T + b1) on the raw y with the folded weights
            if (l == 0 && fold_on_side) RLX_CUDA_TRY(cudaStreamWaitEvent(st, e->fold_event, 0));
            lf = LnFold();
            lf.eps = c.ln_eps;
            lf.cvec = (const float*)(fb + a.f_c1); lf.dvec = (const float*)(fb + a.f_d1);
            lf.stats_in = stats_y; lf.stats_in_p = P;
            RLX_TRY(launch_gemm(y, (const bf16*)(fb + a.f_w1), lw.b1, nullptr, 4, T, F, H, g, false, status, st, rows, 0, &lf));
            // z = g W2^T + b2 + LN1(y); partial statistics of z.  The previous z is dead by now (its last
            // readers were this layer's QKV and out-projection GEMMs).
            lf = LnFold();
            lf.eps = c.ln_eps;
            lf.stats_in = stats_y; lf.stats_in_p = P; lf.gamma = lw.ln1_g; lf.beta = lw.ln1_b; lf.stats_out = stats_z;
            RLX_TRY(launch_gemm(g, (const bf16*)lw.w2, lw.b2, y, 6, T, H, F, z, false, status, st, rows, 0, &lf));
        }
        const rlx_layer_weights_t& last = w->layers[c.num_layers - 1];
        RLX_TRY(launch_pool_ln(z, mask, B, S, H, out, st, pk, stats_z, last.ln2_g, last.ln2_b, c.ln_eps));
        if (forked) RLX_CUDA_TRY(cudaStreamWaitEvent(st, e->join_event, 0));   // join the side branch
        return RLX_OK;
    }
    RLX_TRY(launch_embed_ln(ids, (const bf16*)w->word_emb, (const bf16*)w->pos_emb, (const bf16*)w->type_emb,
                            w->emb_ln_g, w->emb_ln_b, T, S, H, c.vocab, c.ln_eps, x, status, st, pk));
    for (int l = 0; l < c.num_layers; ++l) {
        const rlx_layer_weights_t& lw = w->layers[l];
        RLX_TRY(launch_gemm(x, (const bf16*)lw.wqkv, lw.bqkv, nullptr, RLX_EPI_BIAS, T, 3 * H, H, qkv, simt, status, st, rows));
        if (pack && (c.flags & RLX_FLAG_ATTN_TCGEN05))
            RLX_TRY(launch_attention_tc(qkv, T, pk.seq_start, pk.seq_len, B, S, h, d, ctx,
                                            reinterpret_cast<unsigned int*>(ws + a.status + kAttnTicketOffset), status, st));
        else
            RLX_TRY(launch_attention_bf16(qkv, mask, pk.seq_start, pk.seq_len, B, S, h, d, ctx, st));
        if (fuse_ffn) {
            // everything behind the attention in one kernel: out-projection + residual + LayerNorm, the feed-forward
            // block (the F-wide activation stays on the chip) + residual + LayerNorm; x is read and rewritten by rows
            FfnPre pre{x, (const bf16*)lw.wo, lw.bo, lw.ln1_g, lw.ln1_b};
            RLX_TRY(launch_ffn_fused(ctx, (const bf16*)lw.w1, lw.b1, (const bf16*)lw.w2, lw.b2, T, H, F, x, status, st, rows,
                                     lw.ln2_g, lw.ln2_b, c.ln_eps, &pre));
            continue;
        }
        if (fuse_ln) {
            RLX_TRY(launch_gemm_ln(ctx, (const bf16*)lw.wo, lw.bo, x, lw.ln1_g, lw.ln1_b, c.ln_eps, T, H, H, x1, status, st, rows));
        } else if (fuse_cln) {
            RLX_TRY(launch_gemm_cln(ctx, (const bf16*)lw.wo, lw.bo, x, lw.ln1_g, lw.ln1_b, c.ln_eps, T, H, H, x1, status, st, rows));
        } else {
            RLX_TRY(launch_gemm(ctx, (const bf16*)lw.wo, lw.bo, x, RLX_EPI_BIAS_RESIDUAL, T, H, H, y, simt, status, st, rows));
            RLX_TRY(launch_layernorm(y, lw.ln1_g, lw.ln1_b, T, H, c.ln_eps, x1, st, rows));
        }
        RLX_TRY(launch_gemm(x1, (const bf16*)lw.w1, lw.b1, nullptr, RLX_EPI_BIAS_GELU, T, F, H, g, simt, status, st, rows));
        if (fuse_ln) {
            // x1 is both the residual and (after this kernel) dead; the result goes to x
            RLX_TRY(launch_gemm_ln(g, (const bf16*)lw.w2, lw.b2, x1, lw.ln2_g, lw.ln2_b, c.ln_eps, T, H, F, x, status, st, rows));
        } else if (fuse_cln) {
            RLX_TRY(launch_gemm_cln(g, (const bf16*)lw.w2, lw.b2, x1, lw.ln2_g, lw.ln2_b, c.ln_eps, T, H, F, x, status, st, rows));
        } else {
            RLX_TRY(launch_gemm(g, (const bf16*)lw.w2, lw.b2, x1, RLX_EPI_BIAS_RESIDUAL, T, H, F, y, simt, status, st, rows));
            RLX_TRY(launch_layernorm(y, lw.ln2_g, lw.ln2_b, T, H, c.ln_eps, x, st, rows));
        }
    }
    RLX_TRY(launch_pool(x, mask, B, S, H, out, st, pk));
#undef RLX_TRY
    if (forked) RLX_CUDA_TRY(cudaStreamWaitEvent(st, e->join_event, 0));   // join the side branch
    return RLX_OK;
}

// Token-chunk scheduling (RLX_FLAG_CHUNKED): sequences are independent, so a large batch can run as
// several sub-batches one after the other through the SAME workspace, each small enough that a kernel's
// input is still in the 126 MB L2 when its consumer starts.  Same kernels on fewer rows: the result is bit
// for bit the unchunked one.  The price is launches (chunks x kernels per forward) and shorter grids.
constexpr long long kChunkTokens = 16384;   // padded tokens per sub-batch
bool uses_chunks(const rlx_encoder_config_t& c, int B, int S) {
    return (c.flags & RLX_FLAG_CHUNKED) && !(c.flags & RLX_FLAG_KERNEL_EVENTS) && S % 4 == 0 &&
           (long long)B * S > kChunkTokens && B > 1;
}
int chunk_batch(int B, int S) {
    const long long n_chunks = ((long long)B * S + kChunkTokens - 1) / kChunkTokens;
    return (int)((B + n_chunks - 1) / n_chunks);
}
rlx_status_t enqueue_forward_any(const rlx_encoder* e, const int32_t* ids, const int32_t* mask, int B, int S,
                                 const rlx_encoder_weights_t* w, float* out, unsigned char* ws, cudaStream_t st,
                                 bool capturing, bool with_events = true) {
    if (!uses_chunks(e->cfg, B, S)) return enqueue_forward(e, ids, mask, B, S, w, out, ws, st, capturing, with_events);
    const int bc = chunk_batch(B, S);
    struct WholeCall {
        explicit WholeCall(long long t) { g_whole_call_tokens = t; }
        ~WholeCall() { g_whole_call_tokens = 0; }
    } whole((long long)B * S);
    for (int b0 = 0; b0 < B; b0 += bc) {
        const int nb = std::min(bc, B - b0);
        rlx_status_t s = enqueue_forward(e, ids + (size_t)b0 * S, mask + (size_t)b0 * S, nb, S, w,
                                         out + (size_t)b0 * e->cfg.hidden, ws, st, capturing, false);
        if (s != RLX_OK) return s;
    }
    return RLX_OK;
}

// Tensor-parallel forward (Section 3.4: column / row sharding with an all-reduce inside the layer).
// Rank r of n holds heads r*h/n .. (r+1)*h/n - 1 of every layer: the rows of Wqkv that produce their q, k
// and v (column-parallel: no exchange), the matching COLUMNS of Wo (row-parallel: every rank forms a
// partial sum over its own heads), rows r*F/n .. of W1 and the matching columns of W2.  The two
// row-parallel products of a layer end in the caller's all-reduce; the residual and the bias enter the
// sum once, on rank 0 (the other ranks pass a zero bias vector).  Everything between two all-reduces
// is the single-GPU kernels on narrower operands; LayerNorm and pooling run replicated.  Eager
// launches only: the exchange is the caller's library call, not a node of a captured graph.
rlx_status_t enqueue_forward_tp(const rlx_encoder* e, const int32_t* ids, const int32_t* mask, int B, int S,
                                const rlx_encoder_weights_t* w, int tp_rank, int tp_size,
                                rlx_allreduce_bf16_fn allreduce, void* user, float* out, unsigned char* ws,
                                cudaStream_t st) {
    const rlx_encoder_config_t& c = e->cfg;
    const int H = c.hidden, F = c.ffn, T = B * S, d = e->head_dim;
    const int h_loc = c.num_heads / tp_size, H_loc = h_loc * d, F_loc = F / tp_size;
    const Arena a = plan_arena(B, S, H, F, c.num_layers, false);
    int32_t* status = reinterpret_cast<int32_t*>(ws + a.status);
    bf16* x = reinterpret_cast<bf16*>(ws + a.x);
    bf16* qkv = reinterpret_cast<bf16*>(ws + a.qkv);
    bf16* ctx = reinterpret_cast<bf16*>(ws + a.ctx);
    bf16* y = reinterpret_cast<bf16*>(ws + a.y);
    bf16* x1 = reinterpret_cast<bf16*>(ws + a.x1);
    bf16* g = reinterpret_cast<bf16*>(ws + a.g);
    rlx_status_t s;
#define RLX_TP_TRY(call) do { s = (call); if (s != RLX_OK) return s; } while (0)
    Packing pk;
    {
        int32_t* seq_len = reinterpret_cast<int32_t*>(ws + a.seq_len);
        int32_t* seq_start = reinterpret_cast<int32_t*>(ws + a.seq_start);
        int32_t* pos_of_rank = reinterpret_cast<int32_t*>(ws + a.pos_of_rank);
        RLX_TP_TRY(launch_pack(mask, B, S, seq_len, seq_start, pos_of_rank,
                               reinterpret_cast<unsigned int*>(ws + a.status + kTicketOffset), st));
        pk.seq_len = seq_len; pk.seq_start = seq_start; pk.pos_of_rank = pos_of_rank; pk.B = B;
    }
    const int32_t* rows = pk.total();
    // the partial sums of all T rows are exchanged: the number of packed rows is known on the device only,
    // and rows past it are never read
    const size_t exchange = (size_t)T * H;
    const int row_epi = tp_rank == 0 ? RLX_EPI_BIAS_RESIDUAL : RLX_EPI_BIAS;
    RLX_TP_TRY(launch_embed_ln(ids, (const bf16*)w->word_emb, (const bf16*)w->pos_emb, (const bf16*)w->type_emb,
                               w->emb_ln_g, w->emb_ln_b, T, S, H, c.vocab, c.ln_eps, x, status, st, pk));
    for (int l = 0; l < c.num_layers; ++l) {
        const rlx_layer_weights_t& lw = w->layers[l];
        RLX_TP_TRY(launch_gemm(x, (const bf16*)lw.wqkv, lw.bqkv, nullptr, RLX_EPI_BIAS, T, 3 * H_loc, H, qkv, false, status, st, rows));
        RLX_TP_TRY(launch_attention_bf16(qkv, mask, pk.seq_start, pk.seq_len, B, S, h_loc, d, ctx, st));
        RLX_TP_TRY(launch_gemm(ctx, (const bf16*)lw.wo, lw.bo, tp_rank == 0 ? x : nullptr, row_epi, T, H, H_loc, y, false, status, st, rows));
        if (allreduce(user, y, exchange, st) != 0) return RLX_ERR_CUDA;
        RLX_TP_TRY(launch_layernorm(y, lw.ln1_g, lw.ln1_b, T, H, c.ln_eps, x1, st, rows));
        RLX_TP_TRY(launch_gemm(x1, (const bf16*)lw.w1, lw.b1, nullptr, RLX_EPI_BIAS_GELU, T, F_loc, H, g, false, status, st, rows));
        RLX_TP_TRY(launch_gemm(g, (const bf16*)lw.w2, lw.b2, tp_rank == 0 ? x1 : nullptr, row_epi, T, H, F_loc, y, false, status, st, rows));
        if (allreduce(user, y, exchange, st) != 0) return RLX_ERR_CUDA;
        RLX_TP_TRY(launch_layernorm(y, lw.ln2_g, lw.ln2_b, T, H, c.ln_eps, x, st, rows));
    }
    RLX_TP_TRY(launch_pool(x, mask, B, S, H, out, st, pk));
#undef RLX_TP_TRY
    return RLX_OK;
}

rlx_status_t check_forward_args(const rlx_encoder* e, const void* ids, const void* mask, int B, int S,
                                const rlx_encoder_weights_t* w, const void* out, const void* ws, size_t ws_bytes,
                                bool host_io) {
    if (!e || !ids || !mask || !w || !out || !ws) return RLX_ERR_INVALID_ARG;
    if (w->struct_size != sizeof(rlx_encoder_weights_t) || !w->layers) return RLX_ERR_INVALID_ARG;
    if (B <= 0 || S <= 0 || B > e->cfg.max_batch || S > e->cfg.max_seq) return RLX_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return RLX_ERR_INVALID_ARG;
    if (!host_io && (!aligned16(ids) || !aligned16(mask) || !aligned16(out))) return RLX_ERR_INVALID_ARG;
    const void* tabs[5] = {w->word_emb, w->pos_emb, w->type_emb, w->emb_ln_g, w->emb_ln_b};
    for (const void* p : tabs)
        if (!p || !aligned16(p)) return RLX_ERR_INVALID_ARG;
    for (int l = 0; l < e->cfg.num_layers; ++l) {
        const void* const* ptrs = reinterpret_cast<const void* const*>(&w->layers[l]);
        for (size_t i = 0; i < sizeof(rlx_layer_weights_t) / sizeof(void*); ++i)
            if (!ptrs[i] || !aligned16(ptrs[i])) return RLX_ERR_INVALID_ARG;
    }
    const Arena a = plan_arena(B, S, e->cfg.hidden, e->cfg.ffn, e->cfg.num_layers, uses_fold_ln(e->cfg, B, S));
    if (ws_bytes < a.total) return RLX_ERR_WORKSPACE;
    return RLX_OK;
}

// Device-side address of a pinned host buffer (nullptr when the memory is pageable or not mapped).
void* device_view_of_pinned(const void* host) {
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, host) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    if (attr.type != cudaMemoryTypeHost) return nullptr;
    return attr.devicePointer;
}

rlx_status_t forward_device(rlx_encoder* e, const int32_t* ids, const int32_t* mask, int B, int S,
                            const rlx_encoder_weights_t* w, float* out, unsigned char* ws, cudaStream_t st) {
    int dev = -1;
    RLX_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != e->cfg.device) return RLX_ERR_INVALID_ARG;   // the object is bound to one device; make it current
    RLX_CUDA_TRY(init_kernels_for_current_device());
    if ((e->cfg.flags & RLX_FLAG_KERNEL_EVENTS) && e->events.empty()) {
        e->events.resize(4 + 7 * (size_t)e->cfg.num_layers);   // upper bound: one per kernel + 1
        e->last_kernels = 0;
        for (auto& evt : e->events) RLX_CUDA_TRY(cudaEventCreate(&evt));
    }
    e->last_kernels = kernels_in_forward(e->cfg, B, S);
    if (e->cfg.flags & RLX_FLAG_NO_GRAPH) return enqueue_forward_any(e, ids, mask, B, S, w, out, ws, st, false);

    if (!same_weights(e, w)) {
        drop_graphs(e);
        e->weights = *w;
        e->layers.assign(w->layers, w->layers + e->cfg.num_layers);
        e->weights.layers = e->layers.data();
        e->have_weights = true;
    }
    for (const auto& g : e->graphs)
        if (g.B == B && g.S == S && g.ids == ids && g.mask == mask && g.out == out && g.ws == ws) {
            RLX_CUDA_TRY(cudaGraphLaunch(g.exec, st));
            return RLX_OK;
        }
    // capture once for this (batch, seq, pointer set)
    cudaGraph_t graph = nullptr;
    if (!e->capture_stream) RLX_CUDA_TRY(cudaStreamCreateWithFlags(&e->capture_stream, cudaStreamNonBlocking));
    if (!e->body_stream) RLX_CUDA_TRY(cudaStreamCreateWithFlags(&e->body_stream, cudaStreamNonBlocking));
    if (!e->side_stream) {
        RLX_CUDA_TRY(cudaStreamCreateWithFlags(&e->side_stream, cudaStreamNonBlocking));
        RLX_CUDA_TRY(cudaEventCreateWithFlags(&e->fork_event, cudaEventDisableTiming));
        RLX_CUDA_TRY(cudaEventCreateWithFlags(&e->join_event, cudaEventDisableTiming));
        RLX_CUDA_TRY(cudaEventCreateWithFlags(&e->fold_event, cudaEventDisableTiming));
    }
    RLX_CUDA_TRY(cudaStreamBeginCapture(e->capture_stream, cudaStreamCaptureModeThreadLocal));
    rlx_status_t s = enqueue_forward_any(e, ids, mask, B, S, &e->weights, out, ws, e->capture_stream, true);
    cudaError_t ce = cudaStreamEndCapture(e->capture_stream, &graph);
    if (s != RLX_OK) {
        if (graph) cudaGraphDestroy(graph);
        return s;
    }
    RLX_CUDA_TRY(ce);
    cudaGraphExec_t exec = nullptr;
    ce = cudaGraphInstantiate(&exec, graph, 0);
    cudaGraphDestroy(graph);
    RLX_CUDA_TRY(ce);
    if (e->graphs.size() >= 16) {  // bound the cache
        cudaGraphExecDestroy(e->graphs.front().exec);
        e->graphs.erase(e->graphs.begin());
    }
    e->graphs.push_back(GraphEntry{B, S, ids, mask, out, ws, exec});
    RLX_CUDA_TRY(cudaGraphLaunch(exec, st));
    return RLX_OK;
}

}  // namespace

// =================================================================== C ABI
extern "C" {

rlx_status_t rlx_encoder_create(const rlx_encoder_config_t* c, rlx_encoder_t** out) {
    if (!c || !out) return RLX_ERR_INVALID_ARG;
    *out = nullptr;
    if (c->struct_size != sizeof(rlx_encoder_config_t)) return RLX_ERR_INVALID_ARG;
    if (c->num_layers <= 0 || c->hidden <= 0 || c->num_heads <= 0 || c->ffn <= 0 || c->vocab <= 0 || c->max_pos <= 0 ||
        c->type_vocab <= 0 || c->max_batch <= 0 || c->max_seq <= 0 || c->device < 0 || !(c->ln_eps >= 0.f))
        return RLX_ERR_INVALID_ARG;
    if (c->hidden % 128 != 0 || c->hidden > 1024 || c->hidden % c->num_heads != 0) return RLX_ERR_UNSUPPORTED;
    const int d = c->hidden / c->num_heads;
    if ((d != 32 && d != 64) || c->ffn % 64 != 0 || c->max_seq > c->max_pos || c->max_seq > 512)
        return RLX_ERR_UNSUPPORTED;
    if ((long long)c->max_batch * c->max_seq > (1ll << 30) || c->max_batch > 65535) return RLX_ERR_UNSUPPORTED;
    rlx_encoder* e = new (std::nothrow) rlx_encoder();
    if (!e) return RLX_ERR_INVALID_ARG;
    e->cfg = *c;
    e->head_dim = d;
    *out = e;
    return RLX_OK;
}

void rlx_encoder_destroy(rlx_encoder_t* e) {
    if (!e) return;
    drop_graphs(e);
    if (e->capture_stream) cudaStreamDestroy(e->capture_stream);
    if (e->side_stream) cudaStreamDestroy(e->side_stream);
    if (e->body_stream) cudaStreamDestroy(e->body_stream);
    if (e->fork_event) cudaEventDestroy(e->fork_event);
    if (e->join_event) cudaEventDestroy(e->join_event);
    if (e->fold_event) cudaEventDestroy(e->fold_event);
    for (auto& evt : e->events) cudaEventDestroy(evt);
    delete e;
}

size_t rlx_encoder_workspace_bytes(const rlx_encoder_t* e, int32_t batch, int32_t seq) {
    if (!e || batch <= 0 || seq <= 0 || batch > e->cfg.max_batch || seq > e->cfg.max_seq) return 0;
    return plan_arena(batch, seq, e->cfg.hidden, e->cfg.ffn, e->cfg.num_layers, uses_fold_ln(e->cfg, batch, seq)).total;
}

int32_t rlx_encoder_kernels_per_forward(const rlx_encoder_t* e, int32_t batch, int32_t seq) {
    if (!e || batch <= 0 || seq <= 0) return 0;
    return kernels_in_forward(e->cfg, batch, seq);
}

rlx_status_t rlx_encoder_forward(rlx_encoder_t* e, const int32_t* ids, const int32_t* mask, int32_t B, int32_t S,
                                 const rlx_encoder_weights_t* w, float* out, void* ws, size_t ws_bytes, void* stream) {
    rlx_status_t s = check_forward_args(e, ids, mask, B, S, w, out, ws, ws_bytes, false);
    if (s != RLX_OK) return s;
    return forward_device(e, ids, mask, B, S, w, out, static_cast<unsigned char*>(ws), static_cast<cudaStream_t>(stream));
}

rlx_status_t rlx_encoder_forward_tp(rlx_encoder_t* e, const int32_t* ids, const int32_t* mask, int32_t B, int32_t S,
                                    const rlx_encoder_weights_t* w_shard, int32_t tp_rank, int32_t tp_size,
                                    rlx_allreduce_bf16_fn allreduce, void* allreduce_user, float* out, void* ws,
                                    size_t ws_bytes, void* stream) {
    rlx_status_t s = check_forward_args(e, ids, mask, B, S, w_shard, out, ws, ws_bytes, false);
    if (s != RLX_OK) return s;
    if (!allreduce || tp_size < 1 || tp_rank < 0 || tp_rank >= tp_size) return RLX_ERR_INVALID_ARG;
    const rlx_encoder_config_t& c = e->cfg;
    // every shard must still be whole heads and whole 64-wide contraction blocks
    if (c.num_heads % tp_size != 0 || (c.hidden / tp_size) % 64 != 0 || c.ffn % tp_size != 0 || (c.ffn / tp_size) % 64 != 0)
        return RLX_ERR_UNSUPPORTED;
    if (c.flags & (RLX_FLAG_GEMM_SIMT | RLX_FLAG_NO_PACK | RLX_FLAG_FOLD_LN)) return RLX_ERR_UNSUPPORTED;
    int dev = -1;
    RLX_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != c.device) return RLX_ERR_INVALID_ARG;
    RLX_CUDA_TRY(init_kernels_for_current_device());
    return enqueue_forward_tp(e, ids, mask, B, S, w_shard, tp_rank, tp_size, allreduce, allreduce_user, out,
                              static_cast<unsigned char*>(ws), static_cast<cudaStream_t>(stream));
}

rlx_status_t rlx_encoder_forward_host(rlx_encoder_t* e, const int32_t* ids_h, const int32_t* mask_h, int32_t B,
                                      int32_t S, const rlx_encoder_weights_t* w, float* out_h, void* ws,
                                      size_t ws_bytes, void* stream) {
    rlx_status_t s = check_forward_args(e, ids_h, mask_h, B, S, w, out_h, ws, ws_bytes, true);
    if (s != RLX_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char* base = static_cast<unsigned char*>(ws);
    const Arena a = plan_arena(B, S, e->cfg.hidden, e->cfg.ffn, e->cfg.num_layers, uses_fold_ln(e->cfg, B, S));
    int32_t* ids_d = reinterpret_cast<int32_t*>(base + a.ids);
    int32_t* mask_d = reinterpret_cast<int32_t*>(base + a.mask);
    float* out_d = reinterpret_cast<float*>(base + a.out);
    const size_t tok_bytes = (size_t)B * S * sizeof(int32_t);
    // Pinned (page-locked, mapped) host buffers are addressable from the device: the packing and embedding
    // kernels then read ids / mask, and the pooling kernel writes the embeddings, straight over the bus.
    // Three copy operations (each several microseconds of engine latency in stream order) disappear from
    // the call; the bytes that cross the bus are the same.
    const int32_t* ids_z = static_cast<const int32_t*>(device_view_of_pinned(ids_h));
    const int32_t* mask_z = static_cast<const int32_t*>(device_view_of_pinned(mask_h));
    float* out_z = static_cast<float*>(device_view_of_pinned(out_h));
    if (ids_z && mask_z && out_z && aligned16(ids_z) && aligned16(mask_z) && aligned16(out_z)) {
        s = forward_device(e, ids_z, mask_z, B, S, w, out_z, base, st);
        if (s != RLX_OK) return s;
    } else {
        RLX_CUDA_TRY(cudaMemcpyAsync(ids_d, ids_h, tok_bytes, cudaMemcpyHostToDevice, st));
        RLX_CUDA_TRY(cudaMemcpyAsync(mask_d, mask_h, tok_bytes, cudaMemcpyHostToDevice, st));
        s = forward_device(e, ids_d, mask_d, B, S, w, out_d, base, st);
        if (s != RLX_OK) return s;
        RLX_CUDA_TRY(cudaMemcpyAsync(out_h, out_d, (size_t)B * e->cfg.hidden * sizeof(float), cudaMemcpyDeviceToHost, st));
    }
    RLX_CUDA_TRY(cudaStreamSynchronize(st));
    return RLX_OK;
}

rlx_status_t rlx_encoder_last_device_status(rlx_encoder_t* e, void* ws, void* stream) {
    if (!e || !ws) return RLX_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t word = 0;
    RLX_CUDA_TRY(cudaMemcpyAsync(&word, ws, sizeof(word), cudaMemcpyDeviceToHost, st));
    RLX_CUDA_TRY(cudaMemsetAsync(ws, 0, sizeof(word), st));
    RLX_CUDA_TRY(cudaStreamSynchronize(st));
    if (word & RLX_DEVSTAT_TIMEOUT) return RLX_ERR_DEVICE_TIMEOUT;
    if (word & RLX_DEVSTAT_TOKEN_RANGE) return RLX_ERR_TOKEN_RANGE;
    return RLX_OK;
}

rlx_status_t rlx_encoder_kernel_times(rlx_encoder_t* e, float* ms_host, int32_t count) {
    if (!e || !ms_host) return RLX_ERR_INVALID_ARG;
    if (e->events.empty() || e->last_kernels <= 0) return RLX_ERR_UNSUPPORTED;
    if (count != e->last_kernels) return RLX_ERR_INVALID_ARG;
    RLX_CUDA_TRY(cudaEventSynchronize(e->events[count]));
    for (int i = 0; i < count; ++i) RLX_CUDA_TRY(cudaEventElapsedTime(&ms_host[i], e->events[i], e->events[i + 1]));
    return RLX_OK;
}

const char* rlx_status_string(rlx_status_t s) {
    switch (s) {
        case RLX_OK: return "ok";
        case RLX_ERR_INVALID_ARG: return "invalid argument";
        case RLX_ERR_UNSUPPORTED: return "unsupported shape";
        case RLX_ERR_WORKSPACE: return "workspace too small";
        case RLX_ERR_CUDA: return "CUDA call failed";
        case RLX_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
        case RLX_ERR_TOKEN_RANGE: return "token id out of range (clamped)";
    }
    return "unknown status";
}

// ------------------------------------------------------------------- forward without a caller workspace
}  // extern "C"

// Scratch arena of rlx_encoder_forward_static.  It lives in the library's device image: every GPU
// that loads the library reserves these bytes until the process exits.  In host code the name
// below is only a stand-in for the symbol, not a device address; the address a kernel can use
// is obtained per device with cudaGetSymbolAddress (static_workspace_for_current_device).
static __device__ __align__(256) unsigned char g_static_workspace[RLX_STATIC_WORKSPACE_BYTES];

namespace {
// Resolves the device address of the static arena once per device (the device must be current).
rlx_status_t static_workspace_for_current_device(unsigned char** out) {
    static std::mutex mu;
    static unsigned char* addr[64] = {};
    int dev = 0;
    RLX_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return RLX_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lk(mu);
    if (!addr[dev]) {
        void* p = nullptr;
        RLX_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_workspace));
        if (!p) return RLX_ERR_CUDA;
        addr[dev] = static_cast<unsigned char*>(p);
    }
    *out = addr[dev];
    return RLX_OK;
}
}  // namespace

extern "C" {

rlx_status_t rlx_encoder_forward_static(rlx_encoder_t* e, const int32_t* ids, const int32_t* mask, int32_t B,
                                        int32_t S, const rlx_encoder_weights_t* w, float* out,
                                        int32_t* device_status, void* stream) {
    if (!e) return RLX_ERR_INVALID_ARG;
    // validate everything but the workspace with a stand-in pointer and size
    rlx_status_t s = check_forward_args(e, ids, mask, B, S, w, out, reinterpret_cast<void*>(uintptr_t(256)),
                                        ~size_t(0), false);
    if (s != RLX_OK) return s;
    struct NoAutoFold {
        NoAutoFold() { g_no_auto_fold = true; }
        ~NoAutoFold() { g_no_auto_fold = false; }
    } no_auto_fold;   // the 7-kernel layer unless RLX_FLAG_FOLD_LN asks for the folded one
    const Arena a = plan_arena(B, S, e->cfg.hidden, e->cfg.ffn, e->cfg.num_layers, uses_fold_ln(e->cfg, B, S));
    if (a.total > (size_t)RLX_STATIC_WORKSPACE_BYTES) return RLX_ERR_WORKSPACE;  // beyond the built-in arena
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int dev = -1;
    RLX_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != e->cfg.device) return RLX_ERR_INVALID_ARG;
    unsigned char* ws = nullptr;
    s = static_workspace_for_current_device(&ws);
    if (s != RLX_OK) return s;
    RLX_CUDA_TRY(init_kernels_for_current_device());
    // the arena keeps the previous call's bytes: the status word is the only part read before it is
    // written, so it alone is cleared; every activation row is rewritten by the kernels below
    RLX_CUDA_TRY(cudaMemsetAsync(ws + a.status, 0, sizeof(int32_t), st));
    // direct launches: no graph objects; and no event records even when an ordinary forward of this
    // object created its per-kernel events (they stay those of that forward)
    s = enqueue_forward(e, ids, mask, B, S, w, out, ws, st, false, false);
    if (s != RLX_OK) return s;
    if (device_status)
        RLX_CUDA_TRY(cudaMemcpyAsync(device_status, ws + a.status, sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
    return RLX_OK;
}

// ------------------------------------------------------------------- kernel-level entry points
rlx_status_t rlx_embed_layernorm(const int32_t* ids, const void* word, const void* pos, const void* type,
                                 const float* gamma, const float* beta, int32_t T, int32_t S, int32_t H, int32_t V,
                                 float eps, void* out, int32_t* status, void* stream) {
    if (!ids || !word || !pos || !type || !gamma || !beta || !out || T <= 0 || S <= 0 || V <= 0) return RLX_ERR_INVALID_ARG;
    if (H <= 0 || H % 128 != 0 || H > 1024) return RLX_ERR_UNSUPPORTED;
    if (!aligned16(word) || !aligned16(pos) || !aligned16(type) || !aligned16(gamma) || !aligned16(beta) || !aligned16(out))
        return RLX_ERR_INVALID_ARG;
    return launch_embed_ln(ids, (const bf16*)word, (const bf16*)pos, (const bf16*)type, gamma, beta, T, S, H, V, eps,
                           (bf16*)out, status, static_cast<cudaStream_t>(stream));
}

rlx_status_t rlx_pack_sequences(const int32_t* mask, int32_t B, int32_t S, int32_t* seq_len, int32_t* seq_start,
                                int32_t* pos_of_rank, uint32_t* ticket, void* stream) {
    if (!mask || !seq_len || !seq_start || !pos_of_rank || !ticket || B <= 0 || S <= 0) return RLX_ERR_INVALID_ARG;
    return launch_pack(mask, B, S, seq_len, seq_start, pos_of_rank, ticket, static_cast<cudaStream_t>(stream));
}

rlx_status_t rlx_layernorm(const void* x, const float* gamma, const float* beta, int32_t rows, int32_t H, float eps,
                           void* out, void* stream) {
    if (!x || !gamma || !beta || !out || rows <= 0) return RLX_ERR_INVALID_ARG;
    if (H <= 0 || H % 128 != 0 || H > 1024) return RLX_ERR_UNSUPPORTED;
    if (!aligned16(x) || !aligned16(gamma) || !aligned16(beta) || !aligned16(out)) return RLX_ERR_INVALID_ARG;
    return launch_layernorm((const bf16*)x, gamma, beta, rows, H, eps, (bf16*)out, static_cast<cudaStream_t>(stream));
}

rlx_status_t rlx_gemm_bf16(const void* A, const void* W, const float* bias, const void* residual, rlx_epilogue_t epi,
                           int32_t M, int32_t N, int32_t K, void* out, rlx_gemm_impl_t impl, int32_t* status,
                           void* stream) {
    if (!A || !W || !bias || !out || M <= 0 || N <= 0 || K <= 0) return RLX_ERR_INVALID_ARG;
    if ((int)epi < 0 || (int)epi > 2 || (epi == RLX_EPI_BIAS_RESIDUAL && !residual)) return RLX_ERR_INVALID_ARG;
    if (!aligned16(A) || !aligned16(W) || !aligned16(bias) || !aligned16(out) || (residual && !aligned16(residual)))
        return RLX_ERR_INVALID_ARG;
    if (N % 64 != 0 || K % 8 != 0) return RLX_ERR_UNSUPPORTED;
    if (impl != RLX_GEMM_TCGEN05 && impl != RLX_GEMM_SIMT && impl != RLX_GEMM_TCGEN05_PAIR &&
        impl != RLX_GEMM_TCGEN05_SINGLE && impl != RLX_GEMM_TCGEN05_RESIDENT)
        return RLX_ERR_INVALID_ARG;
    if (impl == RLX_GEMM_TCGEN05_PAIR && N % 128 != 0 && N % 192 != 0) return RLX_ERR_UNSUPPORTED;
    if (impl == RLX_GEMM_TCGEN05_RESIDENT && (K > 384 || (N % 128 != 0 && N % 192 != 0))) return RLX_ERR_UNSUPPORTED;
    RLX_CUDA_TRY(init_kernels_for_current_device());
    const int want_cg = impl == RLX_GEMM_TCGEN05_PAIR ? 2 : impl == RLX_GEMM_TCGEN05_SINGLE ? 1
                        : impl == RLX_GEMM_TCGEN05_RESIDENT ? 3 : 0;
    return launch_gemm((const bf16*)A, (const bf16*)W, bias, (const bf16*)residual, (int)epi, M, N, K, (bf16*)out,
                       impl == RLX_GEMM_SIMT, status, static_cast<cudaStream_t>(stream), nullptr, want_cg);
}

rlx_status_t rlx_gemm_residual_layernorm_bf16(const void* A, const void* W, const float* bias, const void* residual,
                                              const float* gamma, const float* beta, float eps, int32_t M, int32_t N,
                                              int32_t K, void* out, int32_t impl, int32_t* status, void* stream) {
    if (!A || !W || !bias || !residual || !gamma || !beta || !out || M <= 0 || N <= 0 || K <= 0) return RLX_ERR_INVALID_ARG;
    if (!aligned16(A) || !aligned16(W) || !aligned16(bias) || !aligned16(residual) || !aligned16(gamma) ||
        !aligned16(beta) || !aligned16(out))
        return RLX_ERR_INVALID_ARG;
    RLX_CUDA_TRY(init_kernels_for_current_device());
    if (impl == 0)
        return launch_gemm_cln((const bf16*)A, (const bf16*)W, bias, (const bf16*)residual, gamma, beta, eps, M, N, K,
                               (bf16*)out, status, static_cast<cudaStream_t>(stream));
    if (impl != 1) return RLX_ERR_INVALID_ARG;
    return launch_gemm_ln((const bf16*)A, (const bf16*)W, bias, (const bf16*)residual, gamma, beta, eps, M, N, K,
                          (bf16*)out, status, static_cast<cudaStream_t>(stream));
}

rlx_status_t rlx_attention_bf16(const void* qkv, const int32_t* mask, int32_t B, int32_t S, int32_t h, int32_t d,
                                void* ctx, void* stream) {
    if (!qkv || !mask || !ctx || B <= 0 || S <= 0 || h <= 0) return RLX_ERR_INVALID_ARG;
    if (!aligned16(qkv) || !aligned16(ctx)) return RLX_ERR_INVALID_ARG;
    if ((d != 32 && d != 64) || S > 512 || B > 65535 || h > 65535) return RLX_ERR_UNSUPPORTED;
    RLX_CUDA_TRY(init_kernels_for_current_device());
    return launch_attention_bf16((const bf16*)qkv, mask, nullptr, nullptr, B, S, h, d, (bf16*)ctx,
                                 static_cast<cudaStream_t>(stream));
}

rlx_status_t rlx_attention_packed_bf16(const void* qkv, int32_t rows, const int32_t* seq_start, const int32_t* seq_len,
                                       int32_t B, int32_t max_len, int32_t h, int32_t d, void* ctx, int32_t impl,
                                       int32_t* status, void* stream) {
    if (!qkv || !seq_start || !seq_len || !ctx || B <= 0 || max_len <= 0 || h <= 0 || rows <= 0) return RLX_ERR_INVALID_ARG;
    if (!aligned16(qkv) || !aligned16(ctx)) return RLX_ERR_INVALID_ARG;
    if ((d != 32 && d != 64) || max_len > 512 || B > 65535 || h > 65535) return RLX_ERR_UNSUPPORTED;
    RLX_CUDA_TRY(init_kernels_for_current_device());
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (impl == 0)
        {
        // the kernel-level call owns no workspace: its work-item counter is a word inside the library
        // (zero between launches; calls on different streams of one device must therefore not overlap)
        unsigned int* ticket = nullptr;
        RLX_CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void**>(&ticket), g_attn_ticket_standalone));
        return launch_attention_tc((const bf16*)qkv, rows, seq_start, seq_len, B, max_len, h, d, (bf16*)ctx, ticket, status, st);
    }
    if (impl == 1)
        return launch_attention_bf16((const bf16*)qkv, nullptr, seq_start, seq_len, B, max_len, h, d, (bf16*)ctx, st);
    return RLX_ERR_INVALID_ARG;
}

rlx_status_t rlx_attention_kind_bf16(const void* qkv, int32_t rows, const int32_t* seq_start, const int32_t* seq_len,
                                     int32_t B, int32_t max_len, int32_t h, int32_t hkv, int32_t d, int32_t mask_kind,
                                     int32_t window, const float* rope_cos, const float* rope_sin, void* ctx,
                                     void* stream) {
    if (!qkv || !seq_start || !seq_len || !ctx || B <= 0 || max_len <= 0 || h <= 0 || rows <= 0) return RLX_ERR_INVALID_ARG;
    if (!aligned16(qkv) || !aligned16(ctx) || !aligned16(rope_cos) || !aligned16(rope_sin)) return RLX_ERR_INVALID_ARG;
    if ((rope_cos == nullptr) != (rope_sin == nullptr)) return RLX_ERR_INVALID_ARG;
    if (mask_kind != RLX_MASK_NONE && mask_kind != RLX_MASK_CAUSAL && mask_kind != RLX_MASK_SLIDING_WINDOW)
        return RLX_ERR_INVALID_ARG;
    if (mask_kind == RLX_MASK_SLIDING_WINDOW && window < 1) return RLX_ERR_INVALID_ARG;
    if (hkv <= 0 || h % hkv != 0) return RLX_ERR_INVALID_ARG;
    if ((d != 32 && d != 64 && d != 128) || max_len > RLX_ATTENTION_KIND_MAX_LEN || B > 65535 || h > 65535)
        return RLX_ERR_UNSUPPORTED;
    RLX_CUDA_TRY(init_kernels_for_current_device());
    const bool positional = mask_kind != RLX_MASK_NONE;
    const int w = mask_kind == RLX_MASK_SLIDING_WINDOW ? window : (1 << 30);   // causal: the window never cuts
    return launch_attention_bf16((const bf16*)qkv, nullptr, seq_start, seq_len, B, max_len, h, d, (bf16*)ctx,
                                 static_cast<cudaStream_t>(stream), positional, w, rope_cos, rope_sin, h / hkv);
}

rlx_status_t rlx_qk_rope_bf16(void* qkv, int32_t rows, const int32_t* seq_start, const int32_t* seq_len, int32_t B,
                              int32_t max_len, int32_t h, int32_t hkv, int32_t d, const float* rope_cos,
                              const float* rope_sin, void* stream) {
    if (!qkv || !seq_start || !seq_len || !rope_cos || !rope_sin || B <= 0 || max_len <= 0 || h <= 0 || rows <= 0)
        return RLX_ERR_INVALID_ARG;
    if (hkv <= 0 || h % hkv != 0) return RLX_ERR_INVALID_ARG;
    if (!aligned16(qkv) || !aligned16(rope_cos) || !aligned16(rope_sin)) return RLX_ERR_INVALID_ARG;
    if ((d != 32 && d != 64 && d != 128) || max_len > RLX_ATTENTION_KIND_MAX_LEN || B > 65535 || h > 65535)
        return RLX_ERR_UNSUPPORTED;
    dim3 grid((max_len + rlx::kRopeRows - 1) / rlx::kRopeRows, B);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (d == 32)
        rlx::qk_rope_kernel<32><<<grid, rlx::kRopeThreads, 0, st>>>((bf16*)qkv, seq_start, seq_len, h + hkv, (h + 2 * hkv) * d,
                                                                    rope_cos, rope_sin);
    else if (d == 64)
        rlx::qk_rope_kernel<64><<<grid, rlx::kRopeThreads, 0, st>>>((bf16*)qkv, seq_start, seq_len, h + hkv, (h + 2 * hkv) * d,
                                                                    rope_cos, rope_sin);
    else
        rlx::qk_rope_kernel<128><<<grid, rlx::kRopeThreads, 0, st>>>((bf16*)qkv, seq_start, seq_len, h + hkv, (h + 2 * hkv) * d,
                                                                     rope_cos, rope_sin);
    RLX_CUDA_TRY(cudaGetLastError());
    return RLX_OK;
}

rlx_status_t rlx_rope_tables(int32_t max_len, int32_t head_dim, double theta, float* rope_cos, float* rope_sin,
                             void* stream) {
    if (!rope_cos || !rope_sin || max_len <= 0 || !(theta > 0.0)) return RLX_ERR_INVALID_ARG;
    if (!aligned16(rope_cos) || !aligned16(rope_sin)) return RLX_ERR_INVALID_ARG;
    if ((head_dim != 32 && head_dim != 64 && head_dim != 128) || max_len > RLX_ATTENTION_KIND_MAX_LEN) return RLX_ERR_UNSUPPORTED;
    const long long n = (long long)max_len * (head_dim / 2);
    rlx::rope_tables_kernel<<<(unsigned)((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        rope_cos, rope_sin, max_len, head_dim / 2, theta);
    RLX_CUDA_TRY(cudaGetLastError());
    return RLX_OK;
}

namespace {
// format word: (ebits << 8) | (mbits << 4) | special, plus RLX_MINIFLOAT_PACKED4
rlx_status_t parse_minifloat(int32_t format, rlx::MiniFloatFormat* f, bool* packed4) {
    if (format < 0 || (format & ~0x1fff)) return RLX_ERR_INVALID_ARG;
    f->ebits = (format >> 8) & 0xf;
    f->mbits = (format >> 4) & 0xf;
    f->special = format & 0xf;
    *packed4 = (format & RLX_MINIFLOAT_PACKED4) != 0;
    if (f->ebits < 1 || f->special > 2) return RLX_ERR_INVALID_ARG;
    if (1 + f->ebits + f->mbits > (*packed4 ? 4 : 8)) return RLX_ERR_INVALID_ARG;
    return RLX_OK;
}
}  // namespace

rlx_status_t rlx_dequant_block_scaled_bf16(const void* codes, const void* scales, int32_t N, int32_t K, int32_t format,
                                           void* w_bf16, void* stream) {
    if (!codes || !scales || !w_bf16 || N <= 0 || K <= 0) return RLX_ERR_INVALID_ARG;
    if (!aligned16(codes) || !aligned16(w_bf16)) return RLX_ERR_INVALID_ARG;
    rlx::MiniFloatFormat f;
    bool packed4;
    const rlx_status_t fs = parse_minifloat(format, &f, &packed4);
    if (fs != RLX_OK) return fs;
    if (K % 32 != 0) return RLX_ERR_UNSUPPORTED;
    const long long tasks = (long long)N * (K / rlx::kDequantElemsPerThread);
    const int blocks = (int)std::min<long long>((tasks + rlx::kDequantThreads - 1) / rlx::kDequantThreads,
                                                (long long)sm_count() * 16);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (packed4)
        rlx::dequant_block_scaled_kernel<true><<<blocks, rlx::kDequantThreads, 0, st>>>(
            (const uint8_t*)codes, (const uint8_t*)scales, (bf16*)w_bf16, N, K, f);
    else
        rlx::dequant_block_scaled_kernel<false><<<blocks, rlx::kDequantThreads, 0, st>>>(
            (const uint8_t*)codes, (const uint8_t*)scales, (bf16*)w_bf16, N, K, f);
    RLX_CUDA_TRY(cudaGetLastError());
    return RLX_OK;
}

rlx_status_t rlx_scaled_matmul_bf16(const void* A, const void* codes, const void* scales, int32_t format,
                                    const float* bias, const void* residual, rlx_epilogue_t epi, int32_t M, int32_t N,
                                    int32_t K, void* w_scratch, void* out, int32_t* status, void* stream) {
    if (!A || !bias || !out || M <= 0) return RLX_ERR_INVALID_ARG;
    if ((int)epi < 0 || (int)epi > 2 || (epi == RLX_EPI_BIAS_RESIDUAL && !residual)) return RLX_ERR_INVALID_ARG;
    if (!aligned16(A) || !aligned16(bias) || !aligned16(out) || (residual && !aligned16(residual))) return RLX_ERR_INVALID_ARG;
    if (N > 0 && N % 64 != 0) return RLX_ERR_UNSUPPORTED;
    const rlx_status_t ds = rlx_dequant_block_scaled_bf16(codes, scales, N, K, format, w_scratch, stream);
    if (ds != RLX_OK) return ds;
    RLX_CUDA_TRY(init_kernels_for_current_device());
    return launch_gemm((const bf16*)A, (const bf16*)w_scratch, bias, (const bf16*)residual, (int)epi, M, N, K, (bf16*)out,
                       false, status, static_cast<cudaStream_t>(stream), nullptr, 0);
}

rlx_status_t rlx_selftest_bounded_wait(uint32_t budget_us, int32_t* status_word, uint64_t* waited_ns, void* stream) {
    if (!status_word || budget_us == 0 || budget_us > 100000u) return RLX_ERR_INVALID_ARG;   // at most 100 ms
    rlx::tc::bounded_wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(
        status_word, (unsigned long long)budget_us * 1000ull, reinterpret_cast<unsigned long long*>(waited_ns));
    RLX_CUDA_TRY(cudaGetLastError());
    return RLX_OK;
}

rlx_status_t rlx_attention_f32(const float* qkv, const int32_t* mask, int32_t B, int32_t S, int32_t h, int32_t d,
                               float* ctx, void* stream) {
    if (!qkv || !mask || !ctx || B <= 0 || S <= 0 || h <= 0) return RLX_ERR_INVALID_ARG;
    if ((d != 32 && d != 64) || B > 65535 || h > 65535) return RLX_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    dim3 grid((S + rlx::kAttF32Warps - 1) / rlx::kAttF32Warps, h, B);
    const float scale = 1.0f / sqrtf((float)d);
    if (d == 32)
        rlx::attention_f32_kernel<32><<<grid, rlx::kAttF32Warps * 32, 0, st>>>(qkv, mask, ctx, S, h * d, scale);
    else
        rlx::attention_f32_kernel<64><<<grid, rlx::kAttF32Warps * 32, 0, st>>>(qkv, mask, ctx, S, h * d, scale);
    RLX_CUDA_TRY(cudaGetLastError());
    return RLX_OK;
}

// element format of the block-scaled tensor-core path: only the two 8-bit grids
static int mx_element_format(int32_t format) {
    if (format == RLX_FMT_FP8_E4M3) return rlx::tcmx::kFmtE4M3;
    if (format == RLX_FMT_FP8_E5M2) return rlx::tcmx::kFmtE5M2;
    return -1;
}

rlx_status_t rlx_quantise_mx(const void* x_bf16, int32_t M, int32_t K, int32_t format, void* codes, void* scales,
                             void* stream) {
    if (!x_bf16 || !codes || !scales || M <= 0 || K <= 0) return RLX_ERR_INVALID_ARG;
    if (!aligned16(x_bf16) || !aligned16(codes)) return RLX_ERR_INVALID_ARG;
    const int fmt = mx_element_format(format);
    if (fmt < 0 || K % 32 != 0) return RLX_ERR_UNSUPPORTED;
    const long long blocks = (long long)M * (K / 32);
    const unsigned grid = (unsigned)((blocks + rlx::tcmx::kQuantThreads - 1) / rlx::tcmx::kQuantThreads);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (fmt == rlx::tcmx::kFmtE5M2)
        rlx::tcmx::quantise_mx_kernel<true><<<grid, rlx::tcmx::kQuantThreads, 0, st>>>((const bf16*)x_bf16, (uint8_t*)codes, (uint8_t*)scales, blocks);
    else
        rlx::tcmx::quantise_mx_kernel<false><<<grid, rlx::tcmx::kQuantThreads, 0, st>>>((const bf16*)x_bf16, (uint8_t*)codes, (uint8_t*)scales, blocks);
    RLX_CUDA_TRY(cudaGetLastError());
    return RLX_OK;
}

rlx_status_t rlx_mx_matmul_bf16(const void* a_codes, const void* a_scales, int32_t a_format, const void* w_codes,
                                const void* w_scales, int32_t w_format, const float* bias, int32_t M, int32_t N,
                                int32_t K, void* out, int32_t* status, void* stream) {
    if (!a_codes || !a_scales || !w_codes || !w_scales || !out || M <= 0 || N <= 0 || K <= 0) return RLX_ERR_INVALID_ARG;
    if (!aligned16(a_codes) || !aligned16(w_codes) || !aligned16(a_scales) || !aligned16(w_scales) || !aligned16(out) ||
        (bias && !aligned16(bias)))
        return RLX_ERR_INVALID_ARG;
    const int af = mx_element_format(a_format), wf = mx_element_format(w_format);
    if (af < 0 || wf < 0 || K % rlx::tcmx::kBlockK != 0 || (N % rlx::tcmx::kTileN != 0 && N % rlx::tcmx::wide::kTileNW != 0))
        return RLX_ERR_UNSUPPORTED;
    RLX_CUDA_TRY(init_kernels_for_current_device());
    const bool wide_tiles = N % rlx::tcmx::wide::kTileNW == 0;   // persistent 128 x 192 tiles when N allows
    CUtensorMap ta, tw;
    if (!make_tmap_u8(&ta, a_codes, (uint64_t)M, (uint64_t)K, rlx::tcmx::kTileM) ||
        !make_tmap_u8(&tw, w_codes, (uint64_t)N, (uint64_t)K, wide_tiles ? rlx::tcmx::wide::kTileNW : rlx::tcmx::kTileN))
        return RLX_ERR_CUDA;
    rlx::tcmx::MxParams p;
    p.sfa = (const uint8_t*)a_scales; p.sfw = (const uint8_t*)w_scales; p.bias = bias; p.out = (bf16*)out;
    p.M = M; p.N = N; p.K = K; p.a_fmt = af; p.w_fmt = wf; p.status = status;
    const long long m_tiles = (M + rlx::tcmx::kTileM - 1) / rlx::tcmx::kTileM;
    const long long tiles = m_tiles * (wide_tiles ? N / rlx::tcmx::wide::kTileNW : N / rlx::tcmx::kTileN);
    if (tiles > 0x7fffffffLL) return RLX_ERR_UNSUPPORTED;
    if (wide_tiles) {
        const unsigned grid = (unsigned)std::min<long long>(tiles, sm_count());
        CUtensorMap to;   // output chunks: 32 x 32 bf16 boxes with the 64-byte swizzle of the staging buffers
        if (!make_tmap(&to, out, (uint64_t)M, (uint64_t)N, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B)) return RLX_ERR_CUDA;
        rlx::tcmx::wide::gemm_mx192_tcgen05_kernel<<<grid, rlx::tcmx::wide::kThreadsW, rlx::tcmx::wide::kSmemBytesW,
                                                     static_cast<cudaStream_t>(stream)>>>(ta, tw, to, p);
    } else {
        rlx::tcmx::gemm_mx_tcgen05_kernel<<<(unsigned)tiles, rlx::tcmx::kThreads, rlx::tcmx::kSmemBytes,
                                            static_cast<cudaStream_t>(stream)>>>(ta, tw, p);
    }
    RLX_CUDA_TRY(cudaGetLastError());
    return RLX_OK;
}

rlx_status_t rlx_ffn_fused_bf16(const void* x, const void* w1, const float* b1, const void* w2, const float* b2,
                                const float* ln_gamma, const float* ln_beta, float ln_eps,
                                int32_t M, int32_t H, int32_t F, void* out, int32_t* status, void* stream) {
    if (!x || !w1 || !b1 || !w2 || !b2 || !out || M <= 0 || H <= 0 || F <= 0) return RLX_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(w1) || !aligned16(b1) || !aligned16(w2) || !aligned16(b2) || !aligned16(out))
        return RLX_ERR_INVALID_ARG;
    if ((ln_gamma == nullptr) != (ln_beta == nullptr) || !aligned16(ln_gamma) || !aligned16(ln_beta)) return RLX_ERR_INVALID_ARG;
    if (ln_gamma && !(ln_eps > 0.f)) return RLX_ERR_INVALID_ARG;
    if (!ffn_fused_supported(H, F)) return RLX_ERR_UNSUPPORTED;
    RLX_CUDA_TRY(init_kernels_for_current_device());
    return launch_ffn_fused((const bf16*)x, (const bf16*)w1, b1, (const bf16*)w2, b2, M, H, F, (bf16*)out, status,
                            static_cast<cudaStream_t>(stream), nullptr, ln_gamma, ln_beta, ln_eps);
}

rlx_status_t rlx_layer_tail_bf16(const void* ctx, const void* h, const void* wo, const float* bo, const float* ln1_gamma,
                                 const float* ln1_beta, const void* w1, const float* b1, const void* w2, const float* b2,
                                 const float* ln2_gamma, const float* ln2_beta, float ln_eps, int32_t M, int32_t H, int32_t F,
                                 void* out, int32_t* status, void* stream) {
    if (!ctx || !h || !wo || !bo || !ln1_gamma || !ln1_beta || !w1 || !b1 || !w2 || !b2 || !ln2_gamma || !ln2_beta || !out)
        return RLX_ERR_INVALID_ARG;
    if (M <= 0 || H <= 0 || F <= 0 || !(ln_eps > 0.f)) return RLX_ERR_INVALID_ARG;
    const void* ptrs[] = {ctx, h, wo, bo, ln1_gamma, ln1_beta, w1, b1, w2, b2, ln2_gamma, ln2_beta, out};
    for (const void* q : ptrs)
        if (!aligned16(q)) return RLX_ERR_INVALID_ARG;
    if (!ffn_fused_supported(H, F)) return RLX_ERR_UNSUPPORTED;
    RLX_CUDA_TRY(init_kernels_for_current_device());
    FfnPre pre{(const bf16*)h, (const bf16*)wo, bo, ln1_gamma, ln1_beta};
    return launch_ffn_fused((const bf16*)ctx, (const bf16*)w1, b1, (const bf16*)w2, b2, M, H, F, (bf16*)out, status,
                            static_cast<cudaStream_t>(stream), nullptr, ln2_gamma, ln2_beta, ln_eps, &pre);
}

rlx_status_t rlx_pool_l2norm(const void* x, const int32_t* mask, int32_t B, int32_t S, int32_t H, float* out,
                             void* stream) {
    if (!x || !mask || !out || B <= 0 || S <= 0) return RLX_ERR_INVALID_ARG;
    if (H <= 0 || H % 128 != 0 || H > 1024) return RLX_ERR_UNSUPPORTED;
    if (!aligned16(x)) return RLX_ERR_INVALID_ARG;
    return launch_pool((const bf16*)x, mask, B, S, H, out, static_cast<cudaStream_t>(stream));
}

#ifdef RLX_EXPERIMENTS
// Experiments build only (not declared in the header): 0 = CTA grouping, 1 = tile width, 2 = ablation bits
// of the GEMM kernels, 3 = A-resident kernel (-1 off, 0 automatic, 1 whenever it applies).
void rlx_experiment_set(int key, int value) {
    switch (key) {
        case 0: g_exp_cg = value; break;
        case 1: g_exp_bn = value; break;
        case 2: g_exp_debug = value; break;
        case 3: g_exp_resident = value; break;
    }
}
void rlx_experiment_trace(void* buf) { g_exp_trace = static_cast<unsigned long long*>(buf); }
int rlx_experiment_pairs(int resident) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (init_kernels_for_current_device() != cudaSuccess) return -1;
    return resident ? g_max_pairs_resident[dev] : g_max_pairs[dev];
}
#endif

}  // extern "C"
