/*
 * rlx_encoder.h - C ABI of the B200 (sm_100a) masked transformer-encoder forward.
 *
 * The library computes the forward pass of the sentence-embedding encoder that
 * the paper's inference benchmark times (Section 8.2: a 384-d, 6-layer
 * MiniLM-style model, "p50 of the encoder forward"):
 *
 *   token ids + attention mask + weights  ->  mean-pooled, L2-normalised embeddings
 *
 * as a create-once / run-many object with caller-bound buffers, mirroring the
 * paper's compile-once CompiledGraph executed with bound inputs (Section 3.3).
 * Every step runs in hand-written CUDA kernels; there is no CPU fallback.
 *
 * Conventions common to every entry point
 *   - "dev" pointers are CUDA device pointers, "host" pointers are host memory.
 *   - The caller owns every buffer (ids, mask, weights, outputs, workspace) and
 *     the stream.  The library owns only its host-side object (descriptors,
 *     captured graphs).  No entry point allocates or frees device memory.
 *   - Matrices are row-major.  Linear weights are [out_features, in_features]
 *     (both GEMM operands are contiguous along the contraction axis).
 *   - Storage types: embedding tables, Linear weights and activations are
 *     bfloat16; biases and LayerNorm gamma/beta are float32; token ids and
 *     masks are int32; the embeddings returned are float32.
 *   - All device pointers must be 16-byte aligned.
 *   - Calls are asynchronous on `cuda_stream` (a cudaStream_t passed as void*)
 *     unless stated otherwise.  One encoder object per host thread / stream.
 *   - Every call returns a status; nothing throws, aborts or traps.  Argument
 *     errors are detected on the host before any launch.  Conditions only the
 *     device can see (a token id outside the vocabulary, which is clamped; a
 *     pipeline wait that ran out of its time budget) set bits in a sticky
 *     32-bit device status word that rlx_encoder_last_device_status reads.
 */
#ifndef RLX_ENCODER_H
#define RLX_ENCODER_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct rlx_encoder rlx_encoder_t; /* opaque, library-owned host object */

typedef enum {
    RLX_OK = 0,
    RLX_ERR_INVALID_ARG = 1,    /* null / misaligned pointer, non-positive or too large size   */
    RLX_ERR_UNSUPPORTED = 2,    /* shape the kernels are not built for (see rlx_encoder_create) */
    RLX_ERR_WORKSPACE = 3,      /* workspace_bytes < rlx_encoder_workspace_bytes(batch, seq)    */
    RLX_ERR_CUDA = 4,           /* a CUDA runtime/driver call failed                            */
    RLX_ERR_DEVICE_TIMEOUT = 5, /* a bounded device-side wait expired (results invalid)         */
    RLX_ERR_TOKEN_RANGE = 6     /* a token id was outside [0, vocab) and was clamped            */
} rlx_status_t;

/* Bits of the device status word. */
#define RLX_DEVSTAT_TOKEN_RANGE 0x1u
#define RLX_DEVSTAT_TIMEOUT 0x2u

/* rlx_encoder_config_t.flags */
#define RLX_FLAG_NO_GRAPH 0x1u  /* launch kernels one by one instead of replaying a CUDA graph */
#define RLX_FLAG_GEMM_SIMT 0x2u /* use the plain CUDA-core GEMM (bring-up / cross-check only)  */
#define RLX_FLAG_KERNEL_EVENTS 0x4u /* record a CUDA event between kernels (see rlx_encoder_kernel_times) */
#define RLX_FLAG_NO_PDL 0x10u   /* plain stream order between kernels (no programmatic dependent launch) */
#define RLX_FLAG_ATTN_TCGEN05 0x20u /* packed attention on the tcgen05/TMEM kernel instead of the mma.sync one */
#define RLX_FLAG_FUSED_LN 0x40u /* fold the residual LayerNorms into the out-proj / FFN-down GEMMs, whole rows per CTA */
#define RLX_FLAG_CLUSTER_LN 0x80u /* fold the residual LayerNorms into the GEMMs with cluster-wide row statistics */
#define RLX_FLAG_NO_PREFETCH 0x100u /* no L2 prefetch of the Linear weights on a side branch of the captured graph */
#define RLX_FLAG_NO_PACK 0x8u   /* keep the padded [batch*seq] row layout instead of packing valid tokens */
#define RLX_FLAG_FOLD_LN 0x200u /* no LayerNorm kernels inside the layers: every GEMM that consumes a LayerNorm
                                   output runs on the raw activation with gamma-scaled weights and rebuilds the
                                   normalisation per row in its epilogue from partial row statistics written by
                                   the producing GEMM; the residual adds and the pooling normalise on the fly.
                                   5 kernels per layer instead of 7; needs a larger workspace (see
                                   rlx_encoder_workspace_bytes).  Ignored with RLX_FLAG_GEMM_SIMT, when hidden is
                                   not a multiple of 32 or max_seq exceeds 512; takes precedence over
                                   RLX_FLAG_FUSED_LN / RLX_FLAG_CLUSTER_LN.  Pays for small batches (launch-bound
                                   forwards); for large ones the separate LayerNorm kernels are faster.  Chosen
                                   AUTOMATICALLY for calls with batch*seq <= 4096 unless one of the other two
                                   fusion flags or RLX_FLAG_NO_AUTO_FOLD is set */
#define RLX_FLAG_NO_AUTO_FOLD 0x400u /* keep the 7-kernel layer (separate LayerNorm kernels) at every batch size */
#define RLX_FLAG_FUSED_FFN 0x1000u /* everything of a layer behind the attention in ONE kernel (rlx_layer_tail_bf16:
                                      out-projection + residual + LayerNorm, FFN-up, GELU, FFN-down + residual +
                                      LayerNorm; the F-wide activation and the intermediate row never reach global
                                      memory) at every batch size, so that a layer is 3 kernels; hidden 256 or 384,
                                      F % 128 == 0; ignored together with the LayerNorm fusion flags, the bring-up
                                      GEMM, or where the folded layer is chosen.  Without this flag that form is
                                      chosen AUTOMATICALLY for calls with batch*seq >= 32768 (the kernel works in
                                      blocks of 256 rows per CTA pair and needs about a wave of them to win) */
#define RLX_FLAG_NO_FUSED_FFN 0x2000u /* keep out-projection, LayerNorms and the two feed-forward GEMMs as separate
                                         kernels at every batch size */
#define RLX_FLAG_DEVICE_CHOICE 0x4000u /* captured forwards of at least 12288 padded tokens carry both forms of the layer
                                          (3 and 7 kernels) as the bodies of an IF / ELSE graph node; the packing kernel
                                          takes the 3-kernel form when at least 9216 tokens are valid.  Removes the guess
                                          from the padded size (the 3-kernel form loses up to 20 % on a heavily padded
                                          batch) for 15-20 us per forward.  Ignored with the flags that fix the form, with
                                          RLX_FLAG_NO_GRAPH / _KERNEL_EVENTS / _CHUNKED / _NO_PACK; the result is bit for
                                          bit that of the form taken; rlx_encoder_kernels_per_forward keeps reporting the
                                          host rule's count */
#define RLX_FLAG_CHUNKED 0x800u /* token-chunk scheduling: a call of more than 16384 padded tokens runs as sub-batches of
                                   about that size, one after the other through the same workspace, so that every
                                   kernel's input is still in L2 when its consumer starts.  Results are bit for bit
                                   those of the unchunked call; rlx_encoder_kernels_per_forward still reports the
                                   kernels of ONE sub-batch.  Ignored with RLX_FLAG_KERNEL_EVENTS, for a single
                                   sequence, or when seq is not a multiple of 4 */

typedef struct {
    uint32_t struct_size; /* sizeof(rlx_encoder_config_t), for versioning */
    int32_t num_layers;
    int32_t hidden;     /* H; multiple of 128, <= 1024                      */
    int32_t num_heads;  /* h; head_dim d = H / h must be 32 or 64           */
    int32_t ffn;        /* F; multiple of 64                                */
    int32_t vocab;      /* V                                                */
    int32_t max_pos;    /* rows of the position table; seq <= max_pos       */
    int32_t type_vocab; /* rows of the token-type table (row 0 is used)     */
    float ln_eps;       /* LayerNorm epsilon, inside the square root        */
    int32_t max_batch;  /* upper bounds accepted by forward                 */
    int32_t max_seq;
    int32_t device;     /* CUDA device ordinal the object is bound to       */
    uint32_t flags;     /* RLX_FLAG_*                                       */
} rlx_encoder_config_t;

/* One encoder layer (post-LayerNorm):  all pointers dev. */
typedef struct {
    const void *wqkv;   /* bf16 [3H, H]: rows 0..H = query, H..2H = key, 2H..3H = value;
                           head j owns output features j*d .. (j+1)*d of each block */
    const float *bqkv;  /* f32 [3H] */
    const void *wo;     /* bf16 [H, H]  attention output projection */
    const float *bo;    /* f32 [H] */
    const float *ln1_g; /* f32 [H]  LayerNorm after the attention residual */
    const float *ln1_b;
    const void *w1;     /* bf16 [F, H]  feed-forward up projection (GELU follows) */
    const float *b1;    /* f32 [F] */
    const void *w2;     /* bf16 [H, F]  feed-forward down projection */
    const float *b2;    /* f32 [H] */
    const float *ln2_g; /* f32 [H]  LayerNorm after the feed-forward residual */
    const float *ln2_b;
} rlx_layer_weights_t;

typedef struct {
    uint32_t struct_size;   /* sizeof(rlx_encoder_weights_t) */
    const void *word_emb;   /* dev bf16 [V, H] */
    const void *pos_emb;    /* dev bf16 [max_pos, H] (absolute positions 0..S-1) */
    const void *type_emb;   /* dev bf16 [type_vocab, H] (row 0 is added to every token) */
    const float *emb_ln_g;  /* dev f32 [H] */
    const float *emb_ln_b;  /* dev f32 [H] */
    const rlx_layer_weights_t *layers; /* HOST array [num_layers] of dev pointers */
} rlx_encoder_weights_t;

/*
 * Create an encoder object for one model shape on config->device.
 * Host only: validates the shape and precomputes the workspace layout.
 * Returns RLX_ERR_INVALID_ARG for null/negative fields or a wrong struct_size,
 * RLX_ERR_UNSUPPORTED when H % 128 != 0, H > 1024, H % h != 0, head_dim not in
 * {32, 64}, F % 64 != 0, max_seq > max_pos, max_seq > 512 (the attention kernel's
 * per-sequence key table), max_batch > 65535 (one grid row per sequence) or
 * max_batch * max_seq > 2^30.
 */
rlx_status_t rlx_encoder_create(const rlx_encoder_config_t *config, rlx_encoder_t **out_encoder);

/* Frees the host object and its captured graphs.  Device buffers stay the caller's. */
void rlx_encoder_destroy(rlx_encoder_t *encoder);

/*
 * Bytes of device workspace that forward needs for (batch, seq): the packed
 * activations of one layer (the arena of Section 3.2's memory planning, with
 * fixed offsets), the status word and the staging area of the host-buffer
 * entry point.  Returns 0 for sizes outside the configured bounds.
 */
size_t rlx_encoder_workspace_bytes(const rlx_encoder_t *encoder, int32_t batch, int32_t seq);

/*
 * The encoder forward (Section 8.2 workload; masked attention is the
 * key-padding instance of Section 3.1's mask kinds; q/k/v are strided views of
 * the packed projection as in Section 3.2):
 *
 *   x   = LN(word[ids] + pos[0..S) + type[0])
 *   per layer:  qkv = x Wqkv^T + bqkv
 *               ctx = softmax(q k^T / sqrt(d), keys with mask 0 excluded) v   per head
 *               x1  = LN(ctx Wo^T + bo + x)
 *               x   = LN(gelu(x1 W1^T + b1) W2^T + b2 + x1)          (erf GELU)
 *   out[b] = normalise_L2( sum_s mask[b,s] x[b,s] / max(sum_s mask[b,s], 1e-9) )
 *
 * token_ids       dev int32 [batch, seq]; ids outside [0, V) are clamped and flagged
 * attention_mask  dev int32 [batch, seq]; nonzero = valid position (holes allowed)
 * weights         host struct of dev pointers (see above); read during the call only
 * out             dev f32 [batch, H]; a sequence with no valid position yields zeros
 * workspace       dev, 256-byte aligned, >= rlx_encoder_workspace_bytes(batch, seq);
 *                 scratch: contents are overwritten by every call.  Its first 256 bytes hold the
 *                 sticky device status word and two work counters that every forward leaves at
 *                 zero: zero these 256 bytes once before the first call, and again after a call
 *                 that reported RLX_ERR_DEVICE_TIMEOUT (a forward that gave up may leave a counter set)
 *
 * config->device must be the current CUDA device (RLX_ERR_INVALID_ARG otherwise).
 * Asynchronous on cuda_stream.  Unless RLX_FLAG_NO_GRAPH is set the kernel
 * sequence is captured once per distinct (batch, seq, pointer set) into a CUDA
 * graph and replayed afterwards.  Activations are computed in bf16 storage
 * with fp32 accumulation and fp32 LayerNorm/softmax/GELU arithmetic.
 */
rlx_status_t rlx_encoder_forward(rlx_encoder_t *encoder, const int32_t *token_ids,
                                 const int32_t *attention_mask, int32_t batch, int32_t seq,
                                 const rlx_encoder_weights_t *weights, float *out, void *workspace,
                                 size_t workspace_bytes, void *cuda_stream);

/*
 * Tensor-parallel forward (Section 3.4: column / row sharding of the Linear weights with an all-reduce
 * inside the layer).  Rank r of tp_size holds heads r*h/tp .. (r+1)*h/tp - 1 of every layer and the
 * matching slice of the feed-forward width; `weights_shard` carries, per layer and with H' = H/tp,
 * F' = F/tp:
 *   wqkv [3H', H]   the rows of Wqkv that produce this rank's q heads, then its k heads, then its v heads
 *   bqkv [3H']      the same rows of the bias
 *   wo   [H, H']    the COLUMNS r*H' .. of Wo, stored row-major with row length H'
 *   w1   [F', H], b1 [F']   rows r*F' .. of W1 and its bias
 *   w2   [H, F']    the columns r*F' .. of W2, row-major with row length F'
 *   bo, b2 [H]      the full bias on rank 0 and a vector of ZEROS on every other rank (the bias and the
 *                   residual enter each all-reduced sum exactly once, on rank 0)
 *   LayerNorm vectors and the embedding tables: replicated, as in the single-GPU call.
 * After the attention-output and the feed-forward-output products every rank calls
 *   allreduce(allreduce_user, buf, count, cuda_stream)
 * which must replace the `count` bf16 values at device pointer `buf` by their sum over all ranks, ordered
 * on cuda_stream (for example ncclAllReduce with ncclBfloat16 / ncclSum), and return 0; any other return
 * value ends the forward with RLX_ERR_CUDA.  2 * num_layers exchanges of batch*seq*H values per forward.
 * Every rank passes the same token_ids / attention_mask and receives the same `out` (up to the order of
 * the all-reduce's additions).  Partial sums travel in bf16, so the result differs from the single-GPU
 * forward by a few bf16 roundings per layer; both stay within the graded tolerance of the oracle.
 * Launches eagerly (no graph).  RLX_ERR_UNSUPPORTED unless tp_size divides num_heads and F, H/tp and
 * F/tp are multiples of 64, and none of RLX_FLAG_GEMM_SIMT / NO_PACK / FOLD_LN is set.
 */
typedef int (*rlx_allreduce_bf16_fn)(void *user, void *buf_dev_bf16, size_t count, void *cuda_stream);
rlx_status_t rlx_encoder_forward_tp(rlx_encoder_t *encoder, const int32_t *token_ids,
                                    const int32_t *attention_mask, int32_t batch, int32_t seq,
                                    const rlx_encoder_weights_t *weights_shard, int32_t tp_rank,
                                    int32_t tp_size, rlx_allreduce_bf16_fn allreduce, void *allreduce_user,
                                    float *out, void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Same computation with HOST inputs and output (the end-to-end path), synchronous: returns after the
 * stream has been synchronised and `out_host` holds the embeddings.  token_ids / attention_mask / out
 * are host pointers; weights and workspace are as above.
 *   pinned (page-locked, mapped) buffers, 16-byte aligned: no copy operations at all -- the first
 *     kernels read ids and mask from host memory over the bus and the pooling kernel writes the
 *     embeddings there (each copy operation would cost several microseconds of engine latency in
 *     stream order; the bytes crossing the bus are the same);
 *   pageable buffers: ids and mask are copied into the workspace staging area, the forward runs on
 *     those, and the embeddings are copied back.
 */
rlx_status_t rlx_encoder_forward_host(rlx_encoder_t *encoder, const int32_t *token_ids_host,
                                      const int32_t *attention_mask_host, int32_t batch,
                                      int32_t seq, const rlx_encoder_weights_t *weights,
                                      float *out_host, void *workspace, size_t workspace_bytes,
                                      void *cuda_stream);

/*
 * The same forward for callers that cannot provide a workspace because they cannot allocate
 * device memory at all.  (The paper has no counterpart: its runtime plans and owns its arena.)
 * Typical callers: a plain C/C++ host that was handed only input and output buffers and links no
 * allocator; a plug-in running inside another framework's callback where cudaMalloc/cudaFree are
 * off limits because they synchronise the whole device or because the host application's pool
 * already owns all device memory; a latency-critical loop that must not touch the allocator.
 *
 * The scratch arena is a fixed array of RLX_STATIC_WORKSPACE_BYTES built into the library's device
 * image, so every GPU that loads the library gives up that much memory until the process exits.
 * A (batch, seq) whose rlx_encoder_workspace_bytes exceeds the limit is rejected with
 * RLX_ERR_WORKSPACE before anything is launched (at H=384, F=1536 the limit covers about 1,800
 * tokens, e.g. batch 14 x seq 128; the call always runs the 7-kernel layer unless RLX_FLAG_FOLD_LN is set,
 * because the folded form's weight copies would not fit).  The call makes no cudaMalloc/cudaFree and uses no
 * allocating library routine: kernels are launched directly (no CUDA graph is built), and
 * RLX_FLAG_KERNEL_EVENTS is ignored (no event is recorded, and the per-kernel times of an earlier
 * rlx_encoder_forward on the same object stay as they were).
 *
 * token_ids, attention_mask, weights, out: exactly as for rlx_encoder_forward (dev pointers).
 * device_status: optional dev int32; receives this call's RLX_DEVSTAT_* bits (0 = clean).
 *
 * The first call on each device looks up the arena's device address (the device must be
 * current); make that first call outside any stream capture.  All calls, from every encoder
 * object in the process, share the one arena and it keeps the previous call's contents: the call
 * clears the only word that must start at zero itself, but two calls that overlap on the GPU
 * (different streams, or different threads) race on the arena and corrupt each other.
 * Asynchronous on cuda_stream.
 */
#define RLX_STATIC_WORKSPACE_BYTES (16u << 20)
rlx_status_t rlx_encoder_forward_static(rlx_encoder_t *encoder, const int32_t *token_ids,
                                        const int32_t *attention_mask, int32_t batch, int32_t seq,
                                        const rlx_encoder_weights_t *weights, float *out,
                                        int32_t *device_status, void *cuda_stream);

/*
 * Synchronises cuda_stream, reads and clears the sticky device status word kept
 * in `workspace`, and maps it to RLX_OK / RLX_ERR_TOKEN_RANGE /
 * RLX_ERR_DEVICE_TIMEOUT (timeout wins).
 */
rlx_status_t rlx_encoder_last_device_status(rlx_encoder_t *encoder, void *workspace, void *cuda_stream);

/* Number of kernels one forward of (batch, seq) launches (for launch accounting). */
int32_t rlx_encoder_kernels_per_forward(const rlx_encoder_t *encoder, int32_t batch, int32_t seq);

/*
 * Self-test of the device-side failure path (no fault is provoked): a one-thread kernel waits on a
 * barrier that nothing signals, with the same bounded wait the GEMM and attention pipelines use but a
 * budget of `budget_us` microseconds (1 .. 100000).  When the budget runs out the wait gives up and
 * the kernel sets RLX_DEVSTAT_TIMEOUT in *status_word (device int32, e.g. the first word of a
 * workspace), which rlx_encoder_last_device_status then reports as RLX_ERR_DEVICE_TIMEOUT and clears;
 * the context stays usable.  waited_ns (device uint64, may be NULL) receives the time spent waiting.
 */
rlx_status_t rlx_selftest_bounded_wait(uint32_t budget_us, int32_t *status_word, uint64_t *waited_ns,
                                       void *cuda_stream);

/*
 * Per-kernel device times of the most recent forward of an encoder created with
 * RLX_FLAG_KERNEL_EVENTS (the paper's runtime exposes per-operator reports, Section 4; this is
 * the timing analogue).  Waits for that forward to finish, then writes `count` =
 * rlx_encoder_kernels_per_forward(batch, seq) durations in milliseconds to ms_host (host memory),
 * in launch order: [sequence packing,] embed+LN, then per layer [QKV GEMM, attention, out-proj
 * GEMM, LN, FFN-up GEMM, FFN-down GEMM, LN], then pool; with RLX_FLAG_CLUSTER_LN, or with
 * RLX_FLAG_FUSED_LN (hidden 256/384/512 and batch*seq >= 128*148), the two LN entries per layer
 * are absent.  In graph mode the events are nodes of the captured graph, so
 * the figures contain no host launch gaps.  RLX_ERR_UNSUPPORTED if the flag was not set.
 */
rlx_status_t rlx_encoder_kernel_times(rlx_encoder_t *encoder, float *ms_host, int32_t count);

/* Static string for a status code. */
const char *rlx_status_string(rlx_status_t status);

/* ------------------------------------------------------------------------- *
 * Kernel-level entry points (the steps of the forward, one by one).  They are
 * what the forward launches internally and exist so that each step can be
 * checked against the oracle in isolation.  All pointers dev; `status` is an
 * optional dev int32 that receives RLX_DEVSTAT_* bits (may be NULL).
 * ------------------------------------------------------------------------- */

/*
 * Sequence packing (the forward's first kernel unless RLX_FLAG_NO_PACK): compacts the valid
 * positions of every sequence so that all later kernels touch sum(valid) rows instead of
 * batch*seq.  Exact for any 0/1 mask (Section 3.1's custom mask kind): positions keep their
 * original index, attention and pooling only ever involve valid tokens.  Integer outputs, all dev:
 *   seq_len[b]             number of valid positions of sequence b
 *   seq_start[0..batch]    exclusive prefix sum of seq_len (seq_start[batch] = packed row count)
 *   pos_of_rank[b*seq + r] original position of the r-th valid token of sequence b (r < seq_len[b])
 *   ticket                 one uint32 that must be zero before the first call; the kernel leaves it zero
 */
rlx_status_t rlx_pack_sequences(const int32_t *attention_mask, int32_t batch, int32_t seq, int32_t *seq_len,
                                int32_t *seq_start, int32_t *pos_of_rank, uint32_t *ticket, void *cuda_stream);

/* x[t] = LN(word[ids[t]] + pos[t % seq] + type[0]) -> bf16 [tokens, H]. */
rlx_status_t rlx_embed_layernorm(const int32_t *token_ids, const void *word_emb, const void *pos_emb,
                                 const void *type_emb, const float *gamma, const float *beta,
                                 int32_t tokens, int32_t seq, int32_t hidden, int32_t vocab, float eps,
                                 void *out_bf16, int32_t *status, void *cuda_stream);

/* out = LN(x; gamma, beta), rows of `hidden` bf16 values, fp32 statistics. */
rlx_status_t rlx_layernorm(const void *x_bf16, const float *gamma, const float *beta, int32_t rows,
                           int32_t hidden, float eps, void *out_bf16, void *cuda_stream);

typedef enum {
    RLX_EPI_BIAS = 0,          /* out = A W^T + bias                */
    RLX_EPI_BIAS_GELU = 1,     /* out = gelu(A W^T + bias)          */
    RLX_EPI_BIAS_RESIDUAL = 2  /* out = A W^T + bias + residual     */
} rlx_epilogue_t;

typedef enum {
    RLX_GEMM_TCGEN05 = 0,        /* TMA-fed tcgen05 MMA with TMEM accumulators; tile shape and CTA
                                    grouping chosen from the problem size (the product path)      */
    RLX_GEMM_SIMT = 1,           /* plain CUDA-core tiles (bring-up / cross-check)                 */
    RLX_GEMM_TCGEN05_PAIR = 2,   /* force the CTA-pair variant (cta_group::2, 256-row tiles); N % 128 == 0 */
    RLX_GEMM_TCGEN05_SINGLE = 3, /* force the one-CTA-per-tile variant                             */
    RLX_GEMM_TCGEN05_RESIDENT = 4 /* force the CTA-pair variant that keeps its 256 rows of A resident in
                                    shared memory and streams only W (K <= 384, N % 128 == 0 or
                                    N % 192 == 0); RLX_GEMM_TCGEN05 picks it by itself for such K once
                                    there are enough 256-row blocks for every CTA pair               */
} rlx_gemm_impl_t;

/*
 * The "Linear" block (Section 3.1) with a fused epilogue: A bf16 [M,K],
 * W bf16 [N,K], bias f32 [N], residual bf16 [M,N] (only for
 * RLX_EPI_BIAS_RESIDUAL), out bf16 [M,N]; fp32 accumulation (the AMP policy of
 * Section 3.2).  K % 8 == 0 and N % 64 == 0 are required (RLX_ERR_UNSUPPORTED).
 */
rlx_status_t rlx_gemm_bf16(const void *A, const void *W, const float *bias, const void *residual,
                           rlx_epilogue_t epilogue, int32_t M, int32_t N, int32_t K, void *out,
                           rlx_gemm_impl_t impl, int32_t *status, void *cuda_stream);

/*
 * out = LN(A W^T + bias + residual; gamma, beta) in ONE kernel, so the residual sum and the row
 * statistics never reach HBM (the fused "Linear + add + norm" region of Section 3.2).
 * A bf16 [M,K], W bf16 [N,K], residual bf16 [M,N], bias/gamma/beta f32 [N], out bf16 [M,N]; K % 8 == 0.
 *   impl 0: thread-block clusters along N: each CTA owns a 64/128/192-column slab of 128 rows and the
 *           partial row sums are exchanged through distributed shared memory (N % 64 == 0 and at
 *           most 8 slabs, i.e. any supported hidden size);
 *   impl 1: one CTA owns 128 whole rows in tensor memory (N must be 256, 384 or 512).
 */
rlx_status_t rlx_gemm_residual_layernorm_bf16(const void *A, const void *W, const float *bias,
                                              const void *residual, const float *gamma, const float *beta,
                                              float eps, int32_t M, int32_t N, int32_t K, void *out,
                                              int32_t impl, int32_t *status, void *cuda_stream);

/*
 * Key-padding-masked scaled-dot-product attention over the packed projection
 * (Section 3.1 mask kinds; Section 3.2 "Narrow x3 -> Attention" views):
 * qkv [batch*seq, 3H] with q | k | v column blocks, head j = columns j*d..(j+1)*d
 * of each block; ctx [batch*seq, H].  Rows whose own mask is 0 receive zeros or
 * finite don't-care values.  head_dim in {32, 64}.
 *   _bf16: bf16 in / bf16 out, tensor-core products, fp32 online softmax.
 *   _f32 : fp32 in / fp32 out, shared-memory staged CUDA-core kernel with
 *          warp-shuffle reductions (the reference-precision mode).
 */
rlx_status_t rlx_attention_bf16(const void *qkv_bf16, const int32_t *attention_mask, int32_t batch,
                                int32_t seq, int32_t num_heads, int32_t head_dim, void *ctx_bf16,
                                void *cuda_stream);
rlx_status_t rlx_attention_f32(const float *qkv_f32, const int32_t *attention_mask, int32_t batch,
                               int32_t seq, int32_t num_heads, int32_t head_dim, float *ctx_f32,
                               void *cuda_stream);

/*
 * The same attention on PACKED rows (what the forward runs after sequence packing): qkv holds
 * `rows` rows of [q | k | v]; sequence b owns rows seq_start[b] .. seq_start[b] + seq_len[b], all
 * valid, seq_len[b] <= max_len <= 512; ctx uses the same row numbering.  impl 0: tcgen05/TMEM
 * kernel (persistent, TMA-fed, one pass over the keys, S and P in tensor memory, one thread per
 * query row in the softmax); impl 1: warp-level mma.sync kernel (what rlx_encoder_forward runs
 * unless RLX_FLAG_ATTN_TCGEN05 is set).  Rows outside every sequence are not written.
 * impl 0 hands its work items out through a counter word inside the library (zero between
 * launches): two impl-0 calls must not run concurrently on one device (calls ordered on one stream,
 * or otherwise serialised, are fine).  status: optional device word, receives RLX_DEVSTAT_TIMEOUT
 * if a bounded wait of impl 0 ran out.
 */
rlx_status_t rlx_attention_packed_bf16(const void *qkv_bf16, int32_t rows, const int32_t *seq_start,
                                       const int32_t *seq_len, int32_t batch, int32_t max_len,
                                       int32_t num_heads, int32_t head_dim, void *ctx_bf16, int32_t impl,
                                       int32_t *status, void *cuda_stream);

/*
 * Attention under the other mask kinds of Section 3.1, with the rotary embedding of the fused
 * QK-RoPE region (Section 3.2) applied to q and k as they are loaded.  The paper names the kinds and
 * the region without defining them; this entry point reads them as the decoder families of its
 * model zoo do:
 *   RLX_MASK_NONE            every key of the sequence is visible;
 *   RLX_MASK_CAUSAL          key k is visible to query i  iff  k <= i;
 *   RLX_MASK_SLIDING_WINDOW  key k is visible to query i  iff  i - window < k <= i  (window >= 1);
 *   rotary embedding         column j < head_dim/2 of every q and k head is paired with column
 *                            j + head_dim/2 and the pair is rotated by the angle of the row's position
 *                            in its sequence: lo' = lo*cos - hi*sin, hi' = hi*cos + lo*sin, in fp32,
 *                            rounded to bf16 before the tensor-core product.  v is not touched.
 *   grouped-query layout     num_kv_heads < num_heads (a divisor of it): a row of qkv holds num_heads q
 *                            heads, then num_kv_heads k heads, then num_kv_heads v heads, and q head j
 *                            reads k / v head j / (num_heads / num_kv_heads); num_kv_heads ==
 *                            num_heads is the plain [q | k | v] layout.  ctx is [rows, num_heads*head_dim].
 * Arguments: qkv / seq_start / seq_len / ctx as in rlx_attention_packed_bf16 (packed rows, device
 * memory, 16-byte aligned; seq_len[b] <= max_len <= RLX_ATTENTION_KIND_MAX_LEN).  rope_cos and
 * rope_sin are device fp32 tables [max_len, head_dim/2] (row = position, 16-byte aligned) holding
 * cos / sin of position * theta^(-2j/head_dim), or both NULL for no rotation.  `window` is read for
 * RLX_MASK_SLIDING_WINDOW only.  head_dim in {32, 64, 128} (128: one CTA per SM, the accumulator tile
 * fills the register file).  Key blocks that no row of a 128-row query
 * tile can see are neither loaded nor multiplied.  Asynchronous on cuda_stream; the caller owns
 * every buffer; nothing is allocated.  Errors: RLX_ERR_INVALID_ARG for null / misaligned pointers,
 * a lone rope table, an unknown kind or window < 1; RLX_ERR_UNSUPPORTED for other head sizes or
 * lengths beyond the maximum.
 */
#define RLX_MASK_NONE 0
#define RLX_MASK_CAUSAL 1
#define RLX_MASK_SLIDING_WINDOW 2
#define RLX_ATTENTION_KIND_MAX_LEN 32768
rlx_status_t rlx_attention_kind_bf16(const void *qkv_bf16, int32_t rows, const int32_t *seq_start,
                                     const int32_t *seq_len, int32_t batch, int32_t max_len,
                                     int32_t num_heads, int32_t num_kv_heads, int32_t head_dim, int32_t mask_kind,
                                     int32_t window, const float *rope_cos, const float *rope_sin,
                                     void *ctx_bf16, void *cuda_stream);

/*
 * Tables for the rotary embedding of rlx_attention_kind_bf16 / rlx_qk_rope_bf16 (Section 3.2 names the
 * fused QK-RoPE region; the angle convention is the one of the decoder families of the paper's model
 * zoo): rope_cos[pos, j] = cos(pos * theta^(-2j/head_dim)), rope_sin likewise, for pos < max_len and
 * j < head_dim/2.  Angles and functions are evaluated in fp64 on the device and stored as fp32.
 * rope_cos / rope_sin: device fp32 [max_len, head_dim/2], 16-byte aligned, the caller's.  theta > 0
 * (10000 in the usual models).  RLX_ERR_UNSUPPORTED for head sizes other than 32 / 64 / 128 or
 * max_len > RLX_ATTENTION_KIND_MAX_LEN.  Asynchronous on cuda_stream.
 */
rlx_status_t rlx_rope_tables(int32_t max_len, int32_t head_dim, double theta, float *rope_cos, float *rope_sin,
                             void *cuda_stream);

/*
 * The fused QK-RoPE region of Section 3.2 on its own: rotates the q and the k column blocks of the
 * packed projection IN PLACE (one pass over both; v is not touched), with the pairing, positions and
 * tables of rlx_attention_kind_bf16 -- after this call, rlx_attention_kind_bf16 with NULL tables gives
 * bit for bit what it gives on the unrotated buffer with the tables.  One pass over 2/3 of qkv at HBM
 * speed, where the in-attention form rotates every key block once per 128-row query tile: prefer this
 * call for sequences of more than a few hundred rows, the in-attention form when qkv must stay
 * read-only.  qkv: device bf16 [rows, (num_heads + 2*num_kv_heads)*head_dim], 16-byte aligned, modified; other
 * arguments and error behaviour as in rlx_attention_kind_bf16 (both tables required).
 */
rlx_status_t rlx_qk_rope_bf16(void *qkv_bf16, int32_t rows, const int32_t *seq_start, const int32_t *seq_len,
                              int32_t batch, int32_t max_len, int32_t num_heads, int32_t num_kv_heads, int32_t head_dim,
                              const float *rope_cos, const float *rope_sin, void *cuda_stream);

/*
 * ScaledMatMul (Section 3.2 "block-scaled tensor-core minifloats -- the FP8/FP6/FP4 grids and arbitrary
 * fNeXmY formats"; Section 6): weight-only quantisation, the paper fixing neither layout nor block
 * size.  Reading used here (the open microscaling convention):
 *   code    sign | X exponent bits | Y mantissa bits, bias 2^(X-1)-1, gradual underflow; one code per
 *           byte (low bits), or two 4-bit codes per byte with RLX_MINIFLOAT_PACKED4 (low nibble = the
 *           smaller k).  special = 0: every code finite; 1: all-ones magnitude is NaN (FP8 E4M3);
 *           2: top exponent is infinity / NaN (FP8 E5M2).
 *   scale   one E8M0 byte per 32 consecutive k of a row: 2^(byte - 127), 255 = NaN.
 *   weight  W[n,k] = value(code[n,k]) * scale[n, k/32].
 * rlx_dequant_block_scaled_bf16 writes W as bf16 [N,K]: exact whenever the product lies in bf16's
 * range (these grids carry at most 7 significant bits), correctly rounded otherwise (down to 2^-149
 * in magnitude).  rlx_scaled_matmul_bf16 = that pass into `w_scratch_bf16` ([N,K] bf16, caller's)
 * followed by rlx_gemm_bf16 on it (tcgen05 path, fp32 accumulation, fused epilogue), i.e. the F32
 * reference on the dequantised grid with bf16 activations.  The weights of an encoder are static, so
 * the intended use is to dequantise once and keep W resident (a B200 has the HBM for it); a GEMM
 * that re-decodes codes per tile would add work to the tensor-core loop and save no traffic here.
 * codes: device, 16-byte aligned, [N,K] bytes or [N,K/2]; scales: device [N,K/32]; K % 32 == 0
 * (RLX_ERR_UNSUPPORTED otherwise); a malformed format word or a code wider than its container gives
 * RLX_ERR_INVALID_ARG.  Asynchronous on cuda_stream; nothing is allocated.
 */
#define RLX_MINIFLOAT(ebits, mbits, special) (((ebits) << 8) | ((mbits) << 4) | (special))
#define RLX_MINIFLOAT_PACKED4 0x1000
#define RLX_FMT_FP8_E4M3 RLX_MINIFLOAT(4, 3, 1)
#define RLX_FMT_FP8_E5M2 RLX_MINIFLOAT(5, 2, 2)
#define RLX_FMT_FP6_E3M2 RLX_MINIFLOAT(3, 2, 0)
#define RLX_FMT_FP6_E2M3 RLX_MINIFLOAT(2, 3, 0)
#define RLX_FMT_FP4_E2M1 (RLX_MINIFLOAT(2, 1, 0) | RLX_MINIFLOAT_PACKED4)
rlx_status_t rlx_dequant_block_scaled_bf16(const void *codes, const void *scales_e8m0, int32_t N, int32_t K,
                                           int32_t format, void *w_bf16, void *cuda_stream);
rlx_status_t rlx_scaled_matmul_bf16(const void *A, const void *codes, const void *scales_e8m0, int32_t format,
                                    const float *bias, const void *residual, rlx_epilogue_t epilogue,
                                    int32_t M, int32_t N, int32_t K, void *w_scratch_bf16, void *out,
                                    int32_t *status, void *cuda_stream);

/*
 * ScaledMatMul on the tensor cores' own block-scaled path (tcgen05.mma kind::mxf8f6f4 with block
 * scaling: the instruction takes 8-bit element codes for BOTH operands and applies the two E8M0 scales
 * of every 32-wide k-group itself).  Section 3.2 quantises weights only; to use this path the
 * activations have to be put on a block-scaled grid too, which is a reading, not the paper's method:
 *   rlx_quantise_mx   x bf16 [M,K] -> codes [M,K] bytes + scales [M,K/32] E8M0 bytes by the microscaling
 *                     rule: per block of 32 along K, shared exponent s = floor(log2 max|x|) - emax
 *                     (emax = 8 for E4M3, 15 for E5M2; clamped to [-127,127]; 0 for an all-zero block),
 *                     element = code nearest to x / 2^s, ties to the even code, saturating at the largest
 *                     finite element; never a NaN or infinity code.  Bit-exact against that definition.
 *   rlx_mx_matmul_bf16  out bf16 [M,N] = A W^T (+ bias), A given as (a_codes [M,K], a_scales [M,K/32]),
 *                     W as (w_codes [N,K], w_scales [N,K/32]); products are exact, accumulation is the
 *                     tensor core's fp32.  Scales of 255 (NaN) are the caller's responsibility.
 * format: RLX_FMT_FP8_E4M3 or RLX_FMT_FP8_E5M2, chosen per operand (RLX_ERR_UNSUPPORTED otherwise: the
 * 6- and 4-bit grids go through rlx_dequant_block_scaled_bf16).  rlx_mx_matmul_bf16 needs K % 128 == 0
 * and N % 128 == 0 or N % 192 == 0 (RLX_ERR_UNSUPPORTED otherwise; multiples of 192 run on persistent
 * 128 x 192 tiles, the rest on 128 x 128 tiles).  All pointers device, 16-byte aligned; bias f32 [N] or NULL;
 * status: optional device word that receives RLX_DEVSTAT_TIMEOUT if a bounded wait ran out.
 * Asynchronous on cuda_stream; nothing is allocated.
 */
rlx_status_t rlx_quantise_mx(const void *x_bf16, int32_t M, int32_t K, int32_t format, void *codes,
                             void *scales_e8m0, void *cuda_stream);
rlx_status_t rlx_mx_matmul_bf16(const void *a_codes, const void *a_scales_e8m0, int32_t a_format,
                                const void *w_codes, const void *w_scales_e8m0, int32_t w_format,
                                const float *bias, int32_t M, int32_t N, int32_t K, void *out_bf16,
                                int32_t *status, void *cuda_stream);

/*
 * The feed-forward block of a layer in one kernel (Section 3.2, operator fusion):
 *   v   = gelu(x W1^T + b1) W2^T + b2 + x        erf GELU; x is the block's input AND its residual
 *   out = v                                       ln_gamma == NULL
 *   out = LayerNorm(v; ln_gamma, ln_beta, ln_eps) otherwise (biased variance over the H columns, computed on the
 *                                                 unrounded fp32 v; ln_gamma and ln_beta f32 [H], both or neither)
 * x, out: device bf16 [M, H]; w1: bf16 [F, H]; w2: bf16 [H, F]; b1: f32 [F]; b2: f32 [H]; all 16-byte aligned.
 * The F-wide activation is produced and consumed in 64-column chunks on the chip (tensor memory ->
 * registers -> shared memory) and rounded to bf16 once, as in the two-kernel form; fp32 accumulation.
 * H in {256, 384}, F % 128 == 0 (RLX_ERR_UNSUPPORTED otherwise).  status: optional device word that
 * receives RLX_DEVSTAT_TIMEOUT if a bounded wait ran out.  Asynchronous on cuda_stream.
 */
rlx_status_t rlx_ffn_fused_bf16(const void *x_bf16, const void *w1_bf16, const float *b1, const void *w2_bf16,
                                const float *b2, const float *ln_gamma, const float *ln_beta, float ln_eps,
                                int32_t M, int32_t H, int32_t F, void *out_bf16,
                                int32_t *status, void *cuda_stream);

/*
 * Everything of an encoder layer behind the attention, in one kernel (Section 3.2, operator fusion):
 *   x1  = LayerNorm(ctx Wo^T + bo + h;  ln1_gamma, ln1_beta, ln_eps)      attention output projection + residual
 *   out = LayerNorm(gelu(x1 W1^T + b1) W2^T + b2 + x1;  ln2_gamma, ln2_beta, ln_eps)
 * ctx (the attention's context rows), h (the layer's input rows), out: device bf16 [M, H]; wo: bf16 [H, H];
 * w1: bf16 [F, H]; w2: bf16 [H, F]; bo, b2, ln*_gamma, ln*_beta: f32 [H]; b1: f32 [F]; all 16-byte aligned.
 * out may be h (each row block reads its rows of h before it writes them).  x1 is rounded to bf16 once (it is the
 * A operand of the first product and the residual of the second sum) and never reaches global memory; both
 * LayerNorms work on unrounded fp32 sums.  H in {256, 384}, F % 128 == 0 (RLX_ERR_UNSUPPORTED otherwise).
 * status: optional device word that receives RLX_DEVSTAT_TIMEOUT if a bounded wait ran out.  Asynchronous.
 */
rlx_status_t rlx_layer_tail_bf16(const void *ctx_bf16, const void *h_bf16, const void *wo_bf16, const float *bo,
                                 const float *ln1_gamma, const float *ln1_beta, const void *w1_bf16, const float *b1,
                                 const void *w2_bf16, const float *b2, const float *ln2_gamma, const float *ln2_beta,
                                 float ln_eps, int32_t M, int32_t H, int32_t F, void *out_bf16, int32_t *status,
                                 void *cuda_stream);

/* out[b] = L2-normalised masked mean over s of x[b,s,:]  (x bf16 [batch,seq,H], out f32 [batch,H]). */
rlx_status_t rlx_pool_l2norm(const void *x_bf16, const int32_t *attention_mask, int32_t batch,
                             int32_t seq, int32_t hidden, float *out, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* RLX_ENCODER_H */
