/*
 * fp64 CPU oracle for the masked transformer-encoder forward pass.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA path is checked against.  It shares no code with the CUDA library and
 * must never be linked into, imported by, or called from the product path;
 * only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * What it follows.  The paper names the workload (Section 8.2: the 384-d,
 * 6-layer sentence-embedding encoder, p50 of the encoder forward) and the
 * primitive ("masked attention parameterized by MaskKind", Section 3.1; the
 * packed q/k/v "Narrow x3 -> Attention" view pattern, Section 3.2) but prints
 * no equations for the encoder.  The arithmetic below is therefore the
 * standard post-LayerNorm BERT-style encoder that the named model uses, with
 * these readings fixed:
 *   - embeddings: word[id] + position[s] (absolute, s = 0..S-1) + type[0], then LN
 *   - LayerNorm: biased variance, eps inside the square root
 *   - attention: scores scaled by 1/sqrt(d); keys with mask 0 are EXCLUDED
 *     (the key-padding mask is the "Custom" mask kind, one flag per key,
 *     broadcast over queries and heads); softmax over the remaining keys
 *   - GELU: exact erf form
 *   - pooling: masked mean (denominator clamped at 1e-9), then L2 normalise
 *     (norm clamped at 1e-12); a sequence with no valid token yields zeros
 *   - query rows with mask 0 never influence the output; they are skipped
 *     unless compute_all_rows is set (used for per-stage dumps)
 *
 * All arithmetic is IEEE double.  Parameters arrive as float (the values are
 * exactly representable: bf16-rounded matrices, fp32 vectors) and are widened
 * on read.  Loops are the textbook ones: no blocking, no fusion, no reordering.
 * OpenMP only distributes independent rows / (sequence, head, query) triples.
 *
 * Parity pins: every function here is pinned by tests/test_oracle_pins.py
 * (closed forms, brute force, invariants, library cross-checks).  Parity with
 * the TRAINED checkpoint of the named model is unpinned (weights unavailable).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int32_t num_layers, hidden, num_heads, ffn, vocab, max_pos, type_vocab;
    double ln_eps;
} oracle_config_t;

typedef struct {
    const float *wqkv, *bqkv, *wo, *bo, *ln1_g, *ln1_b, *w1, *b1, *w2, *b2, *ln2_g, *ln2_b;
} oracle_layer_t;

typedef struct {
    const float *word_emb, *pos_emb, *type_emb, *emb_ln_g, *emb_ln_b;
    const oracle_layer_t *layers;
} oracle_weights_t;

/* Optional per-stage dumps; any pointer may be NULL.  Per-layer buffers hold
 * num_layers consecutive [T, width] blocks. */
typedef struct {
    double *x_emb; /* [T,H]   after embedding LN            */
    double *qkv;   /* [L,T,3H] packed q,k,v                  */
    double *ctx;   /* [L,T,H] attention output               */
    double *x1;    /* [L,T,H] after first residual LN        */
    double *g;     /* [L,T,F] after GELU                     */
    double *x;     /* [L,T,H] layer output                   */
} oracle_dumps_t;

/* LN(v)_j = (v_j - mu) / sqrt(var + eps) * gamma_j + beta_j, biased variance. */
void rlx_oracle_layernorm(const double *v, const float *gamma, const float *beta, int64_t rows,
                          int H, double eps, double *out)
{
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        const double *x = v + r * H;
        double mu = 0.0;
        for (int j = 0; j < H; ++j) mu += x[j];
        mu /= H;
        double var = 0.0;
        for (int j = 0; j < H; ++j) var += (x[j] - mu) * (x[j] - mu);
        var /= H;
        double inv = 1.0 / sqrt(var + eps);
        for (int j = 0; j < H; ++j)
            out[r * H + j] = (x[j] - mu) * inv * (double)gamma[j] + (double)beta[j];
    }
}

/* Y[t,n] = sum_k X[t,k] * W[n,k] + bias[n]   (W is [out,in], the "Linear" block). */
void rlx_oracle_linear(const double *X, const float *W, const float *bias, int64_t T, int N, int K,
                       double *Y)
{
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t)
        for (int n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int k = 0; k < K; ++k) acc += X[t * K + k] * (double)W[(int64_t)n * K + k];
            Y[t * N + n] = acc + (bias ? (double)bias[n] : 0.0);
        }
}

/* gelu(u) = 0.5 u (1 + erf(u / sqrt 2)) */
void rlx_oracle_gelu(const double *u, int64_t n, double *out)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) out[i] = 0.5 * u[i] * (1.0 + erf(u[i] / sqrt(2.0)));
}

/*
 * Key-padding-masked scaled-dot-product attention on packed rows.
 * qkv: [B*S, 3H]; row t holds q (cols 0..H), k (H..2H), v (2H..3H); head j
 * owns columns j*d..(j+1)*d of each.  For query i of sequence b and head j:
 *   s_k = (q_i . k_k) / sqrt(d)      over keys k with mask[b,k] != 0 only
 *   p_k = exp(s_k - max s) / sum exp(s - max s)
 *   ctx_i = sum_k p_k v_k
 * probs (optional, [B,h,S,S]) receives p with zeros at masked keys.
 * Rows whose own mask is 0 are computed only if compute_all_rows; else zeroed.
 * A sequence with no valid key gives ctx = 0.
 */
void rlx_oracle_attention(const double *qkv, const int32_t *mask, int B, int S, int h, int d,
                          int compute_all_rows, double *ctx, double *probs)
{
    const int H = h * d;
    const double scale = 1.0 / sqrt((double)d);
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < B; ++b)
        for (int j = 0; j < h; ++j) {
            double *s = (double *)malloc(sizeof(double) * (size_t)S);
            for (int i = 0; i < S; ++i) {
                double *o = ctx + ((int64_t)b * S + i) * H + j * d;
                double *pr = probs ? probs + (((int64_t)b * h + j) * S + i) * S : NULL;
                for (int c = 0; c < d; ++c) o[c] = 0.0;
                if (pr) for (int k = 0; k < S; ++k) pr[k] = 0.0;
                if (!compute_all_rows && mask[b * S + i] == 0) continue;
                const double *q = qkv + ((int64_t)b * S + i) * 3 * H + j * d;
                double mx = -INFINITY;
                for (int k = 0; k < S; ++k) {
                    if (mask[b * S + k] == 0) continue;
                    const double *kk = qkv + ((int64_t)b * S + k) * 3 * H + H + j * d;
                    double acc = 0.0;
                    for (int c = 0; c < d; ++c) acc += q[c] * kk[c];
                    s[k] = acc * scale;
                    if (s[k] > mx) mx = s[k];
                }
                if (mx == -INFINITY) continue; /* no valid key */
                double den = 0.0;
                for (int k = 0; k < S; ++k)
                    if (mask[b * S + k] != 0) { s[k] = exp(s[k] - mx); den += s[k]; }
                for (int k = 0; k < S; ++k) {
                    if (mask[b * S + k] == 0) continue;
                    double p = s[k] / den;
                    if (pr) pr[k] = p;
                    const double *vv = qkv + ((int64_t)b * S + k) * 3 * H + 2 * H + j * d;
                    for (int c = 0; c < d; ++c) o[c] += p * vv[c];
                }
            }
            free(s);
        }
}

/* pool_b = sum_s [mask] x[b,s] / max(n_b, 1e-9); out_b = pool_b / max(||pool_b||, 1e-12) */
void rlx_oracle_pool_l2(const double *x, const int32_t *mask, int B, int S, int H, double *out)
{
    for (int b = 0; b < B; ++b) {
        double n = 0.0;
        for (int c = 0; c < H; ++c) out[(int64_t)b * H + c] = 0.0;
        for (int s = 0; s < S; ++s) {
            if (mask[b * S + s] == 0) continue;
            n += 1.0;
            for (int c = 0; c < H; ++c) out[(int64_t)b * H + c] += x[((int64_t)b * S + s) * H + c];
        }
        double den = n > 1e-9 ? n : 1e-9;
        double nrm = 0.0;
        for (int c = 0; c < H; ++c) {
            out[(int64_t)b * H + c] /= den;
            nrm += out[(int64_t)b * H + c] * out[(int64_t)b * H + c];
        }
        nrm = sqrt(nrm);
        if (nrm < 1e-12) nrm = 1e-12;
        for (int c = 0; c < H; ++c) out[(int64_t)b * H + c] /= nrm;
    }
}

/* e[t] = word[ids[t]] + pos[s] + type[0] */
void rlx_oracle_embed_sum(const oracle_config_t *cfg, const oracle_weights_t *w, const int32_t *ids,
                          int B, int S, double *e)
{
    const int H = cfg->hidden;
    for (int b = 0; b < B; ++b)
        for (int s = 0; s < S; ++s) {
            int64_t t = (int64_t)b * S + s;
            int64_t id = ids[t];
            for (int c = 0; c < H; ++c)
                e[t * H + c] = (double)w->word_emb[id * H + c] + (double)w->pos_emb[(int64_t)s * H + c] +
                               (double)w->type_emb[c];
        }
}

static void zero_masked_rows(double *a, const int32_t *mask, int64_t T, int width)
{
    for (int64_t t = 0; t < T; ++t)
        if (mask[t] == 0) memset(a + t * width, 0, sizeof(double) * (size_t)width);
}

/*
 * Whole encoder: ids, mask -> pooled, L2-normalised embeddings out[B,H].
 * Returns 0, or -1 on a bad argument (id out of range, S > max_pos, H % h != 0).
 */
int rlx_oracle_encoder_forward(const oracle_config_t *cfg, const oracle_weights_t *w,
                               const int32_t *ids, const int32_t *mask, int B, int S,
                               int compute_all_rows, double *out, const oracle_dumps_t *dumps)
{
    const int H = cfg->hidden, F = cfg->ffn, h = cfg->num_heads, L = cfg->num_layers;
    if (H % h != 0 || S > cfg->max_pos || B <= 0 || S <= 0) return -1;
    const int d = H / h;
    const int64_t T = (int64_t)B * S;
    for (int64_t t = 0; t < T; ++t)
        if (ids[t] < 0 || ids[t] >= cfg->vocab) return -1;

    double *x = (double *)malloc(sizeof(double) * T * H);
    double *tmp = (double *)malloc(sizeof(double) * T * H);
    double *x1 = (double *)malloc(sizeof(double) * T * H);
    double *ctx = (double *)malloc(sizeof(double) * T * H);
    double *qkv = (double *)malloc(sizeof(double) * T * 3 * H);
    double *u = (double *)malloc(sizeof(double) * T * F);
    double *g = (double *)malloc(sizeof(double) * T * F);

    /* step 1: embeddings + LN */
    rlx_oracle_embed_sum(cfg, w, ids, B, S, tmp);
    rlx_oracle_layernorm(tmp, w->emb_ln_g, w->emb_ln_b, T, H, cfg->ln_eps, x);
    if (!compute_all_rows) zero_masked_rows(x, mask, T, H);
    if (dumps && dumps->x_emb) memcpy(dumps->x_emb, x, sizeof(double) * T * H);

    for (int l = 0; l < L; ++l) {
        const oracle_layer_t *lw = &w->layers[l];
        /* 2a: packed q,k,v projection */
        rlx_oracle_linear(x, lw->wqkv, lw->bqkv, T, 3 * H, H, qkv);
        if (dumps && dumps->qkv) memcpy(dumps->qkv + (int64_t)l * T * 3 * H, qkv, sizeof(double) * T * 3 * H);
        /* 2b: masked attention on views of the packed buffer */
        rlx_oracle_attention(qkv, mask, B, S, h, d, compute_all_rows, ctx, NULL);
        if (dumps && dumps->ctx) memcpy(dumps->ctx + (int64_t)l * T * H, ctx, sizeof(double) * T * H);
        /* 2c: output projection + residual, LN */
        rlx_oracle_linear(ctx, lw->wo, lw->bo, T, H, H, tmp);
        for (int64_t i = 0; i < T * H; ++i) tmp[i] += x[i];
        rlx_oracle_layernorm(tmp, lw->ln1_g, lw->ln1_b, T, H, cfg->ln_eps, x1);
        if (!compute_all_rows) zero_masked_rows(x1, mask, T, H);
        if (dumps && dumps->x1) memcpy(dumps->x1 + (int64_t)l * T * H, x1, sizeof(double) * T * H);
        /* 2d: feed-forward with GELU + residual, LN */
        rlx_oracle_linear(x1, lw->w1, lw->b1, T, F, H, u);
        rlx_oracle_gelu(u, T * F, g);
        if (dumps && dumps->g) memcpy(dumps->g + (int64_t)l * T * F, g, sizeof(double) * T * F);
        rlx_oracle_linear(g, lw->w2, lw->b2, T, H, F, tmp);
        for (int64_t i = 0; i < T * H; ++i) tmp[i] += x1[i];
        rlx_oracle_layernorm(tmp, lw->ln2_g, lw->ln2_b, T, H, cfg->ln_eps, x);
        if (!compute_all_rows) zero_masked_rows(x, mask, T, H);
        if (dumps && dumps->x) memcpy(dumps->x + (int64_t)l * T * H, x, sizeof(double) * T * H);
    }
    /* step 3: masked mean pool + L2 normalise */
    rlx_oracle_pool_l2(x, mask, B, S, H, out);

    free(x); free(tmp); free(x1); free(ctx); free(qkv); free(u); free(g);
    return 0;
}
