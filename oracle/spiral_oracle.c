/*
 * spiral_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, obviously-correct CPU restatement of what one rollout-decoding step computes:
 * the policy pi_theta of Algorithm 1 (line "y_t ~ pi_theta(.|s_t, p, G_i)") evaluated one token at
 * a time for one game, followed by the Actor sampling rule of the hyperparameter table
 * (temperature 1.0, top-p 1.0, top-k -1: untruncated categorical sampling), realised as a
 * Gumbel-max draw with noise handed in by the caller.
 *
 * The paper names the model families (Qwen3, Llama-3.1, R1-Distill-Qwen; Section 4) and gives no
 * arithmetic for them; the decoder below is the standard pre-norm definition of those
 * architectures, written out step by step:
 *     x = E[token]
 *     per layer:  h = RMSNorm(x) g1 ; q,k,v = W h (+b) ; optional per-head RMSNorm of q,k ;
 *                 rotate-half RoPE at the token's absolute position ; append k,v to the game's
 *                 cache ; causal softmax attention with grouped KV heads ; x += Wo o ;
 *                 h = RMSNorm(x) g2 ; x += Wd ( SiLU(Wg h) * (Wu h) )
 *     logits = W_lm RMSNorm(x) g_f ;   token = argmax_v ( logits_v / T + gumbel_v )
 *
 * Rules this file keeps: every floating-point value is an IEEE double ("real"); weights arrive
 * as bf16 bit patterns and are widened exactly; there is no blocking, fusion or reordering
 * beyond the definition; OpenMP is used over independent output rows / heads for wall time
 * only (each output element is still one sequential sum).  The sampling decision is taken in
 * fp32 (z = fl32(logit) / T + gumbel, lowest index wins ties) because that is the precision the
 * decision is defined in for every implementation compared with this one.
 *
 * Nothing here is shared with the CUDA path: no headers, tables, constants or helpers.
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * Pins (tests/test_oracle_pins.py): library decoders of the same architectures (HF
 * transformers Qwen3 / Llama / Qwen2 on the CPU in fp64), torch's softmax / rms_norm / silu /
 * scaled_dot_product_attention, closed forms (zero-weight layers, single-key attention,
 * identical keys, 2-d rotation), invariants (RoPE relative position, norm preservation,
 * softmax shift invariance, paged == contiguous, decode == last row of prefill) and a
 * brute-force frequency check of the Gumbel-max sampler.  No function is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef double real;

typedef struct {
    int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ff, vocab;
    double rope_theta, rms_eps;
    int32_t qk_norm, qkv_bias, tied_embed;
} oracle_desc;

/* bf16 bit patterns, every matrix [out_features][in_features] row-major; per-layer arrays of
 * pointers.  bq/bk/bv may be NULL (no bias), q_norm/k_norm may be NULL (no q/k norm),
 * lm_head is ignored when tied_embed != 0. */
typedef struct {
    const uint16_t *embed, *lm_head, *final_norm;
    const uint16_t *const *ln1, *const *wq, *const *wk, *const *wv;
    const uint16_t *const *bq, *const *bk, *const *bv;
    const uint16_t *const *q_norm, *const *k_norm;
    const uint16_t *const *wo, *const *ln2, *const *w_gate, *const *w_up, *const *w_down;
} oracle_weights;

/* One game's K/V history.  page_size == 0: contiguous, position p lives at row p.
 * page_size > 0: position p lives in pool page block_table[p / page_size], slot p % page_size. */
typedef struct {
    int32_t n_layers, n_kv_heads, head_dim, max_ctx, len;
    int32_t page_size, n_rows;
    int32_t *block_table;
    real *k, *v; /* [layer][row][kv_head][head_dim] */
} oracle_cache;

static real widen(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (real)f;
}

/* round a real to the nearest bf16 (ties to even) and widen again; used only by the optional
 * "KV stored as bf16" bisecting switch */
static real round_bf16(real x)
{
    float f = (float)x;
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7fffffffu) > 0x7f800000u) return x; /* NaN */
    u += 0x7fffu + ((u >> 16) & 1u);
    u &= 0xffff0000u;
    memcpy(&f, &u, sizeof f);
    return (real)f;
}

/* ------------------------------------------------------------------------------------------ */
/* elementary pieces                                                                          */
/* ------------------------------------------------------------------------------------------ */

/* out_i = x_i * g_i / sqrt(mean(x^2) + eps); gain applied after normalisation, eps inside sqrt */
void oracle_rmsnorm(const real *x, const uint16_t *gain, double eps, int32_t n, real *out)
{
    real ss = 0;
    for (int32_t i = 0; i < n; ++i) ss += x[i] * x[i];
    real inv = 1.0 / sqrt(ss / n + eps);
    for (int32_t i = 0; i < n; ++i) out[i] = x[i] * inv * widen(gain[i]);
}

/* rotate-half RoPE in place on one head vector: pair (i, i + hd/2) turns by pos * theta^(-2i/hd) */
void oracle_rope(real *vec, int32_t head_dim, int32_t pos, double theta)
{
    int32_t half = head_dim / 2;
    for (int32_t i = 0; i < half; ++i) {
        double phi = (double)pos * pow(theta, -2.0 * i / head_dim);
        double c = cos(phi), s = sin(phi);
        real a = vec[i], b = vec[i + half];
        vec[i] = a * c - b * s;
        vec[i + half] = b * c + a * s;
    }
}

/* in-place softmax: subtract the maximum, exponentiate, divide by the sum */
void oracle_softmax(real *s, int32_t n)
{
    real m = s[0];
    for (int32_t i = 1; i < n; ++i) if (s[i] > m) m = s[i];
    real sum = 0;
    for (int32_t i = 0; i < n; ++i) { s[i] = exp(s[i] - m); sum += s[i]; }
    for (int32_t i = 0; i < n; ++i) s[i] /= sum;
}

real oracle_silu(real u) { return u / (1.0 + exp(-u)); }

/* y = W x (+ b), W bf16 [rows][cols] */
void oracle_matvec(const uint16_t *w, const uint16_t *bias, const real *x, int32_t rows,
                   int32_t cols, real *y)
{
#pragma omp parallel for schedule(static)
    for (int32_t r = 0; r < rows; ++r) {
        const uint16_t *row = w + (size_t)r * cols;
        real acc = 0;
        for (int32_t c = 0; c < cols; ++c) acc += widen(row[c]) * x[c];
        y[r] = acc + (bias ? widen(bias[r]) : 0.0);
    }
}

/* ------------------------------------------------------------------------------------------ */
/* cache                                                                                      */
/* ------------------------------------------------------------------------------------------ */

oracle_cache *oracle_cache_new(const oracle_desc *d, int32_t max_ctx, int32_t page_size,
                               int32_t n_pool_pages, const int32_t *block_table)
{
    oracle_cache *c = (oracle_cache *)calloc(1, sizeof *c);
    if (!c) return NULL;
    c->n_layers = d->n_layers; c->n_kv_heads = d->n_kv_heads; c->head_dim = d->head_dim;
    c->max_ctx = max_ctx; c->len = 0; c->page_size = page_size;
    if (page_size > 0) {
        int32_t n_entries = (max_ctx + page_size - 1) / page_size;
        c->n_rows = n_pool_pages * page_size;
        c->block_table = (int32_t *)malloc(sizeof(int32_t) * (size_t)n_entries);
        if (!c->block_table) { free(c); return NULL; }
        memcpy(c->block_table, block_table, sizeof(int32_t) * (size_t)n_entries);
    } else {
        c->n_rows = max_ctx;
    }
    size_t n = (size_t)c->n_layers * c->n_rows * c->n_kv_heads * c->head_dim;
    c->k = (real *)calloc(n, sizeof(real));
    c->v = (real *)calloc(n, sizeof(real));
    if (!c->k || !c->v) { free(c->k); free(c->v); free(c->block_table); free(c); return NULL; }
    return c;
}

void oracle_cache_free(oracle_cache *c)
{
    if (!c) return;
    free(c->k); free(c->v); free(c->block_table); free(c);
}

int32_t oracle_cache_len(const oracle_cache *c) { return c->len; }
void oracle_cache_set_len(oracle_cache *c, int32_t len) { c->len = len; }

static size_t cache_row(const oracle_cache *c, int32_t layer, int32_t pos)
{
    int32_t row = pos;
    if (c->page_size > 0) row = c->block_table[pos / c->page_size] * c->page_size + pos % c->page_size;
    return ((size_t)layer * c->n_rows + row) * c->n_kv_heads * c->head_dim;
}

/* fill positions 0..n_tokens-1 of one layer from bf16 arrays [n_tokens][kv_head][head_dim] */
void oracle_cache_load_bf16(oracle_cache *c, int32_t layer, int32_t n_tokens, const uint16_t *k,
                            const uint16_t *v)
{
    int32_t w = c->n_kv_heads * c->head_dim;
    for (int32_t p = 0; p < n_tokens; ++p) {
        size_t o = cache_row(c, layer, p);
        for (int32_t i = 0; i < w; ++i) {
            c->k[o + i] = widen(k[(size_t)p * w + i]);
            c->v[o + i] = widen(v[(size_t)p * w + i]);
        }
    }
}

/* same, from doubles (any value a 2-byte cache type can hold, already widened by the caller) */
void oracle_cache_load_f64(oracle_cache *c, int32_t layer, int32_t n_tokens, const real *k, const real *v)
{
    int32_t w = c->n_kv_heads * c->head_dim;
    for (int32_t p = 0; p < n_tokens; ++p) {
        size_t o = cache_row(c, layer, p);
        memcpy(c->k + o, k + (size_t)p * w, sizeof(real) * (size_t)w);
        memcpy(c->v + o, v + (size_t)p * w, sizeof(real) * (size_t)w);
    }
}

/* copy the cached k and v of (layer, pos) out, [kv_head][head_dim] each */
void oracle_cache_read(const oracle_cache *c, int32_t layer, int32_t pos, real *k_out, real *v_out)
{
    int32_t w = c->n_kv_heads * c->head_dim;
    size_t o = cache_row(c, layer, pos);
    memcpy(k_out, c->k + o, sizeof(real) * (size_t)w);
    memcpy(v_out, c->v + o, sizeof(real) * (size_t)w);
}

/* ------------------------------------------------------------------------------------------ */
/* attention                                                                                  */
/* ------------------------------------------------------------------------------------------ */

/* Grouped-query attention of one new token over cache positions 0..n_ctx-1 of one layer.
 * q [n_q_heads][head_dim]; query head a reads KV head a / (n_q_heads / n_kv_heads).
 * out [n_q_heads][head_dim]. */
void oracle_attention(const real *q, const oracle_cache *c, int32_t layer, int32_t n_ctx,
                      int32_t n_q_heads, real *out)
{
    int32_t hd = c->head_dim, group = n_q_heads / c->n_kv_heads;
    real scale = 1.0 / sqrt((real)hd);
#pragma omp parallel for schedule(static)
    for (int32_t a = 0; a < n_q_heads; ++a) {
        int32_t j = a / group;
        real *s = (real *)malloc(sizeof(real) * (size_t)n_ctx);
        for (int32_t t = 0; t < n_ctx; ++t) {
            const real *kt = c->k + cache_row(c, layer, t) + (size_t)j * hd;
            real dot = 0;
            for (int32_t i = 0; i < hd; ++i) dot += q[(size_t)a * hd + i] * kt[i];
            s[t] = dot * scale;
        }
        oracle_softmax(s, n_ctx);
        for (int32_t i = 0; i < hd; ++i) {
            real acc = 0;
            for (int32_t t = 0; t < n_ctx; ++t)
                acc += s[t] * c->v[cache_row(c, layer, t) + (size_t)j * hd + i];
            out[(size_t)a * hd + i] = acc;
        }
        free(s);
    }
}

/* Combining attention computed over disjoint pieces of the context: each piece i gives its
 * running maximum m_i, its sum l_i = sum exp(s - m_i) and o_i = sum exp(s - m_i) v.  The whole is
 * o = sum_i e^{m_i - M} o_i / sum_i e^{m_i - M} l_i with M = max m_i.  (Oracle-side statement of
 * the split-context identity, pinned against the unsplit attention above.) */
void oracle_attention_piece(const real *q, const oracle_cache *c, int32_t layer, int32_t t0,
                            int32_t t1, int32_t kv_head, real *m_out, real *l_out, real *o_out)
{
    int32_t hd = c->head_dim;
    real scale = 1.0 / sqrt((real)hd);
    real m = -INFINITY;
    for (int32_t t = t0; t < t1; ++t) {
        const real *kt = c->k + cache_row(c, layer, t) + (size_t)kv_head * hd;
        real dot = 0;
        for (int32_t i = 0; i < hd; ++i) dot += q[i] * kt[i];
        if (dot * scale > m) m = dot * scale;
    }
    real l = 0;
    for (int32_t i = 0; i < hd; ++i) o_out[i] = 0;
    for (int32_t t = t0; t < t1; ++t) {
        const real *kt = c->k + cache_row(c, layer, t) + (size_t)kv_head * hd;
        const real *vt = c->v + cache_row(c, layer, t) + (size_t)kv_head * hd;
        real dot = 0;
        for (int32_t i = 0; i < hd; ++i) dot += q[i] * kt[i];
        real p = exp(dot * scale - m);
        l += p;
        for (int32_t i = 0; i < hd; ++i) o_out[i] += p * vt[i];
    }
    *m_out = m; *l_out = l;
}

void oracle_attention_merge(int32_t n_pieces, const real *m, const real *l, const real *o,
                            int32_t head_dim, real *out)
{
    real M = -INFINITY, denom = 0;
    for (int32_t i = 0; i < n_pieces; ++i) if (m[i] > M) M = m[i];
    for (int32_t d = 0; d < head_dim; ++d) out[d] = 0;
    for (int32_t i = 0; i < n_pieces; ++i) {
        real w = exp(m[i] - M);
        denom += w * l[i];
        for (int32_t d = 0; d < head_dim; ++d) out[d] += w * o[(size_t)i * head_dim + d];
    }
    for (int32_t d = 0; d < head_dim; ++d) out[d] /= denom;
}

/* ------------------------------------------------------------------------------------------ */
/* one decode step for one game                                                               */
/* ------------------------------------------------------------------------------------------ */

/* Appends `token` at position cache->len, advances the cache, writes logits [vocab].
 * trace (optional) receives the residual stream x after the embedding and after every layer,
 * [(n_layers + 1)][d_model], and hidden (optional) the final-normed vector [d_model].
 * kv_as_bf16 != 0 rounds k and v to bf16 before caching them (a bisecting aid; the headline
 * comparison keeps them exact).  Returns 0, or -1 on bad token / full cache / no memory. */
int32_t oracle_decode_step(const oracle_desc *d, const oracle_weights *w, oracle_cache *c,
                           int32_t token, int32_t kv_as_bf16, real *logits, real *trace,
                           real *hidden)
{
    int32_t D = d->d_model, Hq = d->n_q_heads, Hkv = d->n_kv_heads, hd = d->head_dim, F = d->d_ff;
    int32_t pos = c->len;
    if (token < 0 || token >= d->vocab || pos >= c->max_ctx) return -1;
    real *x = (real *)malloc(sizeof(real) * (size_t)D);
    real *h = (real *)malloc(sizeof(real) * (size_t)D);
    real *q = (real *)malloc(sizeof(real) * (size_t)Hq * hd);
    real *k = (real *)malloc(sizeof(real) * (size_t)Hkv * hd);
    real *v = (real *)malloc(sizeof(real) * (size_t)Hkv * hd);
    real *o = (real *)malloc(sizeof(real) * (size_t)Hq * hd);
    real *t = (real *)malloc(sizeof(real) * (size_t)D);
    real *gate = (real *)malloc(sizeof(real) * (size_t)F);
    real *up = (real *)malloc(sizeof(real) * (size_t)F);
    if (!x || !h || !q || !k || !v || !o || !t || !gate || !up) {
        free(x); free(h); free(q); free(k); free(v); free(o); free(t); free(gate); free(up);
        return -1;
    }
    for (int32_t i = 0; i < D; ++i) x[i] = widen(w->embed[(size_t)token * D + i]);
    if (trace) memcpy(trace, x, sizeof(real) * (size_t)D);

    for (int32_t l = 0; l < d->n_layers; ++l) {
        oracle_rmsnorm(x, w->ln1[l], d->rms_eps, D, h);
        oracle_matvec(w->wq[l], d->qkv_bias ? w->bq[l] : NULL, h, Hq * hd, D, q);
        oracle_matvec(w->wk[l], d->qkv_bias ? w->bk[l] : NULL, h, Hkv * hd, D, k);
        oracle_matvec(w->wv[l], d->qkv_bias ? w->bv[l] : NULL, h, Hkv * hd, D, v);
        if (d->qk_norm) {
            for (int32_t a = 0; a < Hq; ++a)
                oracle_rmsnorm(q + (size_t)a * hd, w->q_norm[l], d->rms_eps, hd, q + (size_t)a * hd);
            for (int32_t j = 0; j < Hkv; ++j)
                oracle_rmsnorm(k + (size_t)j * hd, w->k_norm[l], d->rms_eps, hd, k + (size_t)j * hd);
        }
        for (int32_t a = 0; a < Hq; ++a) oracle_rope(q + (size_t)a * hd, hd, pos, d->rope_theta);
        for (int32_t j = 0; j < Hkv; ++j) oracle_rope(k + (size_t)j * hd, hd, pos, d->rope_theta);
        size_t row = cache_row(c, l, pos);
        for (int32_t i = 0; i < Hkv * hd; ++i) {
            c->k[row + i] = kv_as_bf16 ? round_bf16(k[i]) : k[i];
            c->v[row + i] = kv_as_bf16 ? round_bf16(v[i]) : v[i];
        }
        oracle_attention(q, c, l, pos + 1, Hq, o);
        oracle_matvec(w->wo[l], NULL, o, D, Hq * hd, t);
        for (int32_t i = 0; i < D; ++i) x[i] += t[i];

        oracle_rmsnorm(x, w->ln2[l], d->rms_eps, D, h);
        oracle_matvec(w->w_gate[l], NULL, h, F, D, gate);
        oracle_matvec(w->w_up[l], NULL, h, F, D, up);
        for (int32_t i = 0; i < F; ++i) gate[i] = oracle_silu(gate[i]) * up[i];
        oracle_matvec(w->w_down[l], NULL, gate, D, F, t);
        for (int32_t i = 0; i < D; ++i) x[i] += t[i];
        if (trace) memcpy(trace + (size_t)(l + 1) * D, x, sizeof(real) * (size_t)D);
    }
    oracle_rmsnorm(x, w->final_norm, d->rms_eps, D, h);
    if (hidden) memcpy(hidden, h, sizeof(real) * (size_t)D);
    if (logits)
        oracle_matvec(d->tied_embed ? w->embed : w->lm_head, NULL, h, d->vocab, D, logits);
    c->len = pos + 1;
    free(x); free(h); free(q); free(k); free(v); free(o); free(t); free(gate); free(up);
    return 0;
}

/* Prefill is the same recurrence run token by token; logits of the last token are returned
 * (last_logits may be NULL). */
int32_t oracle_prefill(const oracle_desc *d, const oracle_weights *w, oracle_cache *c,
                       const int32_t *tokens, int32_t n, int32_t kv_as_bf16, real *last_logits)
{
    for (int32_t i = 0; i < n; ++i) {
        int32_t rc = oracle_decode_step(d, w, c, tokens[i], kv_as_bf16,
                                        i == n - 1 ? last_logits : NULL, NULL, NULL);
        if (rc) return rc;
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------ */
/* sampling                                                                                   */
/* ------------------------------------------------------------------------------------------ */

/* Gumbel-max draw from softmax(logits / T): token = argmax_v ( fl32(logit_v) / T + gumbel_v ),
 * every operation rounded to fp32, lowest index wins ties.  best_z / gap (optional) return the
 * winning score and its distance to the runner-up. */
int32_t oracle_sample(const real *logits, const float *gumbel, float temperature, int32_t vocab,
                      float *best_z, float *gap)
{
    int32_t best = 0;
    float zb = -INFINITY, z2 = -INFINITY;
    for (int32_t v = 0; v < vocab; ++v) {
        volatile float scaled = (float)logits[v] / temperature;
        float z = scaled + gumbel[v];
        if (z > zb) { z2 = zb; zb = z; best = v; }
        else if (z > z2) z2 = z;
    }
    if (best_z) *best_z = zb;
    if (gap) *gap = zb - z2;
    return best;
}
