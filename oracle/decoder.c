/*
 * CPU ORACLE -- test infrastructure, not product code.
 *
 * A plain, slow decoder-only transformer forward pass, once with full recompute
 * and once against a key/value cache, written from the definitions.  Storage is
 * fp32; every reduction (dot product, norm statistic, softmax sum) accumulates in
 * float64 and is rounded to fp32 once.  The only other roundings are declared
 * storage points: matrices of a bf16 model hold bf16 values, and keys/values of a
 * bf16 model are rounded to bf16 (nearest-even) when they are stored.
 *
 * What each routine follows:
 *   - autoregressive conditional p(x_{n+1} | x_1..x_n): Eq. 1 (Section
 *     "Autoregressive vs Speculative Sampling"): orc_forward_full returns the
 *     logits of that conditional for every position of a token string.
 *   - KV caching: Section "KV Caching" and Figure 1: keys and values of past
 *     positions are stored once and reused; orc_forward_cached feeds only new
 *     tokens.  The two must agree (the cache "poses no risk to accuracy").
 *   - verification of K candidates in one target pass: Section "Autoregressive vs
 *     Speculative Sampling" ("batch size of K"), Figure 2: orc_forward_cached with
 *     m > 1 rows.
 * Block definitions (pre-norm decoder, LayerNorm/RMSNorm, erf-GELU/SwiGLU MLP,
 * learned or rotary positions, sequential or parallel residual) are the standard
 * ones of the GPT-2, GPT-NeoX and Llama families the paper names as workloads.
 *
 * No blocking, fusion or reordering: loops run in the order of the definition.
 * OpenMP only splits independent output features / heads over host threads.
 *
 * Pins (tests/test_oracle_*.py): library routines for each primitive, hand case,
 * causality and cached == recomputed invariants.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int32_t n_layers, d_model, n_heads, head_dim, d_ff, vocab, max_pos;
    int32_t norm;               /* 0 LayerNorm, 1 RMSNorm */
    int32_t act;                /* 0 GELU (erf form), 1 SwiGLU */
    int32_t pos;                /* 0 learned absolute, 1 rotary (half-split pairing) */
    int32_t parallel_residual;  /* 1: x + Attn(LN1 x) + MLP(LN2 x) */
    int32_t has_bias, tie_lm_head;
    int32_t dtype;              /* 0 fp32 matrices, 1 bf16 matrices and bf16-valued cache */
    int32_t rotary_dim;
    float rotary_base, norm_eps;
} orc_arch;

enum { T_TOK = 0, T_POS = 1, T_LAYER0 = 2, PER_LAYER = 12 };
enum { L_LN1G, L_LN1B, L_WQKV, L_BQKV, L_WO, L_BO, L_LN2G, L_LN2B, L_WIN, L_BIN, L_WOUT, L_BOUT };

static int g_threads = 1;
void orc_set_threads(int n) { g_threads = n > 0 ? n : 1; }
int orc_get_threads(void) { return g_threads; }

static inline float bf16_bits_to_f32(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* fp32 -> nearest bf16 value (ties to even), returned as fp32 */
float orc_round_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return f; /* NaN */
    u += 0x7fffu + ((u >> 16) & 1u);
    u &= 0xffff0000u;
    memcpy(&f, &u, 4);
    return f;
}

static inline double mat_at(const void *w, int dtype, size_t idx) {
    return dtype ? (double)bf16_bits_to_f32(((const uint16_t *)w)[idx]) : (double)((const float *)w)[idx];
}

/* y[m,n] = sum_k x[m,k] * W[n,k] (+ b[n]);  W row-major [N,Kd] */
void orc_linear(float *y, const float *x, const void *W, const float *b, int M, int N, int Kd, int dtype) {
#pragma omp parallel for num_threads(g_threads) schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int m = 0; m < M; ++m) {
            double acc = 0.0;
            const float *xr = x + (size_t)m * Kd;
            if (dtype) {
                const uint16_t *wr = (const uint16_t *)W + (size_t)n * Kd;
                for (int k = 0; k < Kd; ++k) acc += (double)xr[k] * (double)bf16_bits_to_f32(wr[k]);
            } else {
                const float *wr = (const float *)W + (size_t)n * Kd;
                for (int k = 0; k < Kd; ++k) acc += (double)xr[k] * (double)wr[k];
            }
            if (b) acc += (double)b[n];
            y[(size_t)m * N + n] = (float)acc;
        }
    }
}

/* LayerNorm: (x - mean) / sqrt(var + eps) * g + b, biased variance.  RMSNorm: x / sqrt(mean(x^2) + eps) * g */
void orc_norm(float *y, const float *x, const float *g, const float *b, int M, int d, int kind, float eps) {
    for (int m = 0; m < M; ++m) {
        const float *xr = x + (size_t)m * d;
        float *yr = y + (size_t)m * d;
        if (kind == 0) {
            double mean = 0.0, var = 0.0;
            for (int i = 0; i < d; ++i) mean += xr[i];
            mean /= d;
            for (int i = 0; i < d; ++i) { double c = xr[i] - mean; var += c * c; }
            var /= d;
            double rstd = 1.0 / sqrt(var + (double)eps);
            for (int i = 0; i < d; ++i)
                yr[i] = (float)((xr[i] - mean) * rstd * (double)g[i] + (b ? (double)b[i] : 0.0));
        } else {
            double ms = 0.0;
            for (int i = 0; i < d; ++i) ms += (double)xr[i] * xr[i];
            ms /= d;
            double r = 1.0 / sqrt(ms + (double)eps);
            for (int i = 0; i < d; ++i) yr[i] = (float)(xr[i] * r * (double)g[i]);
        }
    }
}

float orc_gelu(float v) { return (float)(0.5 * (double)v * (1.0 + erf((double)v / sqrt(2.0)))); }
float orc_silu(float v) { return (float)((double)v / (1.0 + exp(-(double)v))); }

/* Rotary embedding on one head vector, half-split pairing: (j, j + rd/2), angle pos * base^(-2j/rd) */
void orc_rotary(float *v, int rd, int pos, float base) {
    int half = rd / 2;
    for (int j = 0; j < half; ++j) {
        double theta = (double)pos * pow((double)base, -2.0 * j / rd);
        double c = cos(theta), s = sin(theta);
        double a = v[j], bb = v[j + half];
        v[j] = (float)(a * c - bb * s);
        v[j + half] = (float)(a * s + bb * c);
    }
}

/* attention of one query over keys/values [n_ctx, Dh] (row stride given): softmax(q.k / sqrt(Dh)) . v */
void orc_attend(float *out, const float *q, const float *keys, const float *vals, int n_ctx, int Dh,
                size_t stride) {
    double *s = (double *)malloc(sizeof(double) * (size_t)n_ctx);
    double scale = 1.0 / sqrt((double)Dh), mx = -INFINITY;
    for (int j = 0; j < n_ctx; ++j) {
        double acc = 0.0;
        const float *kr = keys + (size_t)j * stride;
        for (int e = 0; e < Dh; ++e) acc += (double)q[e] * (double)kr[e];
        s[j] = acc * scale;
        if (s[j] > mx) mx = s[j];
    }
    double z = 0.0;
    for (int j = 0; j < n_ctx; ++j) { s[j] = exp(s[j] - mx); z += s[j]; }
    for (int e = 0; e < Dh; ++e) {
        double acc = 0.0;
        for (int j = 0; j < n_ctx; ++j) acc += s[j] * (double)vals[(size_t)j * stride + e];
        out[e] = (float)(acc / z);
    }
    free(s);
}

static void embed(const orc_arch *a, const void *const *w, const int32_t *tok, int m, int pos0, float *x) {
    int d = a->d_model;
    for (int r = 0; r < m; ++r)
        for (int i = 0; i < d; ++i) {
            float v = (float)mat_at(w[T_TOK], a->dtype, (size_t)tok[r] * d + i);
            if (a->pos == 0) v = v + (float)mat_at(w[T_POS], a->dtype, (size_t)(pos0 + r) * d + i);
            x[(size_t)r * d + i] = v;
        }
}

/* MLP on normalised rows h[m,d] -> out[m,d] */
static void mlp(const orc_arch *a, const void *const *lw, const float *h, int m, float *out) {
    int d = a->d_model, F = a->d_ff;
    int n_in = a->act == 1 ? 2 * F : F;
    float *t = (float *)malloc(sizeof(float) * (size_t)m * n_in);
    float *g = (float *)malloc(sizeof(float) * (size_t)m * F);
    orc_linear(t, h, lw[L_WIN], (const float *)lw[L_BIN], m, n_in, d, a->dtype);
    for (int r = 0; r < m; ++r)
        for (int i = 0; i < F; ++i) {
            if (a->act == 1) /* rows [0,F) gate, [F,2F) up */
                g[(size_t)r * F + i] = orc_silu(t[(size_t)r * n_in + i]) * t[(size_t)r * n_in + F + i];
            else
                g[(size_t)r * F + i] = orc_gelu(t[(size_t)r * n_in + i]);
        }
    orc_linear(out, g, lw[L_WOUT], (const float *)lw[L_BOUT], m, d, F, a->dtype);
    free(t);
    free(g);
}

static void lm_head(const orc_arch *a, const void *const *w, const float *x, int m, float *logits) {
    int d = a->d_model;
    const void *const *fw = w + T_LAYER0 + (size_t)PER_LAYER * a->n_layers;
    float *h = (float *)malloc(sizeof(float) * (size_t)m * d);
    orc_norm(h, x, (const float *)fw[0], (const float *)fw[1], m, d, a->norm, a->norm_eps);
    orc_linear(logits, h, a->tie_lm_head ? w[T_TOK] : fw[2], NULL, m, a->vocab, d, a->dtype);
    free(h);
}

/*
 * One decoder block on m rows.  `attend_rows` supplies the attention output for the block
 * (that is where the full-recompute and the cached variants differ).
 */
typedef void (*attn_fn)(const orc_arch *, int layer, const float *qkv, int m, int pos0, float *o, void *ctx);

static void block(const orc_arch *a, const void *const *lw, int layer, float *x, int m, int pos0, attn_fn attn,
                  void *ctx) {
    int d = a->d_model;
    size_t md = (size_t)m * d;
    float *h = (float *)malloc(sizeof(float) * md);
    float *qkv = (float *)malloc(sizeof(float) * md * 3);
    float *o = (float *)malloc(sizeof(float) * md);
    float *att = (float *)malloc(sizeof(float) * md);
    float *ml = (float *)malloc(sizeof(float) * md);

    orc_norm(h, x, (const float *)lw[L_LN1G], (const float *)lw[L_LN1B], m, d, a->norm, a->norm_eps);
    orc_linear(qkv, h, lw[L_WQKV], (const float *)lw[L_BQKV], m, 3 * d, d, a->dtype);
    attn(a, layer, qkv, m, pos0, o, ctx);
    orc_linear(att, o, lw[L_WO], (const float *)lw[L_BO], m, d, d, a->dtype);

    if (a->parallel_residual) {
        orc_norm(h, x, (const float *)lw[L_LN2G], (const float *)lw[L_LN2B], m, d, a->norm, a->norm_eps);
        mlp(a, lw, h, m, ml);
        for (size_t i = 0; i < md; ++i) x[i] = x[i] + att[i] + ml[i];
    } else {
        for (size_t i = 0; i < md; ++i) x[i] = x[i] + att[i];
        orc_norm(h, x, (const float *)lw[L_LN2G], (const float *)lw[L_LN2B], m, d, a->norm, a->norm_eps);
        mlp(a, lw, h, m, ml);
        for (size_t i = 0; i < md; ++i) x[i] = x[i] + ml[i];
    }
    free(h); free(qkv); free(o); free(att); free(ml);
}

/* position-encode q and k of row r in place, and apply the cache's storage rounding to k and v */
static void prepare_qkv_row(const orc_arch *a, float *row /* [3d] */, int pos) {
    int d = a->d_model, Dh = a->head_dim;
    for (int h = 0; h < a->n_heads; ++h) {
        if (a->pos == 1) {
            orc_rotary(row + (size_t)h * Dh, a->rotary_dim, pos, a->rotary_base);
            orc_rotary(row + d + (size_t)h * Dh, a->rotary_dim, pos, a->rotary_base);
        }
    }
    if (a->dtype)
        for (int i = d; i < 3 * d; ++i) row[i] = orc_round_bf16(row[i]);
}

/* ---------------- full recompute: all keys/values of the string are rebuilt ---------------- */
static void attn_full(const orc_arch *a, int layer, const float *qkv_in, int m, int pos0, float *o, void *ctx) {
    (void)layer; (void)ctx; (void)pos0;
    int d = a->d_model, Dh = a->head_dim;
    float *qkv = (float *)malloc(sizeof(float) * (size_t)m * 3 * d);
    memcpy(qkv, qkv_in, sizeof(float) * (size_t)m * 3 * d);
    for (int r = 0; r < m; ++r) prepare_qkv_row(a, qkv + (size_t)r * 3 * d, r);
#pragma omp parallel for num_threads(g_threads) schedule(dynamic)
    for (int hr = 0; hr < a->n_heads * m; ++hr) {
        int h = hr / m, r = hr % m;
        /* row r sees positions 0..r */
        orc_attend(o + (size_t)r * d + (size_t)h * Dh, qkv + (size_t)r * 3 * d + (size_t)h * Dh,
                   qkv + d + (size_t)h * Dh, qkv + 2 * d + (size_t)h * Dh, r + 1, Dh, (size_t)3 * d);
    }
    free(qkv);
}

/* logits[n, V] for every position of tokens[0..n) with no cache */
int orc_forward_full(const orc_arch *a, const void *const *w, const int32_t *tokens, int n, float *logits) {
    int d = a->d_model;
    float *x = (float *)malloc(sizeof(float) * (size_t)n * d);
    embed(a, w, tokens, n, 0, x);
    for (int l = 0; l < a->n_layers; ++l)
        block(a, w + T_LAYER0 + (size_t)PER_LAYER * l, l, x, n, 0, attn_full, NULL);
    lm_head(a, w, x, n, logits);
    free(x);
    return 0;
}

/* ---------------- cached: only new rows are fed ---------------- */
typedef struct {
    float *kv;      /* [L][2][H][S_max][Dh], fp32 storage (bf16-valued for bf16 models) */
    int s_max, len; /* len = rows already stored */
} orc_cache_view;

static void attn_cached(const orc_arch *a, int layer, const float *qkv_in, int m, int pos0, float *o, void *ctx) {
    orc_cache_view *c = (orc_cache_view *)ctx;
    int d = a->d_model, Dh = a->head_dim, H = a->n_heads;
    size_t plane = (size_t)H * c->s_max * Dh;
    float *Kc = c->kv + (size_t)layer * 2 * plane, *Vc = Kc + plane;
    float *qkv = (float *)malloc(sizeof(float) * (size_t)m * 3 * d);
    memcpy(qkv, qkv_in, sizeof(float) * (size_t)m * 3 * d);
    for (int r = 0; r < m; ++r) {
        float *row = qkv + (size_t)r * 3 * d;
        prepare_qkv_row(a, row, pos0 + r);
        for (int h = 0; h < H; ++h) { /* append */
            memcpy(Kc + ((size_t)h * c->s_max + pos0 + r) * Dh, row + d + (size_t)h * Dh, sizeof(float) * Dh);
            memcpy(Vc + ((size_t)h * c->s_max + pos0 + r) * Dh, row + 2 * d + (size_t)h * Dh, sizeof(float) * Dh);
        }
    }
#pragma omp parallel for num_threads(g_threads) schedule(dynamic)
    for (int hr = 0; hr < H * m; ++hr) {
        int h = hr / m, r = hr % m;
        orc_attend(o + (size_t)r * d + (size_t)h * Dh, qkv + (size_t)r * 3 * d + (size_t)h * Dh,
                   Kc + (size_t)h * c->s_max * Dh, Vc + (size_t)h * c->s_max * Dh, pos0 + r + 1, Dh, (size_t)Dh);
    }
    free(qkv);
}

/*
 * Feed m new tokens at positions len..len+m-1 against the cache; rows len..len+m-1 of the
 * cache are (over)written.  The caller owns the committed length: this routine does not
 * change it, so dropping rejected rows is just not advancing past them.
 * Returns -1 if the rows do not fit.
 */
int orc_forward_cached(const orc_arch *a, const void *const *w, float *kv, int s_max, int len,
                       const int32_t *tokens, int m, float *logits) {
    if (len + m > s_max || m <= 0) return -1;
    if (a->pos == 0 && len + m > a->max_pos) return -1;
    int d = a->d_model;
    orc_cache_view c = {kv, s_max, len};
    float *x = (float *)malloc(sizeof(float) * (size_t)m * d);
    embed(a, w, tokens, m, len, x);
    for (int l = 0; l < a->n_layers; ++l)
        block(a, w + T_LAYER0 + (size_t)PER_LAYER * l, l, x, m, len, attn_cached, &c);
    if (logits) lm_head(a, w, x, m, logits);
    free(x);
    return 0;
}

/* attention-only entry: m query rows [m, H*Dh] (already position-encoded) over a filled cache slab
 * of one layer [2][H][S_max][Dh]; row r sees positions 0..len+r.  For long-context checks. */
void orc_attention_rows(const float *q, const float *kv_layer, int H, int Dh, int s_max, int len, int m,
                        float *o) {
    size_t plane = (size_t)H * s_max * Dh;
#pragma omp parallel for num_threads(g_threads) schedule(dynamic)
    for (int hr = 0; hr < H * m; ++hr) {
        int h = hr / m, r = hr % m;
        orc_attend(o + (size_t)r * H * Dh + (size_t)h * Dh, q + (size_t)r * H * Dh + (size_t)h * Dh,
                   kv_layer + (size_t)h * s_max * Dh, kv_layer + plane + (size_t)h * s_max * Dh, len + r + 1, Dh,
                   (size_t)Dh);
    }
}
