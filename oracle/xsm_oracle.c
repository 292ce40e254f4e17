/*
 * CPU oracle for multi-head speculative decoding of a cross-attention
 * conditioned auto-regressive mesh transformer.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of the
 * method that the CUDA library is checked against and that the benchmark times
 * as its CPU baseline.  It shares no code with the CUDA path, and the product
 * never calls it.
 *
 * What it follows:
 *   - backbone block (self-attention with a key/value cache, cross-attention
 *     to the condition c, feed-forward network) and the backbone decoder
 *     p0 = softmax(W0 h): Sec. 4.1, Eq. 2;
 *   - the causal multi-position forward: Sec. 3.1, Eq. 1;
 *   - decoding heads on the final hidden state: the cross-attention head of
 *     Eq. 3, p(d) = softmax(W(d) CrossAttn(d)(h_s, c)), read as one residual
 *     cross-attention layer with weights of its own (head_kind 1), and the MLP
 *     form of the ablation (Table 3 rows B and C, head_kind 0):
 *     y = g + SiLU(W1 g), logits = Wout y;
 *   - verification, resampling and the outer loop: Sec. 4.2 and Algorithm 1;
 *   - probability-threshold and Top-K_a acceptance: Sec. 5.4;
 *   - independent sampling of the D+1 candidates, and Top-K_s probability
 *     tree sampling over the heads: Appendix (Ablation of Sampling Strategies);
 *   - step compression ratio: Sec. 5.1.
 *
 * Arithmetic: every stored value is fp32; every dot product, norm, softmax and
 * activation is evaluated in double and rounded to fp32 once when stored.
 * Row loops may run on several threads (OpenMP); each output element is
 * computed by one thread in a fixed order, so results do not depend on the
 * thread count.
 *
 * Parity pins live in tests/ (greedy equivalence, dense brute-force forward,
 * RoPE shift invariance, rollback == never-speculated cache, Philox known
 * answers, acceptance special cases, sampling frequencies, Table 3/4 speedup
 * identity).  Unpinned: the paper's quality metrics and its measured SCR
 * values, which are properties of trained weights that do not exist here
 * ("parity unpinned" for those two only).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <stdio.h>

typedef struct {
    int n_layers, d_model, n_heads, d_head, d_ff, vocab, n_cond, d_cond;
    int n_draft, head_hidden;
    int wdtype;            /* 0: weights are fp32, 1: bf16 bit patterns */
    int page_size, n_pages;
    float rope_theta, rms_eps;
    int bos_id, eos_id;    /* eos_id < 0: no EOS */
    int head_kind;         /* 0: MLP heads (Table 3 B, C); 1: cross-attention heads (Eq. 3) */
} orc_model_config;

typedef struct {
    int verify_mode;       /* 0 strict greedy, 1 top-K_a, 2 probability threshold */
    int k_accept;
    float delta;
    int sample_mode;       /* 0 argmax, 1 top-k with temperature, 2 top-k_sample probability tree over the heads */
    int k_sample;
    float temperature;
    uint64_t seed;
} orc_decode_config;

typedef struct {
    size_t g1, wq, wk, wv, wo, g2, wqc, wkc, wvc, woc, g3, wgate, wup, wdown;
} layer_off;

typedef struct orc_ctx {
    orc_model_config c;
    const void *w;
    size_t off_E, off_gf, off_W0;
    layer_off *lo;
    size_t *off_W1, *off_Wout;                 /* MLP heads */
    size_t *off_hq, *off_hk, *off_hv, *off_ho; /* cross-attention heads: Wq, Wk, Wv, Wo of head i (then off_Wout) */
    /* shared page pool: page p holds [layer][k|v][slot][d_model] floats */
    float *pool;
    int *free_stack;
    int n_free;
} orc_ctx;

typedef struct orc_seq {
    orc_ctx *ctx;
    int seq_id;
    float *ck, *cv;        /* cross K, V: [layer][n_cond][d_model] */
    float *hk, *hv;        /* cross-attention heads: K, V of the condition per head [head][n_cond][d_model] */
    int *block_table;      /* logical page -> physical page */
    int n_blocks, max_blocks;
    int len;               /* s: positions 0..s-1 are committed in the cache */
    int32_t *window;       /* x_s, x_{s+1..s+K} */
    uint32_t step_idx;
    int finished;
} orc_seq;

/* ------------------------------------------------------------------ utils */

static inline float bf16_to_f32(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* dot(W[row], x) in double; eight running sums in a fixed order. */
static double dot_row(const orc_ctx *ctx, size_t off, int n, const float *x) {
    double a[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    int k = 0;
    if (ctx->c.wdtype == 1) {
        const uint16_t *w = (const uint16_t *)ctx->w + off;
        for (; k + 8 <= n; k += 8)
            for (int j = 0; j < 8; ++j) a[j] += (double)bf16_to_f32(w[k + j]) * (double)x[k + j];
        for (; k < n; ++k) a[0] += (double)bf16_to_f32(w[k]) * (double)x[k];
    } else {
        const float *w = (const float *)ctx->w + off;
        for (; k + 8 <= n; k += 8)
            for (int j = 0; j < 8; ++j) a[j] += (double)w[k + j] * (double)x[k + j];
        for (; k < n; ++k) a[0] += (double)w[k] * (double)x[k];
    }
    return ((a[0] + a[1]) + (a[2] + a[3])) + ((a[4] + a[5]) + (a[6] + a[7]));
}

static inline float wval(const orc_ctx *ctx, size_t off) {
    return ctx->c.wdtype == 1 ? bf16_to_f32(((const uint16_t *)ctx->w)[off])
                              : ((const float *)ctx->w)[off];
}

/* y = W x, W is [rows, cols] row-major at element offset off. */
static void matvec(const orc_ctx *ctx, size_t off, int rows, int cols, const float *x, float *y) {
#pragma omp parallel for schedule(static)
    for (int r = 0; r < rows; ++r) y[r] = (float)dot_row(ctx, off + (size_t)r * cols, cols, x);
}

/* RMSNorm: x / sqrt(mean(x^2) + eps) * g */
static void rmsnorm(const orc_ctx *ctx, size_t g_off, const float *x, float *y, int n) {
    double ss = 0;
    for (int i = 0; i < n; ++i) ss += (double)x[i] * (double)x[i];
    double inv = 1.0 / sqrt(ss / n + (double)ctx->c.rms_eps);
    for (int i = 0; i < n; ++i) y[i] = (float)((double)x[i] * inv * (double)wval(ctx, g_off + i));
}

static inline double silu(double v) { return v / (1.0 + exp(-v)); }

/* Rotary embedding, half-split pairing (i, i + dh/2), angle = pos * theta^(-2i/dh). */
static void rope(const orc_ctx *ctx, float *v, int pos) {
    int H = ctx->c.n_heads, dh = ctx->c.d_head, half = dh / 2;
    for (int h = 0; h < H; ++h) {
        float *p = v + h * dh;
        for (int i = 0; i < half; ++i) {
            double ang = (double)pos * pow((double)ctx->c.rope_theta, -2.0 * i / dh);
            double c = cos(ang), s = sin(ang);
            double a = p[i], b = p[i + half];
            p[i] = (float)(a * c - b * s);
            p[i + half] = (float)(a * s + b * c);
        }
    }
}

/* ------------------------------------------------------------ page pool */

static size_t page_floats(const orc_ctx *ctx) {
    return (size_t)ctx->c.n_layers * 2 * ctx->c.page_size * ctx->c.d_model;
}

/* cache row of d_model floats for (layer, k|v, position) of a sequence */
static float *cache_row(const orc_seq *s, int layer, int kv, int pos) {
    const orc_ctx *ctx = s->ctx;
    int P = ctx->c.page_size;
    int phys = s->block_table[pos / P];
    return ctx->pool + (size_t)phys * page_floats(ctx) +
           (((size_t)layer * 2 + kv) * P + (pos % P)) * ctx->c.d_model;
}

/* make positions 0..upto-1 addressable; returns 0 on success, -1 if the pool is empty */
static int seq_reserve(orc_seq *s, int upto) {
    orc_ctx *ctx = s->ctx;
    int need = (upto + ctx->c.page_size - 1) / ctx->c.page_size;
    if (need > s->max_blocks) return -1;
    while (s->n_blocks < need) {
        if (ctx->n_free == 0) return -1;
        s->block_table[s->n_blocks++] = ctx->free_stack[--ctx->n_free];
    }
    return 0;
}

/* give back every page that lies wholly at or beyond position upto */
static void seq_release_beyond(orc_seq *s, int upto) {
    orc_ctx *ctx = s->ctx;
    int keep = (upto + ctx->c.page_size - 1) / ctx->c.page_size;
    while (s->n_blocks > keep) ctx->free_stack[ctx->n_free++] = s->block_table[--s->n_blocks];
}

/* ---------------------------------------------------------- create/destroy */

size_t orc_weight_elements(const orc_model_config *c) {
    size_t d = c->d_model, f = c->d_ff, V = c->vocab, dc = c->d_cond, hd = c->head_hidden;
    size_t per_layer = 3 * d + 6 * d * d + 2 * d * dc + 3 * d * f;
    size_t per_head = c->head_kind == 1 ? 2 * d * d + 2 * d * dc + V * d : hd * d + V * hd;
    return V * d + c->n_layers * per_layer + d + V * d + (size_t)c->n_draft * per_head;
}

int orc_create(const orc_model_config *c, const void *weights, orc_ctx **out) {
    if (!c || !weights || !out) return -1;
    if (c->head_hidden != c->d_model || c->n_heads * c->d_head != c->d_model || (c->d_head & 1)) return -1;
    orc_ctx *ctx = (orc_ctx *)calloc(1, sizeof(orc_ctx));
    ctx->c = *c;
    ctx->w = weights;
    size_t d = c->d_model, f = c->d_ff, V = c->vocab, dc = c->d_cond, hd = c->head_hidden;
    size_t o = 0;
    ctx->off_E = o; o += V * d;
    ctx->lo = (layer_off *)calloc(c->n_layers, sizeof(layer_off));
    for (int l = 0; l < c->n_layers; ++l) {
        layer_off *L = &ctx->lo[l];
        L->g1 = o; o += d;
        L->wq = o; o += d * d;
        L->wk = o; o += d * d;
        L->wv = o; o += d * d;
        L->wo = o; o += d * d;
        L->g2 = o; o += d;
        L->wqc = o; o += d * d;
        L->wkc = o; o += d * dc;
        L->wvc = o; o += d * dc;
        L->woc = o; o += d * d;
        L->g3 = o; o += d;
        L->wgate = o; o += f * d;
        L->wup = o; o += f * d;
        L->wdown = o; o += d * f;
    }
    ctx->off_gf = o; o += d;
    ctx->off_W0 = o; o += V * d;
    ctx->off_W1 = (size_t *)calloc(c->n_draft + 1, sizeof(size_t));
    ctx->off_Wout = (size_t *)calloc(c->n_draft + 1, sizeof(size_t));
    ctx->off_hq = (size_t *)calloc(c->n_draft + 1, sizeof(size_t));
    ctx->off_hk = (size_t *)calloc(c->n_draft + 1, sizeof(size_t));
    ctx->off_hv = (size_t *)calloc(c->n_draft + 1, sizeof(size_t));
    ctx->off_ho = (size_t *)calloc(c->n_draft + 1, sizeof(size_t));
    for (int i = 0; i < c->n_draft; ++i) {
        if (c->head_kind == 1) {
            ctx->off_hq[i] = o; o += d * d;
            ctx->off_hk[i] = o; o += d * dc;
            ctx->off_hv[i] = o; o += d * dc;
            ctx->off_ho[i] = o; o += d * d;
            ctx->off_Wout[i] = o; o += V * d;
        } else {
            ctx->off_W1[i] = o; o += hd * d;
            ctx->off_Wout[i] = o; o += V * hd;
        }
    }
    ctx->pool = (float *)calloc((size_t)c->n_pages * page_floats(ctx), sizeof(float));
    ctx->free_stack = (int *)malloc(sizeof(int) * (c->n_pages > 0 ? c->n_pages : 1));
    if (!ctx->pool || !ctx->free_stack) return -2;
    for (int p = 0; p < c->n_pages; ++p) ctx->free_stack[p] = c->n_pages - 1 - p;
    ctx->n_free = c->n_pages;
    *out = ctx;
    return 0;
}

void orc_destroy(orc_ctx *ctx) {
    if (!ctx) return;
    free(ctx->pool); free(ctx->free_stack); free(ctx->lo); free(ctx->off_W1); free(ctx->off_Wout);
    free(ctx->off_hq); free(ctx->off_hk); free(ctx->off_hv); free(ctx->off_ho);
    free(ctx);
}

int orc_free_pages(const orc_ctx *ctx) { return ctx->n_free; }

/* ------------------------------------------------------------- Philox RNG */

/* Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw: "Parallel random
 * numbers: as easy as 1, 2, 3", SC'11). */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3], k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0, p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0, n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1, n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* 24 random bits for (sequence, step, slot, purpose); u = bits * 2^-24 in [0,1).
 * purpose 0: resampling in a step; purpose 1: the initial drafts. */
uint32_t orc_rand24(uint64_t seed, int seq_id, uint32_t step, uint32_t slot, uint32_t purpose) {
    uint32_t key[2] = {(uint32_t)seed ^ (uint32_t)seq_id, (uint32_t)(seed >> 32)};
    uint32_t ctr[4] = {step, slot, purpose, 0}, o[4];
    orc_philox4x32_10(ctr, key, o);
    return o[0] >> 8;
}

/* ------------------------------------------------- acceptance and sampling */

/* is a ranked before b?  larger logit first, then smaller index */
static inline int before(const float *z, int a, int b) { return z[a] > z[b] || (z[a] == z[b] && a < b); }

/* Acceptance of candidate token x under the backbone logits z (Sec. 4.2, Sec. 5.4). */
int orc_accept(const float *z, int V, int x, const orc_decode_config *dc) {
    if (x < 0 || x >= V) return 0;
    if (dc->verify_mode == 2) {          /* p0(x) > delta, strictly */
        double m = z[0];
        for (int v = 1; v < V; ++v) if (z[v] > m) m = z[v];
        double sum = 0;
        for (int v = 0; v < V; ++v) sum += exp((double)z[v] - m);
        return exp((double)z[x] - m) / sum > (double)dc->delta;
    }
    int ka = dc->verify_mode == 0 ? 1 : dc->k_accept;
    int rank = 0;
    for (int v = 0; v < V; ++v) if (v != x && before(z, v, x)) ++rank;
    return rank < ka;
}

/* Draw one token from logits z with u = r24 * 2^-24. */
int orc_sample(const float *z, int V, const orc_decode_config *dc, uint32_t r24) {
    /* sample_mode 2 draws a single distribution (the backbone's) like sample_mode 1 */
    if (dc->sample_mode == 0) {
        int best = 0;
        for (int v = 1; v < V; ++v) if (before(z, v, best)) best = v;
        return best;
    }
    int k = dc->k_sample < 1 ? 1 : (dc->k_sample > V ? V : dc->k_sample);
    int *cand = (int *)malloc(sizeof(int) * k);
    double *w = (double *)malloc(sizeof(double) * k);
    for (int j = 0; j < k; ++j) {        /* j-th candidate: best not yet taken */
        int best = -1;
        for (int v = 0; v < V; ++v) {
            if (j > 0 && !before(z, cand[j - 1], v)) continue;   /* v is at or before the last pick */
            if (best < 0 || before(z, v, best)) best = v;
        }
        cand[j] = best;
    }
    double total = 0;
    for (int j = 0; j < k; ++j) {
        w[j] = exp(((double)z[cand[j]] - (double)z[cand[0]]) / (double)dc->temperature);
        total += w[j];
    }
    double u = (double)r24 * (1.0 / 16777216.0), cum = 0;
    int pick = cand[k - 1];
    for (int j = 0; j < k; ++j) {
        cum += w[j];
        if (cum > u * total) { pick = cand[j]; break; }
    }
    free(cand); free(w);
    return pick;
}

/* --------------------------------------------------------------- sequence */

int orc_seq_create(orc_ctx *ctx, const float *cond, int seq_id, int max_positions, orc_seq **out) {
    const orc_model_config *c = &ctx->c;
    orc_seq *s = (orc_seq *)calloc(1, sizeof(orc_seq));
    s->ctx = ctx;
    s->seq_id = seq_id;
    size_t d = c->d_model;
    s->ck = (float *)malloc(sizeof(float) * c->n_layers * c->n_cond * d);
    s->cv = (float *)malloc(sizeof(float) * c->n_layers * c->n_cond * d);
    /* cross keys and values of the condition: K_c = Wkc c_j, V_c = Wvc c_j per layer */
    for (int l = 0; l < c->n_layers; ++l)
        for (int j = 0; j < c->n_cond; ++j) {
            matvec(ctx, ctx->lo[l].wkc, c->d_model, c->d_cond, cond + (size_t)j * c->d_cond,
                   s->ck + ((size_t)l * c->n_cond + j) * d);
            matvec(ctx, ctx->lo[l].wvc, c->d_model, c->d_cond, cond + (size_t)j * c->d_cond,
                   s->cv + ((size_t)l * c->n_cond + j) * d);
        }
    /* cross-attention heads: every head projects the condition with its own Wk, Wv */
    if (c->head_kind == 1 && c->n_draft > 0) {
        s->hk = (float *)malloc(sizeof(float) * c->n_draft * c->n_cond * d);
        s->hv = (float *)malloc(sizeof(float) * c->n_draft * c->n_cond * d);
        for (int i = 0; i < c->n_draft; ++i)
            for (int j = 0; j < c->n_cond; ++j) {
                matvec(ctx, ctx->off_hk[i], c->d_model, c->d_cond, cond + (size_t)j * c->d_cond,
                       s->hk + ((size_t)i * c->n_cond + j) * d);
                matvec(ctx, ctx->off_hv[i], c->d_model, c->d_cond, cond + (size_t)j * c->d_cond,
                       s->hv + ((size_t)i * c->n_cond + j) * d);
            }
    }
    s->max_blocks = (max_positions + c->page_size - 1) / c->page_size;
    s->block_table = (int *)malloc(sizeof(int) * (s->max_blocks > 0 ? s->max_blocks : 1));
    s->window = (int32_t *)calloc(c->n_draft + 1, sizeof(int32_t));
    *out = s;
    return 0;
}

void orc_seq_destroy(orc_seq *s) {
    if (!s) return;
    seq_release_beyond(s, 0);
    free(s->ck); free(s->cv); free(s->hk); free(s->hv); free(s->block_table); free(s->window); free(s);
}

int orc_seq_len(const orc_seq *s) { return s->len; }
int orc_seq_blocks(const orc_seq *s) { return s->n_blocks; }
int orc_seq_finished(const orc_seq *s) { return s->finished; }
uint32_t orc_seq_step_idx(const orc_seq *s) { return s->step_idx; }
void orc_seq_get_window(const orc_seq *s, int32_t *w) { memcpy(w, s->window, sizeof(int32_t) * (s->ctx->c.n_draft + 1)); }
void orc_seq_set_window(orc_seq *s, const int32_t *w) { memcpy(s->window, w, sizeof(int32_t) * (s->ctx->c.n_draft + 1)); }
void orc_seq_set_drafts(orc_seq *s, const int32_t *drafts) { memcpy(s->window + 1, drafts, sizeof(int32_t) * s->ctx->c.n_draft); }
void orc_seq_set_len(orc_seq *s, int len) { s->len = len; }
void orc_seq_set_step_idx(orc_seq *s, uint32_t v) { s->step_idx = v; }

/* copy the cached key (kv=0) or value (kv=1) row of one position */
int orc_seq_get_kv(const orc_seq *s, int layer, int kv, int pos, float *out) {
    if (pos < 0 || pos / s->ctx->c.page_size >= s->n_blocks) return -1;
    memcpy(out, cache_row(s, layer, kv, pos), sizeof(float) * s->ctx->c.d_model);
    return 0;
}

/* softmax(q k^T / sqrt(dh)) v for one head over n keys; rows of k, v are `stride` apart */
static void attend(const float *q, int dh, int n, const float *const *krows, const float *const *vrows,
                   int head_off, float *out) {
    double *p = (double *)malloc(sizeof(double) * n);
    double scale = 1.0 / sqrt((double)dh), m = -INFINITY;
    for (int j = 0; j < n; ++j) {
        const float *k = krows[j] + head_off;
        double s = 0;
        for (int i = 0; i < dh; ++i) s += (double)q[i] * (double)k[i];
        p[j] = s * scale;
        if (p[j] > m) m = p[j];
    }
    double sum = 0;
    for (int j = 0; j < n; ++j) { p[j] = exp(p[j] - m); sum += p[j]; }
    for (int i = 0; i < dh; ++i) {
        double o = 0;
        for (int j = 0; j < n; ++j) o += p[j] * (double)vrows[j][head_off + i];
        out[i] = (float)(o / sum);
    }
    free(p);
}

/*
 * One token through the backbone at absolute position pos (Sec. 4.1): its key
 * and value are written to the cache at pos, it attends to positions 0..pos.
 * Outputs: logits0[V] = W0 g (Eq. 2 before the softmax) and g[d] =
 * RMSNorm_f(h^N), the final hidden state that W0 and the heads read.
 */
int orc_forward_row(orc_seq *s, int token, int pos, float *logits0, float *g_out) {
    orc_ctx *ctx = s->ctx;
    const orc_model_config *c = &ctx->c;
    int d = c->d_model, H = c->n_heads, dh = c->d_head, f = c->d_ff;
    if (token < 0 || token >= c->vocab) return -1;
    if (seq_reserve(s, pos + 1)) return -2;
    float *h = (float *)malloc(sizeof(float) * d), *u = (float *)malloc(sizeof(float) * d);
    float *q = (float *)malloc(sizeof(float) * d), *k = (float *)malloc(sizeof(float) * d);
    float *v = (float *)malloc(sizeof(float) * d), *a = (float *)malloc(sizeof(float) * d);
    float *t = (float *)malloc(sizeof(float) * d);
    float *ga = (float *)malloc(sizeof(float) * f), *up = (float *)malloc(sizeof(float) * f);
    int nk = pos + 1 > c->n_cond ? pos + 1 : c->n_cond;
    const float **kr = (const float **)malloc(sizeof(float *) * nk);
    const float **vr = (const float **)malloc(sizeof(float *) * nk);
    for (int i = 0; i < d; ++i) h[i] = wval(ctx, ctx->off_E + (size_t)token * d + i);
    for (int l = 0; l < c->n_layers; ++l) {
        const layer_off *L = &ctx->lo[l];
        /* self-attention */
        rmsnorm(ctx, L->g1, h, u, d);
        matvec(ctx, L->wq, d, d, u, q);
        matvec(ctx, L->wk, d, d, u, k);
        matvec(ctx, L->wv, d, d, u, v);
        rope(ctx, q, pos);
        rope(ctx, k, pos);
        memcpy(cache_row(s, l, 0, pos), k, sizeof(float) * d);
        memcpy(cache_row(s, l, 1, pos), v, sizeof(float) * d);
        for (int j = 0; j <= pos; ++j) { kr[j] = cache_row(s, l, 0, j); vr[j] = cache_row(s, l, 1, j); }
#pragma omp parallel for schedule(static)
        for (int hh = 0; hh < H; ++hh) attend(q + hh * dh, dh, pos + 1, kr, vr, hh * dh, a + hh * dh);
        matvec(ctx, L->wo, d, d, a, t);
        for (int i = 0; i < d; ++i) h[i] = (float)((double)h[i] + (double)t[i]);
        /* cross-attention to the condition */
        rmsnorm(ctx, L->g2, h, u, d);
        matvec(ctx, L->wqc, d, d, u, q);
        for (int j = 0; j < c->n_cond; ++j) {
            kr[j] = s->ck + ((size_t)l * c->n_cond + j) * d;
            vr[j] = s->cv + ((size_t)l * c->n_cond + j) * d;
        }
#pragma omp parallel for schedule(static)
        for (int hh = 0; hh < H; ++hh) attend(q + hh * dh, dh, c->n_cond, kr, vr, hh * dh, a + hh * dh);
        matvec(ctx, L->woc, d, d, a, t);
        for (int i = 0; i < d; ++i) h[i] = (float)((double)h[i] + (double)t[i]);
        /* gated feed-forward network */
        rmsnorm(ctx, L->g3, h, u, d);
        matvec(ctx, L->wgate, f, d, u, ga);
        matvec(ctx, L->wup, f, d, u, up);
        for (int i = 0; i < f; ++i) ga[i] = (float)(silu((double)ga[i]) * (double)up[i]);
        matvec(ctx, L->wdown, d, f, ga, t);
        for (int i = 0; i < d; ++i) h[i] = (float)((double)h[i] + (double)t[i]);
    }
    rmsnorm(ctx, ctx->off_gf, h, u, d);
    if (g_out) memcpy(g_out, u, sizeof(float) * d);
    if (logits0) matvec(ctx, ctx->off_W0, c->vocab, d, u, logits0);
    free(h); free(u); free(q); free(k); free(v); free(a); free(t); free(ga); free(up);
    free(kr); free(vr);
    return 0;
}

/* Decoding head i (1-based) on final hidden state g: logits = Wout (g + SiLU(W1 g)). */
void orc_head(const orc_ctx *ctx, int i, const float *g, float *logits) {
    int d = ctx->c.d_model, hd = ctx->c.head_hidden;
    float *y = (float *)malloc(sizeof(float) * hd);
    matvec(ctx, ctx->off_W1[i - 1], hd, d, g, y);
    for (int j = 0; j < hd; ++j) y[j] = (float)((double)g[j] + silu((double)y[j]));
    matvec(ctx, ctx->off_Wout[i - 1], ctx->c.vocab, hd, y, logits);
    free(y);
}

/* Cross-attention decoding head i (1-based) on final hidden state g (Eq. 3): one residual cross-attention layer with
 * the head's own weights, y = g + Wo Attn(Wq g, Wk c, Wv c) with the backbone's head count and scale, logits = W(i) y. */
void orc_head_ca(const orc_seq *s, int i, const float *g, float *logits) {
    const orc_ctx *ctx = s->ctx;
    const orc_model_config *c = &ctx->c;
    int d = c->d_model, H = c->n_heads, dh = c->d_head;
    float *q = (float *)malloc(sizeof(float) * d), *a = (float *)malloc(sizeof(float) * d);
    float *t = (float *)malloc(sizeof(float) * d), *y = (float *)malloc(sizeof(float) * d);
    const float **kr = (const float **)malloc(sizeof(float *) * c->n_cond);
    const float **vr = (const float **)malloc(sizeof(float *) * c->n_cond);
    matvec(ctx, ctx->off_hq[i - 1], d, d, g, q);
    for (int j = 0; j < c->n_cond; ++j) {
        kr[j] = s->hk + ((size_t)(i - 1) * c->n_cond + j) * d;
        vr[j] = s->hv + ((size_t)(i - 1) * c->n_cond + j) * d;
    }
    for (int hh = 0; hh < H; ++hh) attend(q + hh * dh, dh, c->n_cond, kr, vr, hh * dh, a + hh * dh);
    matvec(ctx, ctx->off_ho[i - 1], d, d, a, t);
    for (int j = 0; j < d; ++j) y[j] = (float)((double)g[j] + (double)t[j]);
    matvec(ctx, ctx->off_Wout[i - 1], c->vocab, d, y, logits);
    free(q); free(a); free(t); free(y); free(kr); free(vr);
}

/* head i of either kind */
void orc_seq_head(const orc_seq *s, int i, const float *g, float *logits) {
    if (s->ctx->c.head_kind == 1) orc_head_ca(s, i, g, logits);
    else orc_head(s->ctx, i, g, logits);
}

/*
 * Top-K_s probability tree sampling over the D heads (Appendix, Ablation of Sampling Strategies).  Level d of the
 * tree branches over the K_s most probable tokens of head d (full-vocabulary softmax probabilities m), the weight of
 * a root-to-leaf path is the product of its m's, branches whose running product falls below 1e-5 are pruned, and
 * one complete path is drawn with probability proportional to its weight: the leaves are walked depth first,
 * children by rank (larger probability first, then smaller token), and the first leaf whose cumulative weight
 * exceeds u * total is taken.  If no complete path survives the pruning, the path of every head's most probable
 * token is returned.  zh: [D][V] logits of the heads (row of the first rejection); out: D tokens.
 */
#define ORC_TREE_PRUNE 1e-5
typedef struct { int D, ks; const int *tok; const double *m; double target, cum; int found; int *path, *best; } tree_walk;
static void tree_dfs(tree_walk *w, int depth, double weight, int pass) {
    if (w->found) return;
    if (depth == w->D) {
        w->cum += weight;
        if (pass == 1 && w->cum > w->target) { memcpy(w->best, w->path, sizeof(int) * w->D); w->found = 1; }
        else if (pass == 1) memcpy(w->best, w->path, sizeof(int) * w->D);   /* rounding at the very end: last leaf */
        return;
    }
    for (int k = 0; k < w->ks; ++k) {
        double nw = weight * w->m[depth * w->ks + k];
        if (nw < ORC_TREE_PRUNE) continue;
        w->path[depth] = w->tok[depth * w->ks + k];
        tree_dfs(w, depth + 1, nw, pass);
        if (w->found) return;
    }
}
void orc_sample_tree(const float *zh, int D, int V, int ks, uint32_t r24, int32_t *out) {
    if (ks < 1) ks = 1;
    if (ks > V) ks = V;
    int *tok = (int *)malloc(sizeof(int) * D * ks), *path = (int *)malloc(sizeof(int) * D), *best = (int *)malloc(sizeof(int) * D);
    double *m = (double *)malloc(sizeof(double) * D * ks);
    for (int d = 0; d < D; ++d) {
        const float *z = zh + (size_t)d * V;
        double mx = z[0], sum = 0;
        for (int v = 1; v < V; ++v) if (z[v] > mx) mx = z[v];
        for (int v = 0; v < V; ++v) sum += exp((double)z[v] - mx);
        for (int j = 0; j < ks; ++j) {           /* j-th candidate: best not yet taken */
            int b = -1;
            for (int v = 0; v < V; ++v) {
                if (j > 0 && !before(z, tok[d * ks + j - 1], v)) continue;
                if (b < 0 || before(z, v, b)) b = v;
            }
            tok[d * ks + j] = b;
            m[d * ks + j] = exp((double)z[b] - mx) / sum;
        }
        best[d] = tok[d * ks];
    }
    tree_walk w = {D, ks, tok, m, 0.0, 0.0, 0, path, best};
    tree_dfs(&w, 0, 1.0, 0);                     /* pass 0: total weight of the surviving leaves */
    if (w.cum > 0.0) {
        w.target = (double)r24 * (1.0 / 16777216.0) * w.cum;
        w.cum = 0.0;
        tree_dfs(&w, 0, 1.0, 1);
    }
    for (int d = 0; d < D; ++d) out[d] = best[d];
    free(tok); free(path); free(best); free(m);
}

/* Algorithm 1, line 1: x_0 = SOS, x_{1:D} ~ U(0, V), s = 0 (prompt longer than
 * one token: all but the last prompt token are run into the cache first). */
int orc_seq_begin(orc_seq *s, const int32_t *prompt, int prompt_len, const orc_decode_config *dc) {
    const orc_model_config *c = &s->ctx->c;
    if (prompt_len < 1) return -1;
    seq_release_beyond(s, 0);
    s->len = 0; s->step_idx = 0; s->finished = 0;
    for (int p = 0; p + 1 < prompt_len; ++p) {
        int rc = orc_forward_row(s, prompt[p], p, NULL, NULL);
        if (rc) return rc;
    }
    s->len = prompt_len - 1;
    s->window[0] = prompt[prompt_len - 1];
    for (int i = 1; i <= c->n_draft; ++i) {
        uint64_t m = orc_rand24(dc->seed, s->seq_id, 0, (uint32_t)i, 1);
        s->window[i] = (int32_t)((m * (uint64_t)c->vocab) >> 24);
    }
    return seq_reserve(s, s->len + c->n_draft + 1);
}

/*
 * One iteration of the while loop of Algorithm 1 (lines 3-12).
 * new_tokens[K+1] receives the tokens committed by this step, x_{s+1..s*},
 * padded with -1; *n_new = s* - s.  Optional outputs: logits0[(K+1) V],
 * head_logits[K (K+1) V] as [head][row][V], and g[(K+1) d].
 */
int orc_step(orc_seq *s, const orc_decode_config *dc, int32_t *new_tokens, int *n_new,
             float *logits0_out, float *head_logits_out, float *g_out) {
    orc_ctx *ctx = s->ctx;
    const orc_model_config *c = &ctx->c;
    int K = c->n_draft, V = c->vocab, d = c->d_model, M = K + 1;
    if (seq_reserve(s, s->len + M)) return -2;
    float *z0 = (float *)malloc(sizeof(float) * (size_t)M * V);
    float *g = (float *)malloc(sizeof(float) * (size_t)M * d);
    float *zh = (float *)malloc(sizeof(float) * (size_t)(K > 0 ? K : 1) * M * V);
    /* line 3: backbone over x_{s:s+D} under the causal mask: row j sees the
     * cache and rows < j, which is what running the rows in order gives */
    for (int j = 0; j < M; ++j) {
        int rc = orc_forward_row(s, s->window[j], s->len + j, z0 + (size_t)j * V, g + (size_t)j * d);
        if (rc) { free(z0); free(g); free(zh); return rc; }
    }
    /* lines 4-6: every head on every row of the window */
    for (int i = 1; i <= K; ++i)
        for (int j = 0; j < M; ++j) orc_seq_head(s, i, g + (size_t)j * d, zh + ((size_t)(i - 1) * M + j) * V);
    /* lines 7-10: accept drafts while the backbone agrees */
    int a = 0;
    while (a < K && orc_accept(z0 + (size_t)a * V, V, s->window[a + 1], dc)) ++a;
    /* line 11: resample D+1 candidates from the row of the first rejection */
    int32_t *nw = (int32_t *)malloc(sizeof(int32_t) * M);
    if (dc->sample_mode == 2) {
        /* x_{s*} from the backbone's own distribution (top-K_s logits at the configured temperature), the D drafts
         * as one path of the probability tree; slot 1's random number draws the path */
        orc_decode_config one = *dc;
        one.sample_mode = 1;
        nw[0] = orc_sample(z0 + (size_t)a * V, V, &one, orc_rand24(dc->seed, s->seq_id, s->step_idx, 0, 0));
        if (K > 0) {
            float *rows = (float *)malloc(sizeof(float) * (size_t)K * V);
            for (int i = 1; i <= K; ++i) memcpy(rows + (size_t)(i - 1) * V, zh + ((size_t)(i - 1) * M + a) * V, sizeof(float) * V);
            orc_sample_tree(rows, K, V, dc->k_sample, orc_rand24(dc->seed, s->seq_id, s->step_idx, 1, 0), nw + 1);
            free(rows);
        }
    } else {
        nw[0] = orc_sample(z0 + (size_t)a * V, V, dc, orc_rand24(dc->seed, s->seq_id, s->step_idx, 0, 0));
        for (int i = 1; i <= K; ++i)
            nw[i] = orc_sample(zh + ((size_t)(i - 1) * M + a) * V, V, dc,
                               orc_rand24(dc->seed, s->seq_id, s->step_idx, (uint32_t)i, 0));
    }
    for (int j = 0; j < M; ++j) new_tokens[j] = -1;
    for (int j = 0; j < a; ++j) new_tokens[j] = s->window[j + 1];
    new_tokens[a] = nw[0];
    *n_new = a + 1;
    /* line 12: s <- s*.  Cache rows at positions >= s* are dead; the next
     * window overwrites them.  Pages wholly beyond the next window go back. */
    s->len += a + 1;
    memcpy(s->window, nw, sizeof(int32_t) * M);
    s->step_idx += 1;
    seq_release_beyond(s, s->len + M);
    int rc = seq_reserve(s, s->len + M);
    if (logits0_out) memcpy(logits0_out, z0, sizeof(float) * (size_t)M * V);
    if (head_logits_out && K > 0) memcpy(head_logits_out, zh, sizeof(float) * (size_t)K * M * V);
    if (g_out) memcpy(g_out, g, sizeof(float) * (size_t)M * d);
    free(z0); free(g); free(zh); free(nw);
    return rc;
}

/*
 * Algorithm 1 as a whole for one sequence: generate until max_new tokens are
 * committed, an EOS is committed, or the position limit is reached.  tokens
 * receives x_1.. (the SOS is not repeated); returns the number written.
 * steps_out: decoding steps taken; accept_hist[a] counts steps that accepted a
 * drafts (size K+1).  SCR = tokens committed / steps (Sec. 5.1).
 */
int orc_generate(orc_seq *s, const orc_decode_config *dc, int max_new, int max_positions,
                 int32_t *tokens, uint64_t *steps_out, uint64_t *accept_hist) {
    const orc_model_config *c = &s->ctx->c;
    int K = c->n_draft, n = 0, base = s->len;
    uint64_t steps = 0;
    int32_t *nt = (int32_t *)malloc(sizeof(int32_t) * (K + 1));
    while (!s->finished && n < max_new && s->len + K + 1 <= max_positions) {
        int nn = 0;
        int rc = orc_step(s, dc, nt, &nn, NULL, NULL, NULL);
        if (rc) { free(nt); return rc; }
        ++steps;
        if (accept_hist) accept_hist[nn - 1] += 1;
        for (int j = 0; j < nn && n < max_new; ++j) {
            tokens[n++] = nt[j];
            if (c->eos_id >= 0 && nt[j] == c->eos_id) { s->finished = 1; break; }
        }
    }
    (void)base;
    if (n >= max_new) s->finished = 1;
    if (steps_out) *steps_out = steps;
    free(nt);
    return n;
}

/*
 * Plain one-token-per-step decoding with the backbone alone (Table 3 row A):
 * an independent loop that never drafts, never rejects and never touches a
 * cache slot twice.  Token t+1 = sample(p0 | x_{0:t}); its random number is
 * the one Algorithm 1 would use when every step commits exactly one token.
 */
int orc_generate_plain(orc_seq *s, const int32_t *prompt, int prompt_len, const orc_decode_config *dc,
                       int max_new, int32_t *tokens) {
    const orc_model_config *c = &s->ctx->c;
    seq_release_beyond(s, 0);
    s->len = 0;
    float *z = (float *)malloc(sizeof(float) * c->vocab);
    int pos = 0, n = 0, x = prompt[0];
    for (; pos + 1 < prompt_len; ++pos) {
        int rc = orc_forward_row(s, prompt[pos], pos, NULL, NULL);
        if (rc) { free(z); return rc; }
    }
    x = prompt[prompt_len - 1];
    while (n < max_new) {
        int rc = orc_forward_row(s, x, pos, z, NULL);
        if (rc) { free(z); return rc; }
        x = orc_sample(z, c->vocab, dc, orc_rand24(dc->seed, s->seq_id, (uint32_t)n, 0, 0));
        tokens[n++] = x;
        ++pos;
        s->len = pos;
        if (c->eos_id >= 0 && x == c->eos_id) break;
    }
    free(z);
    return n;
}
