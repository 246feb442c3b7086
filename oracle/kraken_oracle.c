/*
 * Kraken forward pass: plain CPU oracle.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, by-the-definition implementation that the CUDA path is
 * checked against.  It shares no code with the CUDA path and must never be
 * called from the product path; only tests, the smoke check and the benchmark's
 * CPU-baseline leg may load it.
 *
 * What it computes (one sequence at a time), following the paper:
 *   - shared token + position embedding for all sub-layers of layer 1 (Sec. 3.1);
 *   - per layer, per sub-layer n, Algorithm 1:
 *         res = x;  y = AllReduce(x)  (identity in layer 1);  x = LN(x);
 *         x = res + MHA(x);  res = x;  x = LN(x + y);  out = res + FFN(x);
 *     AllReduce is the element-wise sum of the N sub-layer inputs (Sec. 3.1);
 *   - MHA: per head Softmax(Q K^T / sqrt(h)) V with a causal mask, then Wo (Sec. 2.1);
 *   - FFN: two linear maps with GELU between (Sec. 2.1);
 *   - W_concat applied to the branch-major concatenation of the last layer's N
 *     outputs, then (optionally) a final LayerNorm, then the tied unembedding (Sec. 3.1);
 *   - K, V of every token are kept (KV cache); a decode step evaluates the same
 *     equations at one new position against the cached rows (Sec. 2.1).
 *
 * Arithmetic: values are held as fp32, every reduction (dot products, LayerNorm
 * statistics, softmax sums) accumulates in fp64.  Weights arrive as bf16 bit
 * patterns and are widened exactly.  With bf16_store = 1 the activations that a
 * "bf16 activations, fp32 accumulate" implementation keeps in bf16 are rounded
 * (round-to-nearest-even) at those points: both LayerNorm outputs, q/k/v (hence
 * the cache), the attention output, the GELU output, the W_concat input and the
 * final LayerNorm output.  The residual stream and y always stay fp32.
 * The 16-bit type is bfloat16 unless half = 1 in the configuration (IEEE half, the
 * precision of the paper's engines, Sec. 4.2): then the weight patterns are read as
 * half and the store points round to half.
 *
 * Parity status: every step is pinned by the CPU tests (closed forms, brute
 * force, a library composition for the N = 1 reduction, invariants).  The
 * numerical value of the logits for a concrete input is "parity unpinned": the
 * paper prints no worked example.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct ko_config {
    int32_t n_branch, n_layer, d_model, n_head, d_ff, vocab, max_pos;
    float ln_eps;
    int32_t gelu_tanh;   /* 0: erf form, 1: tanh approximation */
    int32_t final_ln;    /* 1: LayerNorm between W_concat and the unembedding */
    int32_t bf16_store;  /* 1: round activations to bf16 at the store points */
    int32_t y_zero;      /* drop the y term: with N = 1 the layers are a standard pre-LN Transformer's
                            (the comparison architecture of Sec. 4.2) */
    int32_t half;        /* 16-bit type of weights and store points: 0 = bfloat16, 1 = IEEE half */
    int32_t parallel_ffn;/* 1: the FFN reads the first LayerNorm's output, in parallel with attention:
                            out = x + MHA(LN(x)) + FFN(LN(x)), the "Parallel Attention + FeedForward"
                            comparison architecture of Sec. 4.2 (no second LayerNorm, no y) */
    int32_t n_kv_head;   /* key/value heads per sub-layer: 0 or n_head = multi-head attention; fewer =
                            grouped-query attention, 1 = multi-query (the KV-cache mitigation of Sec. 4.2
                            and the KV-cache appendix): query head h reads key/value head
                            h / (n_head / n_kv_head) */
} ko_config;

typedef struct ko_weights { /* host pointers to bf16 bit patterns; bias / beta may be NULL */
    const uint16_t *wte, *wpe;
    const uint16_t *ln1_g, *ln1_b, *w_qkv, *b_qkv, *w_proj, *b_proj;
    const uint16_t *ln2_g, *ln2_b, *w_up, *b_up, *w_down, *b_down;
    const uint16_t *w_concat, *b_concat, *lnf_g, *lnf_b;
} ko_weights;

typedef struct ko_state {
    ko_config cfg;
    ko_weights w;
    int32_t cur_len;
    float *kcache; /* [L][N][H_kv][max_pos][hd] */
    float *vcache;
} ko_state;

/* ---------------------------------------------------------------- scalars */

static inline float bf16_to_f32(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

static inline float round_bf16(float f) { /* RNE to bf16, returned as fp32 */
    uint32_t u;
    memcpy(&u, &f, 4);
    u = (u + 0x7FFFu + ((u >> 16) & 1u)) & 0xFFFF0000u;
    memcpy(&f, &u, 4);
    return f;
}

float ko_round_bf16(float f) { return round_bf16(f); }

/* IEEE half (1 sign, 5 exponent, 10 fraction bits) widened exactly. */
static inline float f16_to_f32(uint16_t b) {
    const int sign = b >> 15, e = (b >> 10) & 31, m = b & 1023;
    double v;
    if (e == 0) v = ldexp((double)m, -24);                    /* zero and subnormals: m * 2^-24 */
    else if (e == 31) v = m ? NAN : INFINITY;
    else v = ldexp(1.0 + m / 1024.0, e - 15);
    return (float)(sign ? -v : v);
}

/* fp32 -> nearest half (ties to even, overflow to infinity), returned as fp32: the compiler's IEEE
 * half type does the rounding; the pins check it against an independent implementation. */
static inline float round_f16(float f) { return (float)(_Float16)f; }

float ko_f16_to_f32(uint16_t b) { return f16_to_f32(b); }
float ko_round_f16(float f) { return round_f16(f); }

/* The 16-bit type in force: set from the configuration at the start of every forward pass, or by
 * ko_set_half for the single-step wrappers.  (The oracle is driven from one thread.) */
static int g_half = 0;
void ko_set_half(int on) { g_half = on != 0; }
static inline float h16_to_f32(uint16_t b) { return g_half ? f16_to_f32(b) : bf16_to_f32(b); }
static inline float round_h16(float f) { return g_half ? round_f16(f) : round_bf16(f); }

float ko_gelu(float x, int tanh_form) {
    double v = x;
    if (tanh_form) {
        double c = 0.7978845608028654; /* sqrt(2/pi) */
        return (float)(0.5 * v * (1.0 + tanh(c * (v + 0.044715 * v * v * v))));
    }
    return (float)(0.5 * v * (1.0 + erf(v * 0.7071067811865476)));
}

int ko_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---------------------------------------------------------------- steps */

/* LayerNorm over the last dimension: gamma * (v - mean) / sqrt(var_biased + eps) + beta.
 * in = a (+ b if b != NULL), rows x d.  gamma/beta bf16 bits (beta may be NULL). */
void ko_layernorm(const float *a, const float *b, int rows, int d, const uint16_t *gamma,
                  const uint16_t *beta, float eps, int round_out, float *out) {
#pragma omp parallel for schedule(static)
    for (int r = 0; r < rows; ++r) {
        const float *pa = a + (size_t)r * d;
        const float *pb = b ? b + (size_t)r * d : NULL;
        double mean = 0.0;
        for (int j = 0; j < d; ++j) mean += (double)(pb ? pa[j] + pb[j] : pa[j]);
        mean /= d;
        double var = 0.0;
        for (int j = 0; j < d; ++j) {
            double v = (double)(pb ? pa[j] + pb[j] : pa[j]) - mean;
            var += v * v;
        }
        var /= d;
        double rstd = 1.0 / sqrt(var + (double)eps);
        for (int j = 0; j < d; ++j) {
            double v = ((double)(pb ? pa[j] + pb[j] : pa[j]) - mean) * rstd;
            double g = gamma ? h16_to_f32(gamma[j]) : 1.0;
            double be = beta ? h16_to_f32(beta[j]) : 0.0;
            float o = (float)(v * g + be);
            out[(size_t)r * d + j] = round_out ? round_h16(o) : o;
        }
    }
}

/* out[t, o] = sum_i in[t, i] * W[o, i] + bias[o];  W bf16 bits, row-major [n_out, n_in]
 * with row stride w_stride (elements).  Plain definition; the loop order keeps one
 * weight row hot while the activations stream. */
void ko_linear(const float *in, int rows, int n_in, const uint16_t *W, int64_t w_stride,
               const uint16_t *bias, int n_out, float *out) {
#pragma omp parallel
    {
        float *wrow = (float *)malloc(sizeof(float) * (size_t)n_in);
#pragma omp for schedule(static)
        for (int o = 0; o < n_out; ++o) {
            const uint16_t *wp = W + (size_t)o * (size_t)w_stride;
            for (int i = 0; i < n_in; ++i) wrow[i] = h16_to_f32(wp[i]);
            double bo = bias ? (double)h16_to_f32(bias[o]) : 0.0;
            for (int t = 0; t < rows; ++t) {
                const float *x = in + (size_t)t * n_in;
                double acc = 0.0;
#pragma omp simd reduction(+ : acc)
                for (int i = 0; i < n_in; ++i) acc += (double)x[i] * (double)wrow[i];
                out[(size_t)t * n_out + o] = (float)(acc + bo);
            }
        }
        free(wrow);
    }
}

/* Causal scaled-dot-product attention for one head.
 * Query rows are positions q_pos0 .. q_pos0 + n_q - 1; key/value rows 0 .. are positions.
 * Query at position p sees keys at positions j <= p.
 * q: [n_q, hd] with row stride q_stride; k, v: [*, hd] with row stride kv_stride;
 * out: [n_q, hd] with row stride o_stride. */
void ko_attention_head(const float *q, int64_t q_stride, const float *k, const float *v,
                       int64_t kv_stride, int n_q, int q_pos0, int hd, float *out,
                       int64_t o_stride) {
    double scale = 1.0 / sqrt((double)hd);
#pragma omp parallel
    {
        double *p = (double *)malloc(sizeof(double) * (size_t)(q_pos0 + n_q));
        double *acc = (double *)malloc(sizeof(double) * (size_t)hd);
#pragma omp for schedule(dynamic, 4)
        for (int i = 0; i < n_q; ++i) {
            int n_keys = q_pos0 + i + 1;
            const float *qi = q + (size_t)i * q_stride;
            double m = -INFINITY;
            for (int j = 0; j < n_keys; ++j) {
                const float *kj = k + (size_t)j * kv_stride;
                double s = 0.0;
#pragma omp simd reduction(+ : s)
                for (int c = 0; c < hd; ++c) s += (double)qi[c] * (double)kj[c];
                s *= scale;
                p[j] = s;
                if (s > m) m = s;
            }
            double denom = 0.0;
            for (int j = 0; j < n_keys; ++j) {
                p[j] = exp(p[j] - m);
                denom += p[j];
            }
            for (int c = 0; c < hd; ++c) acc[c] = 0.0;
            for (int j = 0; j < n_keys; ++j) {
                const float *vj = v + (size_t)j * kv_stride;
                double w = p[j] / denom;
                for (int c = 0; c < hd; ++c) acc[c] += w * (double)vj[c];
            }
            for (int c = 0; c < hd; ++c) out[(size_t)i * o_stride + c] = (float)acc[c];
        }
        free(p);
        free(acc);
    }
}

/* ---------------------------------------------------------------- model */

static int kv_heads(const ko_config *c) { return c->n_kv_head > 0 ? c->n_kv_head : c->n_head; }

size_t ko_cache_floats(const ko_config *c) {
    return (size_t)c->n_layer * c->n_branch * (size_t)c->max_pos * kv_heads(c) * (c->d_model / c->n_head);
}

ko_state *ko_create(const ko_config *cfg, const ko_weights *w) {
    if (!cfg || !w) return NULL;
    if (cfg->n_branch < 1 || cfg->n_layer < 1 || cfg->d_model < 1 || cfg->n_head < 1 ||
        cfg->d_model % cfg->n_head != 0 || cfg->d_ff < 1 || cfg->vocab < 1 || cfg->max_pos < 1)
        return NULL;
    if (cfg->n_kv_head < 0 || (cfg->n_kv_head > 0 && cfg->n_head % cfg->n_kv_head != 0)) return NULL;
    ko_state *s = (ko_state *)calloc(1, sizeof(ko_state));
    if (!s) return NULL;
    s->cfg = *cfg;
    s->w = *w;
    s->kcache = (float *)calloc(ko_cache_floats(cfg), sizeof(float));
    s->vcache = (float *)calloc(ko_cache_floats(cfg), sizeof(float));
    if (!s->kcache || !s->vcache) {
        free(s->kcache);
        free(s->vcache);
        free(s);
        return NULL;
    }
    return s;
}

void ko_destroy(ko_state *s) {
    if (!s) return;
    free(s->kcache);
    free(s->vcache);
    free(s);
}

int ko_cur_len(const ko_state *s) { return s ? s->cur_len : -1; }

/* Pointer to the cached K (which = 0) or V (which = 1) rows of (layer, branch, key/value head):
 * [max_pos, hd] contiguous. */
const float *ko_cache_ptr(const ko_state *s, int layer, int branch, int which, int head) {
    const ko_config *c = &s->cfg;
    int hd = c->d_model / c->n_head;
    size_t off = ((((size_t)layer * c->n_branch + branch) * kv_heads(c) + head) * (size_t)c->max_pos) * hd;
    return (which ? s->vcache : s->kcache) + off;
}

static void maybe_round(float *x, size_t n, int on) {
    if (!on) return;
#pragma omp parallel for schedule(static)
    for (size_t i = 0; i < n; ++i) x[i] = round_h16(x[i]);
}

/* Evaluate positions pos0 .. pos0 + n - 1 of the sequence whose first pos0 positions
 * are already in the cache (pos0 = 0: prefill; n = 1: decode step).
 *   ids         [n] token ids of the new positions
 *   logits      [n - logits_from, V] for new rows logits_from .. n-1 (NULL: skip tail)
 *   layer_out   optional [L][N][n][d]: every sub-layer's output (the x fed to the next layer)
 * Returns 0, or a negative code: -1 bad argument, -2 capacity, -3 token id out of range,
 * -4 out of memory. */
static int forward(ko_state *s, const int32_t *ids, int n, int pos0, float *logits,
                   int logits_from, float *layer_out) {
    const ko_config *c = &s->cfg;
    const ko_weights *w = &s->w;
    g_half = c->half != 0;
    const int N = c->n_branch, L = c->n_layer, d = c->d_model, H = c->n_head, F = c->d_ff, V = c->vocab;
    const int hd = d / H, rb = c->bf16_store;
    const int Hkv = kv_heads(c), kvd = Hkv * hd, qw = d + 2 * kvd; /* q | k | v row: d + 2 H_kv hd columns */
    if (!ids || n < 1 || pos0 < 0) return -1;
    if (pos0 + n > c->max_pos) return -2;
    for (int t = 0; t < n; ++t)
        if (ids[t] < 0 || ids[t] >= V) return -3;

    const size_t nd = (size_t)n * d;
    float *x0 = (float *)malloc(sizeof(float) * nd);
    float *x = (float *)malloc(sizeof(float) * nd * N);     /* x_n, sub-layer inputs  */
    float *xn = (float *)malloc(sizeof(float) * nd * N);    /* next layer's inputs    */
    float *y = (float *)malloc(sizeof(float) * nd);
    float *u = (float *)malloc(sizeof(float) * nd);
    float *qkv = (float *)malloc(sizeof(float) * (size_t)n * qw);
    float *o = (float *)malloc(sizeof(float) * nd);
    float *a = (float *)malloc(sizeof(float) * nd);
    float *hh = (float *)malloc(sizeof(float) * nd);
    float *g = (float *)malloc(sizeof(float) * (size_t)n * F);
    float *tmp = (float *)malloc(sizeof(float) * nd);
    if (!x0 || !x || !xn || !y || !u || !qkv || !o || !a || !hh || !g || !tmp) {
        free(x0); free(x); free(xn); free(y); free(u); free(qkv); free(o); free(a); free(hh); free(g); free(tmp);
        return -4;
    }

    /* shared embedding: token row + position row */
    for (int t = 0; t < n; ++t)
        for (int j = 0; j < d; ++j)
            x0[(size_t)t * d + j] = h16_to_f32(w->wte[(size_t)ids[t] * d + j]) +
                                    h16_to_f32(w->wpe[(size_t)(pos0 + t) * d + j]);
    for (int b = 0; b < N; ++b) memcpy(x + nd * b, x0, sizeof(float) * nd);

    for (int l = 0; l < L; ++l) {
        /* y: identity in the first layer, otherwise the sum over all N sub-layer inputs */
        if (l == 0) {
            memcpy(y, x0, sizeof(float) * nd);
        } else {
            for (size_t i = 0; i < nd; ++i) {
                double acc = 0.0;
                for (int m = 0; m < N; ++m) acc += (double)x[nd * m + i];
                y[i] = (float)acc;
            }
        }
        if (c->y_zero) memset(y, 0, sizeof(float) * nd);

        for (int b = 0; b < N; ++b) {
            const size_t ln = (size_t)l * N + b;
            const float *xb = x + nd * b;
            /* x = LN(x) */
            ko_layernorm(xb, NULL, n, d, w->ln1_g + ln * d, w->ln1_b ? w->ln1_b + ln * d : NULL,
                         c->ln_eps, rb, u);
            /* q | k | v */
            ko_linear(u, n, d, w->w_qkv + ln * (size_t)qw * d, d,
                      w->b_qkv ? w->b_qkv + ln * qw : NULL, qw, qkv);
            maybe_round(qkv, (size_t)n * qw, rb);
            /* memoise k, v (one row per key/value head) */
            for (int h = 0; h < Hkv; ++h) {
                float *kc = (float *)ko_cache_ptr(s, l, b, 0, h);
                float *vc = (float *)ko_cache_ptr(s, l, b, 1, h);
                for (int t = 0; t < n; ++t)
                    for (int e = 0; e < hd; ++e) {
                        kc[(size_t)(pos0 + t) * hd + e] = qkv[(size_t)t * qw + d + h * hd + e];
                        vc[(size_t)(pos0 + t) * hd + e] = qkv[(size_t)t * qw + d + kvd + h * hd + e];
                    }
            }
            /* attention per query head over the cached rows of its key/value head */
            for (int h = 0; h < H; ++h) {
                const int hk = h / (H / Hkv);
                ko_attention_head(qkv + h * hd, (int64_t)qw, ko_cache_ptr(s, l, b, 0, hk),
                                  ko_cache_ptr(s, l, b, 1, hk), hd, n, pos0, hd, o + h * hd, d);
            }
            maybe_round(o, nd, rb);
            /* x = res + MHA */
            ko_linear(o, n, d, w->w_proj + ln * (size_t)d * d, d, w->b_proj ? w->b_proj + ln * d : NULL, d, tmp);
            for (size_t i = 0; i < nd; ++i) a[i] = xb[i] + tmp[i];
            /* x = LN(x + y); in the parallel variant the FFN takes the first LayerNorm's output instead */
            if (c->parallel_ffn)
                memcpy(hh, u, sizeof(float) * nd);
            else
                ko_layernorm(a, y, n, d, w->ln2_g + ln * d, w->ln2_b ? w->ln2_b + ln * d : NULL, c->ln_eps, rb, hh);
            /* out = res + FFN(x) */
            ko_linear(hh, n, d, w->w_up + ln * (size_t)F * d, d, w->b_up ? w->b_up + ln * F : NULL, F, g);
            for (size_t i = 0; i < (size_t)n * F; ++i) {
                float v = ko_gelu(g[i], c->gelu_tanh);
                g[i] = rb ? round_h16(v) : v;
            }
            ko_linear(g, n, F, w->w_down + ln * (size_t)d * F, F, w->b_down ? w->b_down + ln * d : NULL, d, tmp);
            float *ob = xn + nd * b;
            for (size_t i = 0; i < nd; ++i) ob[i] = a[i] + tmp[i];
            if (layer_out) memcpy(layer_out + (ln * (size_t)n) * d, ob, sizeof(float) * nd);
        }
        float *sw = x; x = xn; xn = sw;
    }

    if (logits) {
        const int nr = n - logits_from;
        if (nr > 0) {
            /* branch-major concatenation, then W_concat */
            float *cat = (float *)malloc(sizeof(float) * (size_t)nr * N * d);
            float *z = (float *)malloc(sizeof(float) * (size_t)nr * d);
            float *zf = (float *)malloc(sizeof(float) * (size_t)nr * d);
            if (!cat || !z || !zf) {
                free(cat); free(z); free(zf);
                free(x0); free(x); free(xn); free(y); free(u); free(qkv); free(o); free(a); free(hh); free(g); free(tmp);
                return -4;
            }
            for (int t = 0; t < nr; ++t)
                for (int b = 0; b < N; ++b)
                    for (int j = 0; j < d; ++j) {
                        float v = x[nd * b + (size_t)(logits_from + t) * d + j];
                        cat[((size_t)t * N + b) * d + j] = rb ? round_h16(v) : v;
                    }
            ko_linear(cat, nr, N * d, w->w_concat, (int64_t)N * d, w->b_concat, d, z);
            if (c->final_ln)
                ko_layernorm(z, NULL, nr, d, w->lnf_g, w->lnf_b, c->ln_eps, rb, zf);
            else {
                memcpy(zf, z, sizeof(float) * (size_t)nr * d);
                maybe_round(zf, (size_t)nr * d, rb);
            }
            /* tied unembedding */
            ko_linear(zf, nr, d, w->wte, d, NULL, V, logits);
            free(cat); free(z); free(zf);
        }
    }
    free(x0); free(x); free(xn); free(y); free(u); free(qkv); free(o); free(a); free(hh); free(g); free(tmp);
    return 0;
}

int ko_prefill(ko_state *s, const int32_t *ids, int l, float *logits, int logits_from, float *layer_out) {
    if (!s) return -1;
    if (logits_from < 0 || logits_from > l) return -1;
    int rc = forward(s, ids, l, 0, logits, logits_from, layer_out);
    if (rc == 0) s->cur_len = l;
    return rc;
}

int ko_decode_step(ko_state *s, int32_t id, float *logits) {
    if (!s) return -1;
    if (s->cur_len < 1) return -1;
    int rc = forward(s, &id, 1, s->cur_len, logits, 0, NULL);
    if (rc == 0) s->cur_len += 1;
    return rc;
}
