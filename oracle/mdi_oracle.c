/* CPU checker for recurrent-pipeline autoregressive decoding (MDI-LLM).
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product path may call into this
 * file; it exists so that the CUDA library can be compared, element by
 * element, with a slow and obviously correct implementation.  It shares no
 * code, header, table or constant with the CUDA path.
 *
 * What it computes.  The paper's method (Section III) cuts a decoder-only
 * transformer into contiguous chunks of blocks, keeps one key/value cache per
 * text sample per chunk (Section III-D), and moves one activation vector per
 * sample from chunk to chunk (Section III-C).  None of that changes the
 * mathematics: every sample's output is that of plain greedy decoding with the
 * whole model.  This file therefore provides
 *   - the elementary operations (norms, linear map, activations, rotary
 *     embedding, causal attention, argmax), each callable on its own so that
 *     the tests can pin it to a closed form or to a library routine;
 *   - orc_full_forward: the whole decoder on a whole sequence, no cache;
 *   - orc_blocks_cached: blocks [lo,hi) applied to T new positions of one
 *     sample, extending that sample's cache (a chunk's "forward" in
 *     Algorithms 1 and 2, for the first visit T = prompt length, later T = 1);
 *   - orc_embed / orc_head: the starter node's input and output layers.
 * The schedulers (sequential generation, and the literal two-algorithm
 * simulation with FIFO queues) are written in Python on top of these.
 *
 * Precision.  Storage of weights is what the harness supplies (fp32, or
 * bfloat16 bit patterns widened exactly); activations, caches and logits are
 * fp32; every dot product, norm statistic, softmax and activation function is
 * evaluated in fp64 and rounded once to fp32.  The checker's own rounding
 * error is therefore negligible beside the tolerances of the comparison.
 *
 * The block structure (attention + fully connected layer, each with a residual
 * connection) is the one the paper states in Section III-B; the concrete
 * GPT-2-style and Llama-style formulas are the standard published ones.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int arch;         /* 0: GPT (LayerNorm, learned positions, biases, GELU); 1: Llama (RMSNorm, RoPE, SwiGLU) */
    int n_layer, d_model, n_head, head_dim, n_kv_head, d_ff, vocab, n_ctx;
    int weight_dtype; /* 0 fp32, 1 bfloat16 bits */
    int tied_lm_head, has_bias;
    int act;          /* 0 GELU (tanh form), 1 GELU (erf form), 2 SwiGLU */
    float norm_eps, rope_theta;
} orc_shape;

typedef struct {
    const void *ln1_g, *ln1_b, *wqkv, *bqkv, *wo, *bo, *ln2_g, *ln2_b;
    const void *w1, *b1, *w2, *b2, *wgate, *wup, *wdown;
} orc_layer;

typedef struct {
    orc_shape s;
    const void *wte, *wpe, *lnf_g, *lnf_b, *lm_head;
    orc_layer *layer;
} orc_model;

/* One sample's cache for the blocks [lo,hi) of one chunk. */
typedef struct {
    int lo, hi, n_ctx, kv_width, len;
    float *k, *v; /* [hi-lo][n_ctx][kv_width] */
} orc_cache;

/* ---------- element access ---------- */
static inline float bf16_to_f32(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}
static inline double wget(const void *p, int dt, size_t i) {
    return dt == 0 ? (double)((const float *)p)[i] : (double)bf16_to_f32(((const uint16_t *)p)[i]);
}

/* ---------- model / cache objects ---------- */
orc_model *orc_model_new(const orc_shape *s) {
    orc_model *m = (orc_model *)calloc(1, sizeof(orc_model));
    m->s = *s;
    m->layer = (orc_layer *)calloc((size_t)s->n_layer, sizeof(orc_layer));
    return m;
}
void orc_model_free(orc_model *m) {
    if (!m) return;
    free(m->layer);
    free(m);
}
/* Names: "wte", "wpe", "lnf.g", "lnf.b", "lm_head", "h.<i>.<field>".  The caller keeps the data alive. */
int orc_model_set(orc_model *m, const char *name, const void *data) {
    if (!strcmp(name, "wte")) { m->wte = data; return 0; }
    if (!strcmp(name, "wpe")) { m->wpe = data; return 0; }
    if (!strcmp(name, "lnf.g")) { m->lnf_g = data; return 0; }
    if (!strcmp(name, "lnf.b")) { m->lnf_b = data; return 0; }
    if (!strcmp(name, "lm_head")) { m->lm_head = data; return 0; }
    if (name[0] == 'h' && name[1] == '.') {
        char *end;
        long i = strtol(name + 2, &end, 10);
        if (i < 0 || i >= m->s.n_layer || *end != '.') return -1;
        const char *f = end + 1;
        orc_layer *L = &m->layer[i];
        struct { const char *n; const void **p; } tab[] = {
            {"ln1.g", &L->ln1_g}, {"ln1.b", &L->ln1_b}, {"attn.wqkv", &L->wqkv}, {"attn.bqkv", &L->bqkv},
            {"attn.wo", &L->wo}, {"attn.bo", &L->bo}, {"ln2.g", &L->ln2_g}, {"ln2.b", &L->ln2_b},
            {"mlp.w1", &L->w1}, {"mlp.b1", &L->b1}, {"mlp.w2", &L->w2}, {"mlp.b2", &L->b2},
            {"mlp.wgate", &L->wgate}, {"mlp.wup", &L->wup}, {"mlp.wdown", &L->wdown}};
        for (size_t k = 0; k < sizeof(tab) / sizeof(tab[0]); ++k)
            if (!strcmp(f, tab[k].n)) { *tab[k].p = data; return 0; }
    }
    return -1;
}

orc_cache *orc_cache_new(const orc_model *m, int lo, int hi) {
    orc_cache *c = (orc_cache *)calloc(1, sizeof(orc_cache));
    c->lo = lo; c->hi = hi; c->n_ctx = m->s.n_ctx;
    c->kv_width = m->s.n_kv_head * m->s.head_dim;
    size_t n = (size_t)(hi - lo) * (size_t)c->n_ctx * (size_t)c->kv_width;
    c->k = (float *)calloc(n ? n : 1, sizeof(float));
    c->v = (float *)calloc(n ? n : 1, sizeof(float));
    return c;
}
void orc_cache_free(orc_cache *c) {
    if (!c) return;
    free(c->k); free(c->v); free(c);
}
int orc_cache_len(const orc_cache *c) { return c->len; }

/* ---------- elementary operations ---------- */

/* LayerNorm over the last axis: (x - mean) / sqrt(var + eps) * g + b, biased variance. */
void orc_layernorm(const float *x, const void *g, const void *b, int dt, int d, double eps, float *y) {
    double mean = 0.0, var = 0.0;
    for (int i = 0; i < d; ++i) mean += (double)x[i];
    mean /= d;
    for (int i = 0; i < d; ++i) { double c = (double)x[i] - mean; var += c * c; }
    var /= d;
    double r = 1.0 / sqrt(var + eps);
    for (int i = 0; i < d; ++i) {
        double v = ((double)x[i] - mean) * r * wget(g, dt, (size_t)i);
        if (b) v += wget(b, dt, (size_t)i);
        y[i] = (float)v;
    }
}

/* RMSNorm: x / sqrt(mean(x^2) + eps) * g. */
void orc_rmsnorm(const float *x, const void *g, int dt, int d, double eps, float *y) {
    double ss = 0.0;
    for (int i = 0; i < d; ++i) ss += (double)x[i] * (double)x[i];
    double r = 1.0 / sqrt(ss / d + eps);
    for (int i = 0; i < d; ++i) y[i] = (float)((double)x[i] * r * wget(g, dt, (size_t)i));
}

/* Y[t][o] = sum_i W[o][i] * X[t][i] + b[o];  W row-major [n_out][n_in]. */
void orc_linear(const void *W, const void *b, int dt, int n_out, int n_in, const float *X, int T, float *Y) {
#pragma omp parallel for schedule(static)
    for (int o = 0; o < n_out; ++o) {
        double bias = b ? wget(b, dt, (size_t)o) : 0.0;
        for (int t = 0; t < T; ++t) {
            const float *x = X + (size_t)t * n_in;
            double acc = 0.0;
            if (dt == 0) {
                const float *w = (const float *)W + (size_t)o * n_in;
#pragma omp simd reduction(+ : acc)
                for (int i = 0; i < n_in; ++i) acc += (double)w[i] * (double)x[i];
            } else {
                const uint16_t *w = (const uint16_t *)W + (size_t)o * n_in;
#pragma omp simd reduction(+ : acc)
                for (int i = 0; i < n_in; ++i) acc += (double)bf16_to_f32(w[i]) * (double)x[i];
            }
            Y[(size_t)t * n_out + o] = (float)(acc + bias);
        }
    }
}

double orc_gelu_tanh(double x) {
    return 0.5 * x * (1.0 + tanh(0.79788456080286535587989211986876 * (x + 0.044715 * x * x * x)));
}
double orc_gelu_erf(double x) { return 0.5 * x * (1.0 + erf(x * 0.70710678118654752440084436210485)); }
double orc_silu(double x) { return x / (1.0 + exp(-x)); }

/* Rotary embedding of one head vector at position pos, split-halves pairing:
 * element i pairs with i + hd/2, angle = pos * theta^(-2i/hd).  cos and sin are
 * evaluated in fp64 from the integer position and rounded to fp32 first. */
void orc_rope(float *v, int hd, int pos, double theta) {
    int half = hd / 2;
    for (int i = 0; i < half; ++i) {
        double ang = (double)pos * pow(theta, -2.0 * (double)i / (double)hd);
        double c = (double)(float)cos(ang), s = (double)(float)sin(ang);
        double a = (double)v[i], b = (double)v[i + half];
        v[i] = (float)(a * c - b * s);
        v[i + half] = (float)(b * c + a * s);
    }
}

/* One query head against n_keys cached rows: softmax(q.K_j / sqrt(hd)) weighted sum of V_j.
 * K and V rows are `stride` floats apart. */
void orc_attend(const float *q, const float *K, const float *V, int n_keys, int hd, size_t stride, float *out) {
    double *p = (double *)malloc((size_t)n_keys * sizeof(double));
    double scale = 1.0 / sqrt((double)hd), mx = -INFINITY;
    for (int j = 0; j < n_keys; ++j) {
        double s = 0.0;
        const float *k = K + (size_t)j * stride;
        for (int e = 0; e < hd; ++e) s += (double)q[e] * (double)k[e];
        p[j] = s * scale;
        if (p[j] > mx) mx = p[j];
    }
    double sum = 0.0;
    for (int j = 0; j < n_keys; ++j) { p[j] = exp(p[j] - mx); sum += p[j]; }
    for (int e = 0; e < hd; ++e) {
        double acc = 0.0;
        for (int j = 0; j < n_keys; ++j) acc += p[j] * (double)V[(size_t)j * stride + e];
        out[e] = (float)(acc / sum);
    }
    free(p);
}

/* Index of the largest value; the lowest index wins a tie. */
int orc_argmax(const float *x, int n) {
    int best = 0;
    for (int i = 1; i < n; ++i) if (x[i] > x[best]) best = i;
    return best;
}

/* ---------- model pieces ---------- */

static void norm_rows(const orc_model *m, const void *g, const void *b, const float *X, int T, float *Y) {
    const orc_shape *s = &m->s;
    for (int t = 0; t < T; ++t) {
        if (s->arch == 0) orc_layernorm(X + (size_t)t * s->d_model, g, b, s->weight_dtype, s->d_model, s->norm_eps, Y + (size_t)t * s->d_model);
        else orc_rmsnorm(X + (size_t)t * s->d_model, g, s->weight_dtype, s->d_model, s->norm_eps, Y + (size_t)t * s->d_model);
    }
}

/* Input layers of the starter node: token embedding (+ learned position embedding for GPT). */
void orc_embed(const orc_model *m, const int32_t *tok, int T, int pos0, float *X) {
    const orc_shape *s = &m->s;
    for (int t = 0; t < T; ++t)
        for (int i = 0; i < s->d_model; ++i) {
            double v = wget(m->wte, s->weight_dtype, (size_t)tok[t] * s->d_model + i);
            if (s->arch == 0) v += wget(m->wpe, s->weight_dtype, (size_t)(pos0 + t) * s->d_model + i);
            X[(size_t)t * s->d_model + i] = (float)v;
        }
}

/* Output layers: final norm, then the vocabulary projection (tied to wte if so configured). */
void orc_head(const orc_model *m, const float *x, float *logits) {
    const orc_shape *s = &m->s;
    float *n = (float *)malloc((size_t)s->d_model * sizeof(float));
    norm_rows(m, m->lnf_g, m->lnf_b, x, 1, n);
    orc_linear(s->tied_lm_head ? m->wte : m->lm_head, NULL, s->weight_dtype, s->vocab, s->d_model, n, 1, logits);
    free(n);
}

/* The fully connected half of a block applied to normalised rows N -> M (no residual). */
static void mlp_rows(const orc_model *m, const orc_layer *L, const float *N, int T, float *M) {
    const orc_shape *s = &m->s;
    int d = s->d_model, F = s->d_ff, dt = s->weight_dtype;
    float *f = (float *)malloc((size_t)T * F * sizeof(float));
    if (s->act == 2) {
        float *u = (float *)malloc((size_t)T * F * sizeof(float));
        orc_linear(L->wgate, NULL, dt, F, d, N, T, f);
        orc_linear(L->wup, NULL, dt, F, d, N, T, u);
        for (size_t i = 0; i < (size_t)T * F; ++i) f[i] = (float)(orc_silu((double)f[i]) * (double)u[i]);
        orc_linear(L->wdown, NULL, dt, d, F, f, T, M);
        free(u);
    } else {
        orc_linear(L->w1, L->b1, dt, F, d, N, T, f);
        for (size_t i = 0; i < (size_t)T * F; ++i)
            f[i] = (float)(s->act == 0 ? orc_gelu_tanh((double)f[i]) : orc_gelu_erf((double)f[i]));
        orc_linear(L->w2, L->b2, dt, d, F, f, T, M);
    }
    free(f);
}

/* Blocks [cache->lo, cache->hi) on T new positions of one sample (X in/out, [T][d]).
 * The new positions are cache->len .. cache->len+T-1; their keys and values are
 * appended to the cache and every new position attends to all rows up to itself. */
int orc_blocks_cached(const orc_model *m, orc_cache *c, float *X, int T) {
    const orc_shape *s = &m->s;
    int d = s->d_model, H = s->n_head, hd = s->head_dim, Hk = s->n_kv_head, dt = s->weight_dtype;
    int qw = H * hd, kw = Hk * hd, rows = qw + 2 * kw, p0 = c->len;
    if (p0 + T > c->n_ctx) return -1;
    float *N = (float *)malloc((size_t)T * d * sizeof(float));
    float *QKV = (float *)malloc((size_t)T * rows * sizeof(float));
    float *O = (float *)malloc((size_t)T * qw * sizeof(float));
    float *A = (float *)malloc((size_t)T * d * sizeof(float));
    for (int l = c->lo; l < c->hi; ++l) {
        const orc_layer *L = &m->layer[l];
        float *Kc = c->k + (size_t)(l - c->lo) * c->n_ctx * kw;
        float *Vc = c->v + (size_t)(l - c->lo) * c->n_ctx * kw;
        norm_rows(m, L->ln1_g, L->ln1_b, X, T, N);
        orc_linear(L->wqkv, L->bqkv, dt, rows, d, N, T, QKV);
        for (int t = 0; t < T; ++t) {
            float *q = QKV + (size_t)t * rows, *k = q + qw, *v = k + kw;
            if (s->arch == 1) {
                for (int h = 0; h < H; ++h) orc_rope(q + h * hd, hd, p0 + t, s->rope_theta);
                for (int h = 0; h < Hk; ++h) orc_rope(k + h * hd, hd, p0 + t, s->rope_theta);
            }
            memcpy(Kc + (size_t)(p0 + t) * kw, k, (size_t)kw * sizeof(float));
            memcpy(Vc + (size_t)(p0 + t) * kw, v, (size_t)kw * sizeof(float));
        }
#pragma omp parallel for collapse(2) schedule(static)
        for (int t = 0; t < T; ++t)
            for (int h = 0; h < H; ++h) {
                int hk = h / (H / Hk);
                orc_attend(QKV + (size_t)t * rows + h * hd, Kc + hk * hd, Vc + hk * hd, p0 + t + 1, hd, (size_t)kw,
                           O + (size_t)t * qw + h * hd);
            }
        orc_linear(L->wo, L->bo, dt, d, qw, O, T, A);
        for (size_t i = 0; i < (size_t)T * d; ++i) X[i] = X[i] + A[i];
        norm_rows(m, L->ln2_g, L->ln2_b, X, T, N);
        mlp_rows(m, L, N, T, A);
        for (size_t i = 0; i < (size_t)T * d; ++i) X[i] = X[i] + A[i];
    }
    c->len += T;
    free(N); free(QKV); free(O); free(A);
    return 0;
}

/* The whole decoder on a whole sequence, without any cache: logits for every position.
 * Attention is written as the full T x T score matrix with the entries above the
 * diagonal masked out. */
int orc_full_forward(const orc_model *m, const int32_t *tok, int T, float *logits /* [T][vocab] */) {
    const orc_shape *s = &m->s;
    int d = s->d_model, H = s->n_head, hd = s->head_dim, Hk = s->n_kv_head, dt = s->weight_dtype;
    int qw = H * hd, kw = Hk * hd, rows = qw + 2 * kw;
    if (T > s->n_ctx) return -1;
    float *X = (float *)malloc((size_t)T * d * sizeof(float));
    float *N = (float *)malloc((size_t)T * d * sizeof(float));
    float *QKV = (float *)malloc((size_t)T * rows * sizeof(float));
    float *O = (float *)malloc((size_t)T * qw * sizeof(float));
    float *A = (float *)malloc((size_t)T * d * sizeof(float));
    double *S = (double *)malloc((size_t)T * T * sizeof(double));
    orc_embed(m, tok, T, 0, X);
    for (int l = 0; l < s->n_layer; ++l) {
        const orc_layer *L = &m->layer[l];
        norm_rows(m, L->ln1_g, L->ln1_b, X, T, N);
        orc_linear(L->wqkv, L->bqkv, dt, rows, d, N, T, QKV);
        if (s->arch == 1)
            for (int t = 0; t < T; ++t) {
                for (int h = 0; h < H; ++h) orc_rope(QKV + (size_t)t * rows + h * hd, hd, t, s->rope_theta);
                for (int h = 0; h < Hk; ++h) orc_rope(QKV + (size_t)t * rows + qw + h * hd, hd, t, s->rope_theta);
            }
        for (int h = 0; h < H; ++h) {
            int hk = h / (H / Hk);
            for (int i = 0; i < T; ++i)
                for (int j = 0; j < T; ++j) {
                    if (j > i) { S[(size_t)i * T + j] = -INFINITY; continue; }
                    const float *q = QKV + (size_t)i * rows + h * hd;
                    const float *k = QKV + (size_t)j * rows + qw + hk * hd;
                    double a = 0.0;
                    for (int e = 0; e < hd; ++e) a += (double)q[e] * (double)k[e];
                    S[(size_t)i * T + j] = a / sqrt((double)hd);
                }
            for (int i = 0; i < T; ++i) {
                double mx = -INFINITY, sum = 0.0;
                for (int j = 0; j < T; ++j) if (S[(size_t)i * T + j] > mx) mx = S[(size_t)i * T + j];
                for (int j = 0; j < T; ++j) { S[(size_t)i * T + j] = exp(S[(size_t)i * T + j] - mx); sum += S[(size_t)i * T + j]; }
                for (int e = 0; e < hd; ++e) {
                    double a = 0.0;
                    for (int j = 0; j < T; ++j) a += S[(size_t)i * T + j] * (double)QKV[(size_t)j * rows + qw + kw + hk * hd + e];
                    O[(size_t)i * qw + h * hd + e] = (float)(a / sum);
                }
            }
        }
        orc_linear(L->wo, L->bo, dt, d, qw, O, T, A);
        for (size_t i = 0; i < (size_t)T * d; ++i) X[i] = X[i] + A[i];
        norm_rows(m, L->ln2_g, L->ln2_b, X, T, N);
        mlp_rows(m, L, N, T, A);
        for (size_t i = 0; i < (size_t)T * d; ++i) X[i] = X[i] + A[i];
    }
    for (int t = 0; t < T; ++t) orc_head(m, X + (size_t)t * d, logits + (size_t)t * s->vocab);
    free(X); free(N); free(QKV); free(O); free(A); free(S);
    return 0;
}

int orc_num_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
