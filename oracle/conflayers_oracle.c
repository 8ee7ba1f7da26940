/*
 * ConfLayers CPU oracle -- TEST INFRASTRUCTURE, NOT A PRODUCT PATH.
 *
 * A plain, slow, obviously-correct implementation of what the self-speculative
 * decode hot path computes, written from the paper's statement of the method:
 *   - the Llama-style target model the paper runs on (Section 4.1.1): RMSNorm, rotary
 *     position embedding, softmax attention with a KV cache, SwiGLU FFN, shared LM head;
 *   - the draft model = the same model with the layers of the skip set S left out
 *     (Section 3, Figure 2);
 *   - per-layer early-exit logits through the shared LM head and the entropy
 *     confidence (Section 3.1, Eq. 1-4).
 * The draft/verify/accept cycle and the skip-set selection (Eq. 5-10) live in the Python
 * files beside this one.
 *
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call this; it shares
 * no code with the CUDA library and the CUDA library never calls it.
 *
 * Arithmetic: weights are read in their storage type (fp32, or bf16 / fp16 bit patterns widened
 * exactly); activations are kept as fp32 values; every dot product, norm, softmax and entropy
 * sum is accumulated in double.  There is no blocking, fusion or reordering: each output
 * element is one straight loop over its inputs.  OpenMP only spreads independent output rows
 * over threads.  The KV cache and hidden-state taps are rounded (RNE) to the model's storage
 * type when stored, as a model loaded in a 16-bit type does (parity pinned only for the
 * fp32 path, see tests; the 16-bit storage rounding itself is "parity unpinned" against the
 * authors' stack, which is not available).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int n_layers, d_model, n_heads, head_dim, d_ffn, vocab, max_seq;
    float rms_eps, rope_theta;
    int weight_dtype; /* 0 = fp32, 1 = bf16, 2 = fp16 (also the storage type of KV cache and taps) */
    int n_kv_heads;   /* key/value heads (grouped-query attention): query head h reads key/value head h / (n_heads / n_kv_heads) */
} orc_cfg;

typedef struct {
    orc_cfg c;
    const void *embed, *lm_head;
    const float *final_norm;
    const void **wq, **wk, **wv, **wo, **wg, **wu, **wd;
    const float **norm1, **norm2;
    float *kcache, *vcache; /* [L][max_seq][n_kv_heads * head_dim], values already rounded to the storage type */
} orc_model;

/* ---- storage-type helpers ------------------------------------------------------------ */

static inline float bf16_bits_to_f32(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* round-to-nearest-even fp32 -> bf16 -> fp32 */
float orc_round_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return f; /* NaN */
    u += 0x7fffu + ((u >> 16) & 1u);
    u &= 0xffff0000u;
    memcpy(&f, &u, 4);
    return f;
}

/* IEEE 754 binary16 (1 sign, 5 exponent, 10 fraction bits) -> fp32, exact */
float orc_fp16_bits_to_f32(uint16_t b) {
    const int sign = b >> 15, e = (b >> 10) & 31, frac = b & 1023;
    double v;
    if (e == 31) v = frac ? NAN : INFINITY;
    else if (e == 0) v = ldexp((double)frac, -24);            /* subnormal: frac * 2^-24 */
    else v = ldexp(1.0 + (double)frac / 1024.0, e - 15);
    return (float)(sign ? -v : v);
}

/* all 65536 widenings, filled once: under a lock, and published only after the table is complete (threads of a
 * parallel region may arrive here together) */
static const float *fp16_table(void) {
    static float table[65536];
    static int ready = 0;
    int r;
#pragma omp atomic read
    r = ready;
    if (!r) {
#pragma omp critical(orc_fp16_table)
        {
            if (!ready) {
                for (int b = 0; b < 65536; ++b) table[b] = orc_fp16_bits_to_f32((uint16_t)b);
#pragma omp flush
#pragma omp atomic write
                ready = 1;
            }
        }
    }
    return table;
}

/* round-to-nearest-even fp32 -> fp16 -> fp32, from the definition: the representable neighbours of |f| are
 * multiples of the spacing 2^(E-10) with E = max(floor(log2 |f|), -14); ties go to the even multiple; what rounds to
 * 2^16 or beyond is infinity. */
float orc_round_fp16(float f) {
    if (isnan(f) || isinf(f) || f == 0.0f) return f;
    const double a = fabs((double)f);
    int E;
    frexp(a, &E);      /* a = m * 2^E with m in [0.5, 1): floor(log2 a) = E - 1 */
    E -= 1;
    if (E < -14) E = -14;
    const double ulp = ldexp(1.0, E - 10);
    double q = a / ulp, fl = floor(q), r = q - fl;
    if (r > 0.5 || (r == 0.5 && fmod(fl, 2.0) == 1.0)) fl += 1.0;
    double v = fl * ulp;
    if (v >= 65520.0) v = INFINITY;   /* beyond the largest finite value 65504 plus half a spacing */
    return (float)(f < 0 ? -v : v);
}

static inline float store_round(float f, int dtype) { return dtype == 1 ? orc_round_bf16(f) : dtype == 2 ? orc_round_fp16(f) : f; }

static inline float wload(const void *w, size_t i, int dtype) {
    return dtype == 1   ? bf16_bits_to_f32(((const uint16_t *)w)[i])
           : dtype == 2 ? orc_fp16_bits_to_f32(((const uint16_t *)w)[i])
                        : ((const float *)w)[i];
}

/* ---- elementary steps (exported so tests can pin each against its closed form) --------- */

/* y = W[row,:] . x ; one straight sum in double */
double orc_dot_row(const void *W, int dtype, size_t row, int cols, const float *x) {
    double acc = 0.0;
    size_t base = row * (size_t)cols;
    if (dtype == 1) {
        const uint16_t *w = (const uint16_t *)W + base;
#pragma omp simd reduction(+ : acc)
        for (int c = 0; c < cols; ++c) acc += (double)bf16_bits_to_f32(w[c]) * (double)x[c];
    } else if (dtype == 2) {
        const uint16_t *w = (const uint16_t *)W + base;
        const float *wide = fp16_table();
#pragma omp simd reduction(+ : acc)
        for (int c = 0; c < cols; ++c) acc += (double)wide[w[c]] * (double)x[c];
    } else {
        const float *w = (const float *)W + base;
#pragma omp simd reduction(+ : acc)
        for (int c = 0; c < cols; ++c) acc += (double)w[c] * (double)x[c];
    }
    return acc;
}

/* out[t][r] = sum_c W[r][c] x[t][c] for n activation rows; rows of W spread over threads */
void orc_matmul_rows(const void *W, int dtype, int rows, int cols, const float *x, int n, float *out) {
#pragma omp parallel for schedule(static)
    for (int r = 0; r < rows; ++r)
        for (int t = 0; t < n; ++t)
            out[(size_t)t * rows + r] = (float)orc_dot_row(W, dtype, (size_t)r, cols, x + (size_t)t * cols);
}

/* RMSNorm: out = x / sqrt(mean(x^2) + eps) * g */
void orc_rmsnorm(const float *x, const float *g, int d, float eps, float *out) {
    double ss = 0.0;
    for (int i = 0; i < d; ++i) ss += (double)x[i] * (double)x[i];
    double s = 1.0 / sqrt(ss / d + (double)eps);
    for (int i = 0; i < d; ++i) out[i] = (float)((double)x[i] * s * (double)g[i]);
}

/* Rotary embedding of one head vector, "rotate-half" pairing (i, i + hd/2),
 * angle_i = pos * theta^(-2i/hd). */
void orc_rope(float *v, int hd, int pos, float theta) {
    int half = hd / 2;
    for (int i = 0; i < half; ++i) {
        double ang = (double)pos * pow((double)theta, -2.0 * i / hd);
        double c = cos(ang), s = sin(ang);
        double a = v[i], b = v[i + half];
        v[i] = (float)(a * c - b * s);
        v[i + half] = (float)(b * c + a * s);
    }
}

double orc_silu(double x) { return x / (1.0 + exp(-x)); }

/* One attention head for one query over n cached keys/values (rows `stride` floats apart):
 * softmax(q.k_j / sqrt(hd)) weighted sum of v_j. */
void orc_attention_head(const float *q, const float *k, const float *v, int n, int hd, int stride, float *out) {
    double *s = (double *)malloc(sizeof(double) * (size_t)n);
    double m = -INFINITY, z = 0.0;
    for (int j = 0; j < n; ++j) {
        double acc = 0.0;
        for (int e = 0; e < hd; ++e) acc += (double)q[e] * (double)k[(size_t)j * stride + e];
        s[j] = acc / sqrt((double)hd);
        if (s[j] > m) m = s[j];
    }
    for (int j = 0; j < n; ++j) {
        s[j] = exp(s[j] - m);
        z += s[j];
    }
    for (int e = 0; e < hd; ++e) {
        double acc = 0.0;
        for (int j = 0; j < n; ++j) acc += s[j] * (double)v[(size_t)j * stride + e];
        out[e] = (float)(acc / z);
    }
    free(s);
}

/* Layer confidence of one logits row (Section 3.1): cast to FP32 and clamp, softmax (Eq. 1),
 * Shannon entropy with epsilon inside the log (Eq. 2), confidence = 1 - H / log(V) (Eq. 3-4).
 * Also the top-1 probability and the greedy token (lowest index among equal maxima). */
void orc_confidence(const float *logits, int V, double clamp, double eps_h, double *conf, double *pmax, int *argmax) {
    double m = -INFINITY, z = 0.0, H = 0.0;
    int am = 0;
    for (int i = 0; i < V; ++i) {
        double l = (double)logits[i];
        if (l > clamp) l = clamp;
        if (l < -clamp) l = -clamp;
        if (l > m) {
            m = l;
            am = i;
        }
    }
    for (int i = 0; i < V; ++i) {
        double l = (double)logits[i];
        if (l > clamp) l = clamp;
        if (l < -clamp) l = -clamp;
        z += exp(l - m);
    }
    double pm = 0.0;
    for (int i = 0; i < V; ++i) {
        double l = (double)logits[i];
        if (l > clamp) l = clamp;
        if (l < -clamp) l = -clamp;
        double p = exp(l - m) / z;
        H -= p * log(p + eps_h);
        if (p > pm) pm = p;
    }
    *conf = 1.0 - H / log((double)V);
    *pmax = pm;
    *argmax = am;
}

/* ---- the model ------------------------------------------------------------------------- */

static const void **dup_ptrs(const void *const *p, int n) {
    const void **q = (const void **)malloc(sizeof(void *) * (size_t)n);
    memcpy(q, p, sizeof(void *) * (size_t)n);
    return q;
}

/* Weight pointers are borrowed: the caller keeps them alive for the model's lifetime. */
orc_model *orc_create(const orc_cfg *c, const void *embed, const void *lm_head, const float *final_norm,
                      const void *const *wq, const void *const *wk, const void *const *wv, const void *const *wo,
                      const void *const *wg, const void *const *wu, const void *const *wd,
                      const float *const *norm1, const float *const *norm2) {
    orc_model *m = (orc_model *)calloc(1, sizeof(orc_model));
    m->c = *c;
    m->embed = embed;
    m->lm_head = lm_head;
    m->final_norm = final_norm;
    int L = c->n_layers;
    m->wq = dup_ptrs(wq, L);
    m->wk = dup_ptrs(wk, L);
    m->wv = dup_ptrs(wv, L);
    m->wo = dup_ptrs(wo, L);
    m->wg = dup_ptrs(wg, L);
    m->wu = dup_ptrs(wu, L);
    m->wd = dup_ptrs(wd, L);
    m->norm1 = (const float **)dup_ptrs((const void *const *)norm1, L);
    m->norm2 = (const float **)dup_ptrs((const void *const *)norm2, L);
    size_t kv = (size_t)L * c->max_seq * c->n_kv_heads * c->head_dim;
    m->kcache = (float *)calloc(kv, sizeof(float));
    m->vcache = (float *)calloc(kv, sizeof(float));
    return m;
}

void orc_destroy(orc_model *m) {
    if (!m) return;
    free(m->wq); free(m->wk); free(m->wv); free(m->wo); free(m->wg); free(m->wu); free(m->wd);
    free(m->norm1); free(m->norm2);
    free(m->kcache); free(m->vcache);
    free(m);
}

/* Final RMSNorm + shared LM head on n hidden rows (fp32 [n,d]) -> logits fp32 [n,V]
 * (the per-layer early-exit projection of Section 3.1, and the model's own output head). */
void orc_lm_head(const orc_model *m, const float *hidden, int n, float *logits) {
    int d = m->c.d_model, V = m->c.vocab;
    float *r = (float *)malloc(sizeof(float) * (size_t)n * d);
    for (int t = 0; t < n; ++t) orc_rmsnorm(hidden + (size_t)t * d, m->final_norm, d, m->c.rms_eps, r + (size_t)t * d);
    orc_matmul_rows(m->lm_head, m->c.weight_dtype, V, d, r, n, logits);
    free(r);
}

/*
 * Run n tokens, at cache positions pos0 .. pos0+n-1, through the layers.  skip_mask byte per layer: bit 0 skips
 * the attention half (the stream and that layer's KV entries stay untouched), bit 1 skips the FFN half; 3 skips the
 * whole layer; NULL mask = full model.  Each row attends causally to cache positions <= its own.  Row t's
 * arithmetic does not depend on n: running rows one at a time gives the same bits.
 *   logits_out [n,V] or NULL; hid_attn / hid_ffn [L,n,d] or NULL: the residual stream after
 *   each layer's attention add / FFN add, rounded to the storage type (skipped layers: zeros).
 * Returns 0, or -1 on a bad argument.
 */
int orc_forward(orc_model *m, const uint8_t *skip_mask, const int32_t *tokens, int n, int pos0,
                float *logits_out, float *hid_attn, float *hid_ffn) {
    const orc_cfg *c = &m->c;
    int d = c->d_model, H = c->n_heads, hd = c->head_dim, F = c->d_ffn, dt = c->weight_dtype;
    int Hkv = c->n_kv_heads, kvd = Hkv * hd;   /* keys and values have n_kv_heads heads: [n, kvd] */
    if (n <= 0 || pos0 < 0 || pos0 + n > c->max_seq || H * hd != d || Hkv < 1 || H % Hkv) return -1;
    int group = H / Hkv;
    for (int t = 0; t < n; ++t)
        if (tokens[t] < 0 || tokens[t] >= c->vocab) return -1;

    size_t nd = (size_t)n * d;
    float *x = (float *)malloc(sizeof(float) * nd);
    float *r = (float *)malloc(sizeof(float) * nd);
    float *q = (float *)malloc(sizeof(float) * nd);
    float *k = (float *)malloc(sizeof(float) * nd);
    float *v = (float *)malloc(sizeof(float) * nd);
    float *a = (float *)malloc(sizeof(float) * nd);
    float *o = (float *)malloc(sizeof(float) * nd);
    float *g = (float *)malloc(sizeof(float) * (size_t)n * F);
    float *u = (float *)malloc(sizeof(float) * (size_t)n * F);

    for (int t = 0; t < n; ++t)
        for (int i = 0; i < d; ++i) x[(size_t)t * d + i] = wload(m->embed, (size_t)tokens[t] * d + i, dt);

    for (int l = 0; l < c->n_layers; ++l) {
        size_t tapoff = (size_t)l * nd;
        const int skip_attn = skip_mask && (skip_mask[l] & 1), skip_ffn = skip_mask && (skip_mask[l] & 2);
        if (skip_attn && skip_ffn) {
            if (hid_attn) memset(hid_attn + tapoff, 0, sizeof(float) * nd);
            if (hid_ffn) memset(hid_ffn + tapoff, 0, sizeof(float) * nd);
            continue;
        }
        float *kc = m->kcache + (size_t)l * c->max_seq * kvd;
        float *vc = m->vcache + (size_t)l * c->max_seq * kvd;

        /* attention half */
        if (!skip_attn) {
        for (int t = 0; t < n; ++t) orc_rmsnorm(x + (size_t)t * d, m->norm1[l], d, c->rms_eps, r + (size_t)t * d);
        orc_matmul_rows(m->wq[l], dt, d, d, r, n, q);
        orc_matmul_rows(m->wk[l], dt, kvd, d, r, n, k);
        orc_matmul_rows(m->wv[l], dt, kvd, d, r, n, v);
        for (int t = 0; t < n; ++t) {
            int pos = pos0 + t;
            for (int h = 0; h < H; ++h) orc_rope(q + (size_t)t * d + h * hd, hd, pos, c->rope_theta);
            for (int h = 0; h < Hkv; ++h) orc_rope(k + (size_t)t * kvd + h * hd, hd, pos, c->rope_theta);
            for (int i = 0; i < kvd; ++i) {
                kc[(size_t)pos * kvd + i] = store_round(k[(size_t)t * kvd + i], dt);
                vc[(size_t)pos * kvd + i] = store_round(v[(size_t)t * kvd + i], dt);
            }
        }
#pragma omp parallel for collapse(2) schedule(static)
        for (int t = 0; t < n; ++t)
            for (int h = 0; h < H; ++h)
                orc_attention_head(q + (size_t)t * d + h * hd, kc + (h / group) * hd, vc + (h / group) * hd, pos0 + t + 1, hd,
                                   kvd, a + (size_t)t * d + h * hd);
        orc_matmul_rows(m->wo[l], dt, d, d, a, n, o);
        for (size_t i = 0; i < nd; ++i) x[i] += o[i];
        }
        if (hid_attn)
            for (size_t i = 0; i < nd; ++i) hid_attn[tapoff + i] = store_round(x[i], dt);

        /* FFN half */
        if (!skip_ffn) {
        for (int t = 0; t < n; ++t) orc_rmsnorm(x + (size_t)t * d, m->norm2[l], d, c->rms_eps, r + (size_t)t * d);
        orc_matmul_rows(m->wg[l], dt, F, d, r, n, g);
        orc_matmul_rows(m->wu[l], dt, F, d, r, n, u);
        for (size_t i = 0; i < (size_t)n * F; ++i) g[i] = (float)(orc_silu((double)g[i]) * (double)u[i]);
        orc_matmul_rows(m->wd[l], dt, d, F, g, n, o);
        for (size_t i = 0; i < nd; ++i) x[i] += o[i];
        }
        if (hid_ffn)
            for (size_t i = 0; i < nd; ++i) hid_ffn[tapoff + i] = store_round(x[i], dt);
    }

    if (logits_out) orc_lm_head(m, x, n, logits_out);

    free(x); free(r); free(q); free(k); free(v); free(a); free(o); free(g); free(u);
    return 0;
}

/* Read back one cached K or V row (tests of the cache contract). */
void orc_read_kv(const orc_model *m, int layer, int which, int pos, float *out) {
    const size_t kvd = (size_t)m->c.n_kv_heads * m->c.head_dim;
    const float *src = (which ? m->vcache : m->kcache) + ((size_t)layer * m->c.max_seq + pos) * kvd;
    memcpy(out, src, sizeof(float) * kvd);
}
