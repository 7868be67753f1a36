/*
 * CPU checker ("oracle") for the cloud-side non-autoregressive verification (NAV) pass.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product path may call into this file; it exists so
 * that the CUDA library can be compared, element by element, against a plain definition.  It
 * shares no code with the CUDA path.
 *
 * What NAV returns is fixed by the paper (Sec. 2.2: all draft tokens are checked by the target
 * model in ONE forward pass; drafts are accepted up to the first mismatch, which the target model
 * corrects; App. B: when every draft is accepted the target model contributes one extra token;
 * Sec. 1: the target model's output distribution is preserved exactly) together with the
 * speculative-sampling rule of the works the paper builds on (Leviathan et al. 2023; Chen et
 * al. 2023): accept draft x_i while u_i < min(1, p(x_i)/q(x_i)), otherwise draw the correction
 * from norm(max(0, p - q)); draw the extra token from p.
 *
 * Everything here is the definition written out: fp64 arithmetic throughout, sums taken in
 * ascending index order, no blocking beyond handling several token rows per weight row.  The
 * only roundings are the two storage formats of the workload: bf16 weights (inputs arrive that
 * way) and bf16 K/V rows at cache write (round to nearest even).
 *
 * Pinned (tests/test_oracle_*.py): orc_linear against a library matrix product; orc_rmsnorm,
 * orc_rope, orc_softmax, orc_attend against closed forms and invariants; orc_forward against a
 * hand-worked two-token model, chunking invariance, causality and the GQA==replicated-MHA
 * identity; orc_reject against brute-force enumeration of the output distribution, the greedy
 * longest-matching-prefix property, p == q, one-hot q and the 1 - TV(p,q) acceptance rate;
 * orc_set_kv / orc_set_len / orc_get_kv against a bit-exact round trip, a closed-form attention over
 * hand-set rows and a cache transplanted row by row into a fresh instance.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab, max_pos;
    double rms_eps, rope_base;
} orc_cfg;

typedef struct {
    const uint16_t *wq, *wk, *wv, *wo, *wg, *wu, *wd; /* bf16 bit patterns, row-major [out,in] */
    const float *attn_norm, *ffn_norm;                /* RMSNorm gains */
} orc_layer_w;

typedef struct {
    orc_cfg cfg;
    const uint16_t *tok_emb, *lm_head;
    const float *final_norm;
    orc_layer_w *layers;
    float *kc, *vc; /* [layer][pos][n_kv_heads*head_dim], values already rounded to bf16 */
    int32_t len;    /* number of cached positions */
} orc_ctx;

static inline double bf16_to_f64(uint16_t b) {
    union { float f; uint32_t u; } v;
    v.u = (uint32_t)b << 16;
    return (double)v.f;
}

/* Round a double to the nearest bf16 (via fp32, ties to even) and return it as a float. */
static inline float round_to_bf16(double x) {
    union { float f; uint32_t u; } v;
    v.f = (float)x;
    uint32_t lsb = (v.u >> 16) & 1u;
    v.u += 0x7FFFu + lsb;
    v.u &= 0xFFFF0000u;
    return v.f;
}

/* ------------------------------------------------------------------ building blocks */

/* y = x * rsqrt(mean(x^2) + eps) * g */
void orc_rmsnorm(const double *x, const float *g, int32_t d, double eps, double *y) {
    double ss = 0.0;
    for (int32_t i = 0; i < d; ++i) ss += x[i] * x[i];
    double r = 1.0 / sqrt(ss / (double)d + eps);
    for (int32_t i = 0; i < d; ++i) y[i] = x[i] * r * (double)g[i];
}

/* Rotary embedding, "rotate-half" pairing: element j is paired with j + hd/2,
 * theta_j = base^(-2j/hd), angle = pos * theta_j. In place on one head vector. */
void orc_rope(double *v, int32_t hd, int64_t pos, double base) {
    int32_t half = hd / 2;
    for (int32_t j = 0; j < half; ++j) {
        double theta = pow(base, -2.0 * (double)j / (double)hd);
        double a = (double)pos * theta;
        double c = cos(a), s = sin(a);
        double x0 = v[j], x1 = v[j + half];
        v[j] = x0 * c - x1 * s;
        v[j + half] = x1 * c + x0 * s;
    }
}

/* y[m][n] = sum_k W[n][k] * x[m][k]; W is bf16 [N][K]; k ascending; fp64. */
#define ORC_LINEAR_BODY(MB)                                                              \
    for (int32_t m0 = 0; m0 < M; m0 += (MB)) {                                           \
        int32_t mb = M - m0 < (MB) ? M - m0 : (MB);                                      \
        memset(xT, 0, sizeof(double) * (size_t)K * (MB));                                \
        for (int32_t j = 0; j < mb; ++j)                                                 \
            for (int32_t k = 0; k < K; ++k) xT[(size_t)k * (MB) + j] = x[(size_t)(m0 + j) * K + k]; \
        _Pragma("omp parallel for schedule(static)")                                     \
        for (int32_t n = 0; n < N; ++n) {                                                \
            double acc[MB];                                                              \
            for (int32_t j = 0; j < (MB); ++j) acc[j] = 0.0;                             \
            const uint16_t *w = W + (size_t)n * K;                                       \
            for (int32_t k = 0; k < K; ++k) {                                            \
                double wk = bf16_to_f64(w[k]);                                           \
                const double *xr = xT + (size_t)k * (MB);                                \
                for (int32_t j = 0; j < (MB); ++j) acc[j] += wk * xr[j];                 \
            }                                                                            \
            for (int32_t j = 0; j < mb; ++j) y[(size_t)(m0 + j) * N + n] = acc[j];       \
        }                                                                                \
    }

void orc_linear(const uint16_t *W, int32_t N, int32_t K, const double *x, int32_t M, double *y) {
    int32_t mbmax = M <= 4 ? 4 : 32;
    double *xT = (double *)malloc(sizeof(double) * (size_t)K * mbmax);
    if (M <= 4) {
        ORC_LINEAR_BODY(4)
    } else {
        ORC_LINEAR_BODY(32)
    }
    free(xT);
}

/* p = softmax(l): subtract the max, exponentiate, normalise (fp64). */
void orc_softmax(const double *l, int32_t V, double *p) {
    double m = l[0];
    for (int32_t j = 1; j < V; ++j) if (l[j] > m) m = l[j];
    double z = 0.0;
    for (int32_t j = 0; j < V; ++j) { p[j] = exp(l[j] - m); z += p[j]; }
    for (int32_t j = 0; j < V; ++j) p[j] /= z;
}

/* One query row against n_keys cached rows of one KV head:
 * out = sum_j softmax_j(q.k_j / sqrt(hd)) v_j.  kc/vc point at the head's first row,
 * consecutive rows are `stride` floats apart. */
void orc_attend(const double *q, const float *kc, const float *vc, int64_t stride,
                int32_t n_keys, int32_t hd, double *out) {
    double *s = (double *)malloc(sizeof(double) * (size_t)n_keys);
    double scale = 1.0 / sqrt((double)hd);
    double m = -INFINITY;
    for (int32_t j = 0; j < n_keys; ++j) {
        const float *kr = kc + (size_t)j * stride;
        double acc = 0.0;
        for (int32_t e = 0; e < hd; ++e) acc += q[e] * (double)kr[e];
        s[j] = acc * scale;
        if (s[j] > m) m = s[j];
    }
    double z = 0.0;
    for (int32_t j = 0; j < n_keys; ++j) { s[j] = exp(s[j] - m); z += s[j]; }
    for (int32_t e = 0; e < hd; ++e) out[e] = 0.0;
    for (int32_t j = 0; j < n_keys; ++j) {
        const float *vr = vc + (size_t)j * stride;
        double pj = s[j] / z;
        for (int32_t e = 0; e < hd; ++e) out[e] += pj * (double)vr[e];
    }
    free(s);
}

static inline double silu(double z) { return z / (1.0 + exp(-z)); }

/* ------------------------------------------------------------------ context */

orc_ctx *orc_create(const orc_cfg *cfg, const uint16_t *tok_emb, const uint16_t *lm_head,
                    const float *final_norm, const orc_layer_w *layers) {
    orc_ctx *c = (orc_ctx *)calloc(1, sizeof(orc_ctx));
    c->cfg = *cfg;
    c->tok_emb = tok_emb;
    c->lm_head = lm_head;
    c->final_norm = final_norm;
    c->layers = (orc_layer_w *)malloc(sizeof(orc_layer_w) * (size_t)cfg->n_layers);
    memcpy(c->layers, layers, sizeof(orc_layer_w) * (size_t)cfg->n_layers);
    size_t n = (size_t)cfg->n_layers * cfg->max_pos * cfg->n_kv_heads * cfg->head_dim;
    c->kc = (float *)calloc(n, sizeof(float));
    c->vc = (float *)calloc(n, sizeof(float));
    c->len = 0;
    return c;
}

void orc_destroy(orc_ctx *c) {
    if (!c) return;
    free(c->layers); free(c->kc); free(c->vc); free(c);
}

int32_t orc_len(const orc_ctx *c) { return c->len; }

/* Commit / rollback: keep the first new_len positions; rows beyond are never read again. */
int32_t orc_truncate(orc_ctx *c, int32_t new_len) {
    if (new_len < 0 || new_len > c->len) return -1;
    c->len = new_len;
    return 0;
}

static inline size_t kv_off(const orc_ctx *c, int32_t layer, int32_t pos) {
    return ((size_t)layer * c->cfg.max_pos + pos) * (size_t)(c->cfg.n_kv_heads * c->cfg.head_dim);
}

/* Write one position's K and V rows (bf16 bit patterns, [n_kv_heads*head_dim]) straight into the
 * cache: used to load a seeded synthetic prefix.  Does not change len; see orc_set_len. */
void orc_set_kv(orc_ctx *c, int32_t layer, int32_t pos0, int32_t n_pos, const uint16_t *k, const uint16_t *v) {
    int32_t w = c->cfg.n_kv_heads * c->cfg.head_dim;
    for (int32_t p = 0; p < n_pos; ++p) {
        float *kd = c->kc + kv_off(c, layer, pos0 + p), *vd = c->vc + kv_off(c, layer, pos0 + p);
        for (int32_t e = 0; e < w; ++e) {
            kd[e] = (float)bf16_to_f64(k[(size_t)p * w + e]);
            vd[e] = (float)bf16_to_f64(v[(size_t)p * w + e]);
        }
    }
}

void orc_set_len(orc_ctx *c, int32_t len) { c->len = len; }

/* Read back cached rows as floats (bf16-valued). */
void orc_get_kv(const orc_ctx *c, int32_t layer, int32_t pos, float *k, float *v) {
    int32_t w = c->cfg.n_kv_heads * c->cfg.head_dim;
    memcpy(k, c->kc + kv_off(c, layer, pos), sizeof(float) * (size_t)w);
    memcpy(v, c->vc + kv_off(c, layer, pos), sizeof(float) * (size_t)w);
}

/* ------------------------------------------------------------------ forward */

/* One forward of the target model over n tokens placed at positions len .. len+n-1 (Sec. 2.2:
 * the whole draft sequence is validated in a single pass).  Row i attends to every cached
 * position and to rows <= i of this call.  K/V of all n rows are appended (len += n); the caller
 * truncates afterwards.  Logits (fp64, [n - logits_from][vocab]) are produced for rows
 * >= logits_from; pass logits_from = n for none.  Returns 0, or -1 if the cache would overflow. */
int32_t orc_forward(orc_ctx *c, const int32_t *tokens, int32_t n, int32_t logits_from, double *logits) {
    const orc_cfg *g = &c->cfg;
    const int32_t d = g->d_model, hd = g->head_dim, Hq = g->n_q_heads, Hkv = g->n_kv_heads;
    const int32_t F = g->d_ffn, V = g->vocab, qd = Hq * hd, kvd = Hkv * hd, grp = Hq / Hkv;
    const int32_t P = c->len;
    if (P + n > g->max_pos) return -1;
    for (int32_t i = 0; i < n; ++i) if (tokens[i] < 0 || tokens[i] >= V) return -2;

    double *x = (double *)malloc(sizeof(double) * (size_t)n * d);
    double *h = (double *)malloc(sizeof(double) * (size_t)n * d);
    double *q = (double *)malloc(sizeof(double) * (size_t)n * qd);
    double *k = (double *)malloc(sizeof(double) * (size_t)n * kvd);
    double *v = (double *)malloc(sizeof(double) * (size_t)n * kvd);
    double *att = (double *)malloc(sizeof(double) * (size_t)n * qd);
    double *o = (double *)malloc(sizeof(double) * (size_t)n * d);
    double *ga = (double *)malloc(sizeof(double) * (size_t)n * F);
    double *up = (double *)malloc(sizeof(double) * (size_t)n * F);

    for (int32_t i = 0; i < n; ++i)
        for (int32_t e = 0; e < d; ++e) x[(size_t)i * d + e] = bf16_to_f64(c->tok_emb[(size_t)tokens[i] * d + e]);

    for (int32_t l = 0; l < g->n_layers; ++l) {
        const orc_layer_w *w = &c->layers[l];
        for (int32_t i = 0; i < n; ++i) orc_rmsnorm(x + (size_t)i * d, w->attn_norm, d, g->rms_eps, h + (size_t)i * d);
        orc_linear(w->wq, qd, d, h, n, q);
        orc_linear(w->wk, kvd, d, h, n, k);
        orc_linear(w->wv, kvd, d, h, n, v);
        for (int32_t i = 0; i < n; ++i) {
            for (int32_t a = 0; a < Hq; ++a) orc_rope(q + (size_t)i * qd + (size_t)a * hd, hd, P + i, g->rope_base);
            for (int32_t a = 0; a < Hkv; ++a) orc_rope(k + (size_t)i * kvd + (size_t)a * hd, hd, P + i, g->rope_base);
            float *kd = c->kc + kv_off(c, l, P + i), *vd = c->vc + kv_off(c, l, P + i);
            for (int32_t e = 0; e < kvd; ++e) {
                kd[e] = round_to_bf16(k[(size_t)i * kvd + e]);
                vd[e] = round_to_bf16(v[(size_t)i * kvd + e]);
            }
        }
#pragma omp parallel for schedule(dynamic, 1)
        for (int32_t t = 0; t < n * Hq; ++t) {
            int32_t i = t / Hq, a = t % Hq, kvh = a / grp;
            orc_attend(q + (size_t)i * qd + (size_t)a * hd, c->kc + kv_off(c, l, 0) + (size_t)kvh * hd,
                       c->vc + kv_off(c, l, 0) + (size_t)kvh * hd, kvd, P + i + 1, hd,
                       att + (size_t)i * qd + (size_t)a * hd);
        }
        orc_linear(w->wo, d, qd, att, n, o);
        for (size_t e = 0; e < (size_t)n * d; ++e) x[e] += o[e];
        for (int32_t i = 0; i < n; ++i) orc_rmsnorm(x + (size_t)i * d, w->ffn_norm, d, g->rms_eps, h + (size_t)i * d);
        orc_linear(w->wg, F, d, h, n, ga);
        orc_linear(w->wu, F, d, h, n, up);
        for (size_t e = 0; e < (size_t)n * F; ++e) ga[e] = silu(ga[e]) * up[e];
        orc_linear(w->wd, d, F, ga, n, o);
        for (size_t e = 0; e < (size_t)n * d; ++e) x[e] += o[e];
    }
    if (logits_from < n) {
        int32_t m = n - logits_from;
        for (int32_t i = 0; i < m; ++i)
            orc_rmsnorm(x + (size_t)(logits_from + i) * d, c->final_norm, d, g->rms_eps, h + (size_t)i * d);
        orc_linear(c->lm_head, V, d, h, m, logits);
    }
    c->len = P + n;
    free(x); free(h); free(q); free(k); free(v); free(att); free(o); free(ga); free(up);
    return 0;
}

/* ------------------------------------------------------------------ rejection sampling */

/* Normalised inclusive CDF, in token-id order, of the distribution the final token is drawn from:
 * q == NULL : p = softmax(l)                       (extra token, App. B)
 * q != NULL : norm(max(0, p - q)); if that is identically zero, p   (correction token)
 * cdf[t] = sum_{j<=t} r_j / S.  Returns S (the un-normalised mass). */
double orc_final_cdf(const double *l, const float *q, int32_t V, double *cdf) {
    double *p = (double *)malloc(sizeof(double) * (size_t)V);
    orc_softmax(l, V, p);
    double S = 0.0;
    if (q) {
        for (int32_t j = 0; j < V; ++j) {
            double r = p[j] - (double)q[j];
            cdf[j] = r > 0.0 ? r : 0.0;
            S += cdf[j];
        }
    }
    if (!q || S == 0.0) {
        S = 0.0;
        for (int32_t j = 0; j < V; ++j) { cdf[j] = p[j]; S += p[j]; }
    }
    double run = 0.0;
    for (int32_t j = 0; j < V; ++j) { run += cdf[j]; cdf[j] = run / S; }
    free(p);
    return S;
}

/* Inverse CDF in token-id order: the smallest t whose running mass exceeds u * S. */
static int32_t draw(const double *r, int32_t V, double u) {
    double S = 0.0;
    for (int32_t j = 0; j < V; ++j) S += r[j];
    double target = u * S, run = 0.0;
    int32_t last = 0;
    for (int32_t j = 0; j < V; ++j) {
        if (r[j] > 0.0) last = j;
        run += r[j];
        if (run > target) return j;
    }
    return last; /* only reachable through rounding at the very top of the CDF */
}

static int32_t argmax_lowest(const double *l, int32_t V) {
    int32_t b = 0;
    for (int32_t j = 1; j < V; ++j) if (l[j] > l[b]) b = j;
    return b;
}

/* The accept / correct rule over one request.
 *   logits : fp64 [k+1][V]; row i-1 is the target distribution that scores draft i (i = 1..k),
 *            row k is the distribution of the extra token.
 *   q      : fp32 [k][V] draft distributions (ignored when greedy != 0)
 *   drafts : k draft token ids;  u : k+1 uniforms in [0,1): u[0..k-1] acceptance, u[k] final draw.
 * Stochastic: accept draft i iff u_i < min(1, p_i(x_i) / q_i(x_i)); a zero q with p > 0 accepts,
 * 0/0 rejects.  On the first rejection at row r draw from norm(max(0, p_r - q_r)) (from p_r when
 * that residual is identically zero); when all k pass, draw the extra token from p_k.
 * Greedy (Sec. 2.2 prose): accept while the draft equals the row's argmax (lowest index on
 * ties); emit the argmax of the first mismatching row, or of row k.
 * margins[i] (i < k, may be NULL) = min(1, ratio_i) - u_i for every row examined (NaN beyond).
 */
void orc_reject(const double *logits, const float *q, const int32_t *drafts, const float *u,
                int32_t k, int32_t V, int32_t greedy, int32_t *n_acc_out, int32_t *token_out,
                double *margins) {
    double *p = (double *)malloc(sizeof(double) * (size_t)V);
    int32_t n_acc = 0;
    if (margins) for (int32_t i = 0; i < k; ++i) margins[i] = NAN;
    for (int32_t i = 0; i < k; ++i) {
        const double *l = logits + (size_t)i * V;
        int32_t x = drafts[i];
        int ok;
        if (greedy) {
            ok = (x == argmax_lowest(l, V));
        } else {
            orc_softmax(l, V, p);
            double px = p[x], qx = (double)q[(size_t)i * V + x];
            double ratio;
            if (qx > 0.0) ratio = px / qx;
            else ratio = px > 0.0 ? INFINITY : 0.0;
            double a = ratio < 1.0 ? ratio : 1.0;
            if (margins) margins[i] = a - (double)u[i];
            ok = ((double)u[i] < a);
        }
        if (!ok) break;
        ++n_acc;
    }
    const double *l = logits + (size_t)n_acc * V;
    int32_t tok;
    if (greedy) {
        tok = argmax_lowest(l, V);
    } else {
        orc_softmax(l, V, p);
        if (n_acc < k) {
            double S = 0.0;
            double *r = (double *)malloc(sizeof(double) * (size_t)V);
            for (int32_t j = 0; j < V; ++j) {
                double t = p[j] - (double)q[(size_t)n_acc * V + j];
                r[j] = t > 0.0 ? t : 0.0;
                S += r[j];
            }
            tok = (S > 0.0) ? draw(r, V, (double)u[k]) : draw(p, V, (double)u[k]);
            free(r);
        } else {
            tok = draw(p, V, (double)u[k]);
        }
    }
    *n_acc_out = n_acc;
    *token_out = tok;
    free(p);
}
