/*
 * CPU oracle for the KNN-SSD decode hot path.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain definition the CUDA library is checked against.
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg may build
 * or call it; the product library never links, imports or falls back to it, and
 * it shares no code, header, table or constant generator with the CUDA path.
 *
 * What it computes (paper sections in brackets):
 *   - the LLaMA-style pre-norm decoder the paper runs through a standard
 *     transformer library [App. C.1], one row (token position) at a time per
 *     sublayer, with a KV cache [App. C.1 "KV cache is used"];
 *   - the draft model M(z): the same decoder with the sublayers whose mask bit
 *     z^(j) = 1 left out [Sec. 3.1; Sec. 4.1, definition of z_i];
 *   - greedy drafting, one-pass verification by the full model and acceptance
 *     of the agreeing prefix [Sec. 4.2, drafting equation and the paragraph
 *     after it];
 *   - the domain choice: cosine arg-max over all anchors [Sec. 4.2, Eq. (4)],
 *     applied to the mean of the last-layer hidden states of the prompt.
 *
 * Precision: every tensor the method names (activations, logits, K/V, the
 * pooled vector, cosines) is an fp32 value - the precision the CUDA kernels
 * hold them in - and every reduction (dot product, sum of squares, softmax
 * denominator, mean) is accumulated in fp64 in plain index order and rounded to
 * fp32 once.  Where a bf16 model is configured, weights are bf16 bit patterns
 * widened exactly to fp32, and K and V are rounded to bf16 (nearest even) when
 * they enter the cache.  Arg-max decisions are taken on the fp32 values, lowest
 * index winning ties.
 *
 * Pins (tests/test_oracle_*.py): logits against a standard library decoder of
 * the same architecture; attention/RMSNorm/SwiGLU special cases; losslessness
 * of the speculative loop against plain greedy decoding; all-retained and
 * all-skipped masks; brute-force cosine search; the accept rule by brute force.
 * Absolute logit values beyond those identities have no external golden: the
 * decoder arithmetic is pinned to the library decoder on small shapes only.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ff, vocab, max_seq;
    float rms_eps, rope_theta;
    int dtype; /* 0: fp32 weights and cache; 1: bf16 weights and cache */
} orc_config;

typedef struct {
    const void *tok_embed;   /* [vocab][d_model] */
    const float *final_norm; /* [d_model] */
    const void *lm_head;     /* [vocab][d_model] */
    const float *const *attn_norm; /* [n_layers] -> [d_model] */
    const void *const *wq;   /* [n_heads*head_dim][d_model] */
    const void *const *wk;   /* [n_kv_heads*head_dim][d_model] */
    const void *const *wv;
    const void *const *wo;   /* [d_model][n_heads*head_dim] */
    const float *const *mlp_norm;
    const void *const *w_gate; /* [d_ff][d_model] */
    const void *const *w_up;
    const void *const *w_down; /* [d_model][d_ff] */
} orc_weights;

typedef struct {
    orc_config c;
    orc_weights w;
    float *kcache, *vcache; /* [n_layers][n_kv_heads][max_seq][head_dim] */
    int len;                /* committed context length */
} orc_model;

/* ---- scalar helpers ---------------------------------------------------- */

static float bf16_to_f32(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

static float round_to_bf16(float f) { /* nearest even, finite inputs */
    uint32_t u;
    memcpy(&u, &f, 4);
    u = (u + 0x7FFFu + ((u >> 16) & 1u)) & 0xFFFF0000u;
    memcpy(&f, &u, 4);
    return f;
}

static inline float weight_at(const void *w, int dtype, size_t i) {
    return dtype ? bf16_to_f32(((const uint16_t *)w)[i]) : ((const float *)w)[i];
}

/* y[m][o] = sum_i W[o][i] * x[m][i]   (row-major W [n_out][n_in]) */
static void linear(const void *W, int dtype, int n_out, int n_in, const float *x, int M, float *y) {
#pragma omp parallel for schedule(static)
    for (int o = 0; o < n_out; ++o) {
        double acc[64];
        for (int m = 0; m < M; ++m) acc[m] = 0.0;
        const size_t base = (size_t)o * (size_t)n_in;
        for (int i = 0; i < n_in; ++i) {
            const double w = (double)weight_at(W, dtype, base + (size_t)i);
            for (int m = 0; m < M; ++m) acc[m] += w * (double)x[(size_t)m * n_in + i];
        }
        for (int m = 0; m < M; ++m) y[(size_t)m * n_out + o] = (float)acc[m];
    }
}

/* The linear map on its own, for per-kernel checks: y [M][n_out] = x [M][n_in] . W^T. */
void orc_linear(const void *W, int dtype, int n_out, int n_in, const float *x, int M, float *y) {
    linear(W, dtype, n_out, n_in, x, M, y);
}

/* RMSNorm: h = x * rsqrt(mean(x^2) + eps) * g */
static void rmsnorm(const float *x, const float *g, int d, float eps, float *h) {
    double ss = 0.0;
    for (int i = 0; i < d; ++i) ss += (double)x[i] * (double)x[i];
    const double r = 1.0 / sqrt(ss / (double)d + (double)eps);
    for (int i = 0; i < d; ++i) h[i] = (float)((double)x[i] * r * (double)g[i]);
}

/* Rotary embedding of one head vector at an absolute position; dimension i is
 * paired with i + hd/2 and the pair is turned by pos * theta^(-2i/hd). */
static void rope(float *v, int hd, int pos, float theta) {
    const int half = hd / 2;
    for (int i = 0; i < half; ++i) {
        const double inv_freq = pow((double)theta, -2.0 * (double)i / (double)hd);
        const double ang = (double)pos * inv_freq;
        const float c = (float)cos(ang), s = (float)sin(ang);
        const double a = v[i], b = v[i + half];
        v[i] = (float)(a * (double)c - b * (double)s);
        v[i + half] = (float)(b * (double)c + a * (double)s);
    }
}

static int argmax_f32(const float *p, int n, float *margin) {
    int best = 0;
    for (int i = 1; i < n; ++i)
        if (p[i] > p[best]) best = i;
    if (margin) {
        float second = -INFINITY;
        for (int i = 0; i < n; ++i)
            if (i != best && p[i] > second) second = p[i];
        *margin = p[best] - second;
    }
    return best;
}

/* ---- model ------------------------------------------------------------- */

orc_model *orc_create(const orc_config *c, const orc_weights *w) {
    orc_model *m = (orc_model *)calloc(1, sizeof(orc_model));
    if (!m) return NULL;
    m->c = *c;
    m->w = *w;
    const size_t n = (size_t)c->n_layers * c->n_kv_heads * (size_t)c->max_seq * c->head_dim;
    m->kcache = (float *)calloc(n, sizeof(float));
    m->vcache = (float *)calloc(n, sizeof(float));
    if (!m->kcache || !m->vcache) {
        free(m->kcache);
        free(m->vcache);
        free(m);
        return NULL;
    }
    return m;
}

void orc_destroy(orc_model *m) {
    if (!m) return;
    free(m->kcache);
    free(m->vcache);
    free(m);
}

int orc_len(const orc_model *m) { return m->len; }
void orc_set_len(orc_model *m, int len) { m->len = len; }

static size_t cache_index(const orc_config *c, int layer, int kvh, int pos) {
    return (((size_t)layer * c->n_kv_heads + kvh) * (size_t)c->max_seq + (size_t)pos) * c->head_dim;
}

/* Attention sublayer on M rows at positions pos0..pos0+M-1 (causal):
 * x += W_o * concat_heads( softmax(q K^T / sqrt(hd)) V ). */
static void attention_sublayer(orc_model *m, int layer, float *x, int M, int pos0) {
    const orc_config *c = &m->c;
    const int d = c->d_model, H = c->n_heads, Hkv = c->n_kv_heads, hd = c->head_dim;
    const int nq = H * hd, nkv = Hkv * hd, group = H / Hkv;
    float *h = (float *)malloc(sizeof(float) * (size_t)M * d);
    float *q = (float *)malloc(sizeof(float) * (size_t)M * nq);
    float *k = (float *)malloc(sizeof(float) * (size_t)M * nkv);
    float *v = (float *)malloc(sizeof(float) * (size_t)M * nkv);
    float *o = (float *)malloc(sizeof(float) * (size_t)M * nq);
    float *y = (float *)malloc(sizeof(float) * (size_t)M * d);
    for (int r = 0; r < M; ++r) rmsnorm(x + (size_t)r * d, m->w.attn_norm[layer], d, c->rms_eps, h + (size_t)r * d);
    linear(m->w.wq[layer], c->dtype, nq, d, h, M, q);
    linear(m->w.wk[layer], c->dtype, nkv, d, h, M, k);
    linear(m->w.wv[layer], c->dtype, nkv, d, h, M, v);
    for (int r = 0; r < M; ++r) {
        const int pos = pos0 + r;
        for (int j = 0; j < H; ++j) rope(q + (size_t)r * nq + (size_t)j * hd, hd, pos, c->rope_theta);
        for (int j = 0; j < Hkv; ++j) {
            float *kr = k + (size_t)r * nkv + (size_t)j * hd;
            const float *vr = v + (size_t)r * nkv + (size_t)j * hd;
            rope(kr, hd, pos, c->rope_theta);
            float *kc = m->kcache + cache_index(c, layer, j, pos);
            float *vc = m->vcache + cache_index(c, layer, j, pos);
            for (int e = 0; e < hd; ++e) {
                kc[e] = c->dtype ? round_to_bf16(kr[e]) : kr[e];
                vc[e] = c->dtype ? round_to_bf16(vr[e]) : vr[e];
            }
        }
    }
    const double scale = 1.0 / sqrt((double)hd);
#pragma omp parallel for collapse(2) schedule(static)
    for (int r = 0; r < M; ++r) {
        for (int j = 0; j < H; ++j) {
            const int pos = pos0 + r, kvh = j / group, T = pos + 1;
            const float *qv = q + (size_t)r * nq + (size_t)j * hd;
            float *s = (float *)malloc(sizeof(float) * (size_t)T);
            float smax = -INFINITY;
            for (int t = 0; t < T; ++t) {
                const float *kc = m->kcache + cache_index(c, layer, kvh, t);
                double acc = 0.0;
                for (int e = 0; e < hd; ++e) acc += (double)qv[e] * (double)kc[e];
                s[t] = (float)(acc * scale);
                if (s[t] > smax) smax = s[t];
            }
            double *p = (double *)malloc(sizeof(double) * (size_t)T);
            double denom = 0.0;
            for (int t = 0; t < T; ++t) {
                p[t] = exp((double)s[t] - (double)smax);
                denom += p[t];
            }
            float *ov = o + (size_t)r * nq + (size_t)j * hd;
            for (int e = 0; e < hd; ++e) {
                double acc = 0.0;
                for (int t = 0; t < T; ++t) {
                    const float *vc = m->vcache + cache_index(c, layer, kvh, t);
                    acc += p[t] * (double)vc[e];
                }
                ov[e] = (float)(acc / denom);
            }
            free(p);
            free(s);
        }
    }
    linear(m->w.wo[layer], c->dtype, d, nq, o, M, y);
    for (size_t i = 0; i < (size_t)M * d; ++i) x[i] = x[i] + y[i];
    free(h); free(q); free(k); free(v); free(o); free(y);
}

/* MLP sublayer: x += W_down ( silu(W_gate h) * (W_up h) ),  h = RMSNorm(x). */
static void mlp_sublayer(orc_model *m, int layer, float *x, int M) {
    const orc_config *c = &m->c;
    const int d = c->d_model, F = c->d_ff;
    float *h = (float *)malloc(sizeof(float) * (size_t)M * d);
    float *g = (float *)malloc(sizeof(float) * (size_t)M * F);
    float *u = (float *)malloc(sizeof(float) * (size_t)M * F);
    float *y = (float *)malloc(sizeof(float) * (size_t)M * d);
    for (int r = 0; r < M; ++r) rmsnorm(x + (size_t)r * d, m->w.mlp_norm[layer], d, c->rms_eps, h + (size_t)r * d);
    linear(m->w.w_gate[layer], c->dtype, F, d, h, M, g);
    linear(m->w.w_up[layer], c->dtype, F, d, h, M, u);
    for (size_t i = 0; i < (size_t)M * F; ++i) {
        const double gv = g[i];
        g[i] = (float)(gv / (1.0 + exp(-gv)) * (double)u[i]);
    }
    linear(m->w.w_down[layer], c->dtype, d, F, g, M, y);
    for (size_t i = 0; i < (size_t)M * d; ++i) x[i] = x[i] + y[i];
    free(h); free(g); free(u); free(y);
}

/*
 * One decoder pass over M rows (tokens at positions pos0 .. pos0+M-1, attending
 * to everything in the cache before them and causally to one another).
 *   skip_mask: NULL = full model; else [2*n_layers] bytes, entry 2l = attention
 *              sublayer of layer l, 2l+1 = its MLP sublayer, 1 = skipped.
 *   logits:    NULL or [M][vocab];  hidden: NULL or [M][d_model], the state
 *              after the final RMSNorm;  argmax / margin: NULL or [M]
 *              (margin = top-1 minus top-2 logit).
 *   head_rows: rows >= M - head_rows get logits/argmax (others left untouched);
 *              pass M for all rows.
 * A skipped attention sublayer writes no K/V for these positions.
 * Returns 0, or -1 on a bad argument.  Does not change the committed length.
 */
int orc_forward(orc_model *m, const int *tokens, int M, int pos0, const unsigned char *skip_mask,
                float *logits, float *hidden, int *argmax, float *margin, int head_rows) {
    const orc_config *c = &m->c;
    const int d = c->d_model, V = c->vocab;
    if (M < 1 || M > 64 || pos0 < 0 || pos0 + M > c->max_seq) return -1;
    for (int r = 0; r < M; ++r)
        if (tokens[r] < 0 || tokens[r] >= V) return -1;
    float *x = (float *)malloc(sizeof(float) * (size_t)M * d);
    for (int r = 0; r < M; ++r)
        for (int i = 0; i < d; ++i) x[(size_t)r * d + i] = weight_at(m->w.tok_embed, c->dtype, (size_t)tokens[r] * d + i);
    for (int l = 0; l < c->n_layers; ++l) {
        if (!skip_mask || !skip_mask[2 * l]) attention_sublayer(m, l, x, M, pos0);
        if (!skip_mask || !skip_mask[2 * l + 1]) mlp_sublayer(m, l, x, M);
    }
    float *h = (float *)malloc(sizeof(float) * (size_t)M * d);
    for (int r = 0; r < M; ++r) rmsnorm(x + (size_t)r * d, m->w.final_norm, d, c->rms_eps, h + (size_t)r * d);
    if (hidden) memcpy(hidden, h, sizeof(float) * (size_t)M * d);
    if (head_rows > M) head_rows = M;
    if (head_rows > 0 && (logits || argmax || margin)) {
        const int r0 = M - head_rows;
        float *lg = (float *)malloc(sizeof(float) * (size_t)head_rows * V);
        linear(m->w.lm_head, c->dtype, V, d, h + (size_t)r0 * d, head_rows, lg);
        for (int r = 0; r < head_rows; ++r) {
            float mg;
            const int a = argmax_f32(lg + (size_t)r * V, V, &mg);
            if (argmax) argmax[r0 + r] = a;
            if (margin) margin[r0 + r] = mg;
        }
        if (logits) memcpy(logits + (size_t)r0 * V, lg, sizeof(float) * (size_t)head_rows * V);
        free(lg);
    }
    free(x);
    free(h);
    return 0;
}

/* ---- selection [Sec. 4.2, Eq. (4)] ------------------------------------- */

/* v = (1/T) sum_t h_t */
void orc_pool_mean(const float *hidden, int T, int d, float *v) {
    for (int i = 0; i < d; ++i) {
        double acc = 0.0;
        for (int t = 0; t < T; ++t) acc += (double)hidden[(size_t)t * d + i];
        v[i] = (float)(acc / (double)T);
    }
}

/* (i*, j*) = argmax_{i,j} v.a_ij / (|v| |a_ij|); lowest flat index on ties.
 * Returns 0, or 1 if v or an anchor has zero or non-finite norm. */
int orc_knn_select(const float *v, const float *anchors, int n_domains, int per_domain, int d,
                   int *domain, int *anchor, float *cosine) {
    double vv = 0.0;
    for (int i = 0; i < d; ++i) vv += (double)v[i] * (double)v[i];
    if (!(vv > 0.0) || !isfinite(vv)) return 1;
    int best = -1;
    float best_cos = -INFINITY;
    for (int a = 0; a < n_domains * per_domain; ++a) {
        const float *av = anchors + (size_t)a * d;
        double dot = 0.0, aa = 0.0;
        for (int i = 0; i < d; ++i) {
            dot += (double)v[i] * (double)av[i];
            aa += (double)av[i] * (double)av[i];
        }
        if (!(aa > 0.0) || !isfinite(aa)) return 1;
        const float cs = (float)(dot / (sqrt(vv) * sqrt(aa)));
        if (cs > best_cos) {
            best_cos = cs;
            best = a;
        }
    }
    *domain = best / per_domain;
    *anchor = best % per_domain;
    *cosine = best_cos;
    return 0;
}

/* ---- acceptance [Sec. 4.2, verification paragraph] ---------------------- */

/* draft[0..k-1] are the drafted tokens, target[0..k] the full model's greedy
 * token after [pending], [pending, d_0], ...  The accepted count a is the
 * length of the longest prefix with target[i] == draft[i]; the token emitted
 * after the accepted ones is target[a]. */
void orc_accept(const int *draft, const int *target, int k, int *n_accepted, int *next_token) {
    int a = 0;
    while (a < k && target[a] == draft[a]) ++a;
    *n_accepted = a;
    *next_token = target[a];
}

/* ---- whole-request drivers --------------------------------------------- */

/* Full model over the prompt (rows in chunks; the numbers do not depend on the
 * chunking).  pooled: NULL or [d_model] mean of the final-norm hidden states;
 * first_token: greedy token after the prompt; first_margin: its logit margin.
 * Sets the committed length to T. */
int orc_prefill(orc_model *m, const int *prompt, int T, float *pooled, int *first_token, float *first_margin) {
    const int d = m->c.d_model, CH = 16;
    if (T < 1 || T > m->c.max_seq) return -1;
    float *hid = (float *)malloc(sizeof(float) * (size_t)T * d);
    int am[64];
    float mg[64];
    for (int t0 = 0; t0 < T; t0 += CH) {
        const int M = (T - t0 < CH) ? T - t0 : CH;
        const int last = (t0 + M == T);
        if (orc_forward(m, prompt + t0, M, t0, NULL, NULL, hid + (size_t)t0 * d, am, mg, last ? 1 : 0)) {
            free(hid);
            return -1;
        }
        if (last) {
            if (first_token) *first_token = am[M - 1];
            if (first_margin) *first_margin = mg[M - 1];
        }
    }
    if (pooled) orc_pool_mean(hid, T, d, pooled);
    free(hid);
    m->len = T;
    return 0;
}

typedef struct {
    int rounds, drafted, accepted, tokens;
    float min_margin; /* smallest top-1/top-2 logit gap among the full-model decisions that produced output */
} orc_stats;

/*
 * Greedy self-speculative generation of exactly max_new tokens after the prompt.
 * Each round drafts k_eff = min(k, remaining - 1) tokens with M(z), verifies
 * [pending, d_0 .. d_{k_eff-1}] with the full model in one pass, keeps the
 * agreeing prefix and the full model's own next token, and truncates the cache
 * to the kept rows.  accept_log / draft_log (optional) receive per round the
 * accepted count and the drafted tokens (k entries per round, -1 padded).
 * The model must have been prefilled; first_token is the prefill's token.
 */
int orc_generate(orc_model *m, int first_token, int max_new, int k, const unsigned char *skip_mask,
                 int *out_tokens, orc_stats *st, int *accept_log, int *draft_log, int log_cap) {
    if (max_new < 1 || k < 0 || k > 32) return -1;
    int produced = 0, pending = first_token, n = m->len;
    orc_stats s = {0, 0, 0, 0, INFINITY};
    out_tokens[produced++] = pending;
    while (produced < max_new) {
        const int remaining = max_new - produced;
        const int keff = (k < remaining - 1) ? k : remaining - 1;
        if (n + keff + 1 > m->c.max_seq) return -2;
        int rows[33], target[33], draft[32];
        float mg[33];
        int cur = pending;
        for (int j = 0; j < keff; ++j) {
            int am;
            if (orc_forward(m, &cur, 1, n + j, skip_mask, NULL, NULL, &am, NULL, 1)) return -1;
            draft[j] = am;
            cur = am;
        }
        rows[0] = pending;
        for (int j = 0; j < keff; ++j) rows[j + 1] = draft[j];
        if (orc_forward(m, rows, keff + 1, n, NULL, NULL, NULL, target, mg, keff + 1)) return -1;
        int a, next;
        orc_accept(draft, target, keff, &a, &next);
        for (int j = 0; j <= a; ++j)
            if (mg[j] < s.min_margin) s.min_margin = mg[j];
        for (int j = 0; j < a; ++j) out_tokens[produced++] = draft[j];
        out_tokens[produced++] = next;
        if (s.rounds < log_cap) {
            if (accept_log) accept_log[s.rounds] = a;
            if (draft_log)
                for (int j = 0; j < k; ++j) draft_log[(size_t)s.rounds * k + j] = (j < keff) ? draft[j] : -1;
        }
        pending = next;
        n += a + 1;
        m->len = n;
        s.rounds += 1;
        s.drafted += keff;
        s.accepted += a;
    }
    s.tokens = produced;
    if (st) *st = s;
    return 0;
}

/* Plain greedy decoding with the full model, one token per pass. */
int orc_greedy_full(orc_model *m, int first_token, int max_new, int *out_tokens, float *min_margin) {
    int produced = 0, cur = first_token, n = m->len;
    float mm = INFINITY;
    out_tokens[produced++] = cur;
    while (produced < max_new) {
        int am;
        float mg;
        if (n + 1 > m->c.max_seq) return -2;
        if (orc_forward(m, &cur, 1, n, NULL, NULL, NULL, &am, &mg, 1)) return -1;
        if (mg < mm) mm = mg;
        out_tokens[produced++] = am;
        cur = am;
        n += 1;
        m->len = n;
    }
    if (min_margin) *min_margin = mm;
    return 0;
}
