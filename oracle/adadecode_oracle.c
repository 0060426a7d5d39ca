/*
 * CPU oracle for the layer-parallel decode step of AdaDecode.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, double-precision implementation of
 *   (1) a Llama-style decoder (the model family the paper evaluates, Section 3): token
 *       embedding, L x [RMSNorm, rotary attention with grouped KV heads, SwiGLU FFN], final
 *       RMSNorm, LM head E*;
 *   (2) standard greedy autoregressive decoding (the result the method must reproduce,
 *       Section 2.2 "output parity", Table 2 "Vanilla Decoding");
 *   (3) Algorithm 1 (adaptive layer parallelism) with the early-prediction rule of Eq. 1, the
 *       lightweight head E^(i) = E* T^(i) of Section 2.1, and the verification rule of Eq. 2 in
 *       its greedy (temperature 0, Appendix D) form, including KV-cache rollback;
 *   (4) the same algorithm with sampled tokens: Eq. 1 with a draw from the head's distribution and Eq. 2 with
 *       its acceptance probability and the resampling from Normalize(max(0, p* - q)) (orc_sampling_decode,
 *       at the end of the file; every random number is an input).
 *
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call this file.  It
 * shares no code with the CUDA library and never calls it.  All floating point is IEEE double;
 * weights are widened exactly from their storage type (fp32 or bf16).  Dot products are plain
 * k-ordered sums in double (an `omp simd reduction` lets the compiler reassociate them, which
 * moves results by ~1e-16 relative, far below any tolerance used against it).  OpenMP spreads
 * the output rows of a mat-vec over the host cores; nothing else is blocked, fused or reordered.
 *
 * Pins (tests that do not run the CUDA path): an independent NumPy restatement of the decoder,
 * closed forms (zero weights, identity head), incremental == from-scratch recompute, brute force
 * over every exit-decision tape (output equals plain greedy), the gamma = 0 / gamma = 1 end
 * points of Section 4.4, the worked schedule of Figure 2, the cap of Appendix D; for the sampled form the
 * closed-form law of a verified token (chi-square over seeded runs, with planted wrong rules rejected),
 * gamma = 0 = plain sampling, vanishing temperature = greedy, no exit layers = numpy's inverse CDF.
 * Parity unpinned: the exit and rejection RATES on random weights (they are properties of the
 * synthetic model, not values the paper fixes); they are reported, never asserted.
 */
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#define ORC_MAX_INFLIGHT 64 /* in-flight early tokens the session can hold (cap is max_early) */

typedef struct {
    int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ff, vocab;
    int32_t wdtype; /* storage of every tensor: 0 = fp32, 1 = bf16 */
    int32_t kv_bf16; /* 1: the KV cache holds bf16: K (after rotation) and V are rounded once, to
                        nearest-even, when they are written; everything else stays double */
    double rope_base, rms_eps;
} orc_config;

typedef struct {
    const void *attn_norm, *wq, *wk, *wv, *wo, *ffn_norm, *w_gate, *w_up, *w_down;
} orc_layer;

typedef struct {
    orc_config c;
    const void *tok_embed, *lm_head, *final_norm;
    orc_layer *layers;
    /* intermediate heads, indexed by 1-based layer; head_T NULL = identity */
    int32_t *has_head;
    const void **head_T;
    double *head_scale;
} orc_model;

typedef struct {
    int64_t steps;            /* iterations of the while loop of Algorithm 1 */
    int64_t head_evals;       /* intermediate-head evaluations */
    int64_t early_exits;      /* steps that ended by Eq. 1 */
    int64_t verify_steps;     /* steps that reached layer L */
    int64_t accepted;         /* early predictions verified equal to the full-depth argmax */
    int64_t rejected;         /* first mismatching early prediction of a verification */
    int64_t discarded;        /* early predictions behind a rejection (never examined) */
    int64_t row_layers;       /* sum over processed layers of the rows processed there */
    int64_t truncated;        /* verified tokens dropped to end the call on the requested count */
    int64_t exits_at_layer[256];
} orc_stats;

typedef struct {
    const orc_model *m;
    int32_t max_seq;
    int32_t *tokens;  /* sequence y, prompt included, tentative tail included */
    int32_t len;      /* tokens in the sequence (the last one is the newest, not yet processed) */
    int32_t n_prompt;
    int32_t n_reported; /* generated tokens already returned by decode calls */
    int32_t *kv_len;  /* per layer: positions whose K/V are valid (fill level) */
    double *kcache, *vcache; /* [L][max_seq][n_kv*hd] */
    /* in-flight early tokens: hidden state at the layer where they exited */
    int32_t n_inflight;
    int32_t inflight_pos[ORC_MAX_INFLIGHT];
    int32_t inflight_depth[ORC_MAX_INFLIGHT];
    double *inflight_h; /* [ORC_MAX_INFLIGHT + 1][d] */
    /* optional recordings */
    double *logit_sink;   /* if set: final-layer logits of each verified token, [cap][V] */
    int32_t logit_cap, logit_n;
    int32_t *trace;       /* if set: (step, layer, first_pos, n_rows) per processed layer */
    int32_t trace_cap, trace_n;
    double *head_sink;    /* if set: (step, layer, token, p) per head evaluation, as doubles */
    int32_t head_cap, head_n;
} orc_session;

/* ---------------------------------------------------------------- helpers */

static inline double widen(const void *w, int dt, size_t i) {
    if (dt == 0) return (double)((const float *)w)[i];
    uint32_t b = ((uint32_t)((const uint16_t *)w)[i]) << 16;
    float f;
    memcpy(&f, &b, 4);
    return (double)f;
}

/* Y[m][j] = sum_k W[j][k] * X[m][k];  W is [N][K] row-major in storage type dt. */
static void matmul(const void *W, int dt, int N, int K, const double *X, int n_rows, double *Y) {
#pragma omp parallel for schedule(static)
    for (int j = 0; j < N; ++j) {
        for (int m = 0; m < n_rows; ++m) {
            const double *x = X + (size_t)m * K;
            double acc = 0.0;
            if (dt == 0) {
                const float *w = (const float *)W + (size_t)j * K;
#pragma omp simd reduction(+ : acc)
                for (int k = 0; k < K; ++k) acc += (double)w[k] * x[k];
            } else {
                const uint16_t *w = (const uint16_t *)W + (size_t)j * K;
#pragma omp simd reduction(+ : acc)
                for (int k = 0; k < K; ++k) {
                    union { uint32_t u; float f; } cv;
                    cv.u = ((uint32_t)w[k]) << 16;
                    acc += (double)cv.f * x[k];
                }
            }
            Y[(size_t)m * N + j] = acc;
        }
    }
}

/* RMSNorm: out = x / sqrt(mean(x^2) + eps) * g */
static void rmsnorm(const double *x, const void *g, int dt, int d, double eps, double *out) {
    double ss = 0.0;
    for (int i = 0; i < d; ++i) ss += x[i] * x[i];
    double r = 1.0 / sqrt(ss / d + eps);
    for (int i = 0; i < d; ++i) out[i] = x[i] * r * widen(g, dt, i);
}

/* Rotary embedding, rotate-half pairing (i, i + hd/2), angle = pos * base^(-2i/hd). */
static void rope(double *v, int hd, int pos, double base) {
    int half = hd / 2;
    for (int i = 0; i < half; ++i) {
        double freq = pow(base, -2.0 * i / hd);
        double a = pos * freq, c = cos(a), s = sin(a);
        double x0 = v[i], x1 = v[i + half];
        v[i] = x0 * c - x1 * s;
        v[i + half] = x1 * c + x0 * s;
    }
}

static double silu(double x) { return x / (1.0 + exp(-x)); }

/* Round a double to the nearest bf16 (ties to even), returned as a double.  The double is first
   rounded to fp32 (the type the cache writer holds it in), then the low 16 bits are rounded away. */
static double round_bf16(double x) {
    float f = (float)x;
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7f800000u) != 0x7f800000u) u += 0x7fffu + ((u >> 16) & 1u);
    u &= 0xffff0000u;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* ---------------------------------------------------------------- model */

orc_model *orc_model_create(const orc_config *c, const void *tok_embed, const void *lm_head,
                            const void *final_norm, const orc_layer *layers) {
    orc_model *m = (orc_model *)calloc(1, sizeof(orc_model));
    m->c = *c;
    m->tok_embed = tok_embed;
    m->lm_head = lm_head ? lm_head : tok_embed; /* tied head aliases the embedding */
    m->final_norm = final_norm;
    m->layers = (orc_layer *)malloc(sizeof(orc_layer) * c->n_layers);
    memcpy(m->layers, layers, sizeof(orc_layer) * c->n_layers);
    m->has_head = (int32_t *)calloc(c->n_layers + 1, sizeof(int32_t));
    m->head_T = (const void **)calloc(c->n_layers + 1, sizeof(void *));
    m->head_scale = (double *)calloc(c->n_layers + 1, sizeof(double));
    return m;
}

/* Register the intermediate head of Section 2.1 at 1-based layer `layer` (< L):
   E^(i) = E* T^(i), logits scaled by `scale`; T NULL means T = I. */
int orc_model_set_head(orc_model *m, int layer, const void *T, double scale) {
    if (layer < 1 || layer >= m->c.n_layers) return -1;
    m->has_head[layer] = 1;
    m->head_T[layer] = T;
    m->head_scale[layer] = scale;
    return 0;
}

void orc_model_destroy(orc_model *m) {
    if (!m) return;
    free(m->layers); free(m->has_head); free((void *)m->head_T); free(m->head_scale); free(m);
}

/* ---------------------------------------------------------------- session */

orc_session *orc_session_create(const orc_model *m, int max_seq) {
    const orc_config *c = &m->c;
    orc_session *s = (orc_session *)calloc(1, sizeof(orc_session));
    size_t kvd = (size_t)c->n_kv_heads * c->head_dim;
    s->m = m;
    s->max_seq = max_seq;
    s->tokens = (int32_t *)calloc(max_seq, sizeof(int32_t));
    s->kv_len = (int32_t *)calloc(c->n_layers, sizeof(int32_t));
    s->kcache = (double *)malloc(sizeof(double) * c->n_layers * max_seq * kvd);
    s->vcache = (double *)malloc(sizeof(double) * c->n_layers * max_seq * kvd);
    s->inflight_h = (double *)malloc(sizeof(double) * (ORC_MAX_INFLIGHT + 1) * c->d_model);
    if (!s->tokens || !s->kcache || !s->vcache || !s->inflight_h) return NULL;
    return s;
}

void orc_session_destroy(orc_session *s) {
    if (!s) return;
    free(s->tokens); free(s->kv_len); free(s->kcache); free(s->vcache); free(s->inflight_h); free(s);
}

void orc_session_record_logits(orc_session *s, double *sink, int cap) { s->logit_sink = sink; s->logit_cap = cap; s->logit_n = 0; }
void orc_session_record_trace(orc_session *s, int32_t *trace, int cap) { s->trace = trace; s->trace_cap = cap; s->trace_n = 0; }
void orc_session_record_heads(orc_session *s, double *sink, int cap) { s->head_sink = sink; s->head_cap = cap; s->head_n = 0; }
int orc_session_logits_recorded(const orc_session *s) { return s->logit_n; }
int orc_session_trace_recorded(const orc_session *s) { return s->trace_n; }
int orc_session_heads_recorded(const orc_session *s) { return s->head_n; }
int orc_session_len(const orc_session *s) { return s->len; }
int orc_session_kv_len(const orc_session *s, int layer0) { return s->kv_len[layer0]; }
const int32_t *orc_session_tokens(const orc_session *s) { return s->tokens; }
/* K (which = 0) or V (which = 1) of one cached position, for tests of rollback. */
const double *orc_session_kv(const orc_session *s, int which, int layer0, int pos) {
    size_t kvd = (size_t)s->m->c.n_kv_heads * s->m->c.head_dim;
    const double *base = which ? s->vcache : s->kcache;
    return base + ((size_t)layer0 * s->max_seq + pos) * kvd;
}

/* One decoder layer (0-based l) over n_rows tokens at consecutive positions pos0.. ; H holds
   their hidden states [n_rows][d] and is updated in place.  This is "process all tokens in
   P[l] in parallel" of Algorithm 1: K/V of every row are written first, then each row attends
   to cache positions 0..its own, which makes attention causal among the rows. */
static int layer_forward(orc_session *s, int l, int pos0, int n_rows, double *H) {
    const orc_config *c = &s->m->c;
    const orc_layer *w = &s->m->layers[l];
    const int d = c->d_model, hd = c->head_dim, nq = c->n_q_heads, nkv = c->n_kv_heads;
    const int qd = nq * hd, kvd = nkv * hd, group = nq / nkv, dt = c->wdtype;
    if (pos0 != s->kv_len[l]) return -10;          /* rows must extend the cache contiguously */
    if (pos0 + n_rows > s->max_seq) return -11;

    double *xn = (double *)malloc(sizeof(double) * n_rows * d);
    double *q = (double *)malloc(sizeof(double) * n_rows * qd);
    double *k = (double *)malloc(sizeof(double) * n_rows * kvd);
    double *v = (double *)malloc(sizeof(double) * n_rows * kvd);
    double *att = (double *)malloc(sizeof(double) * n_rows * qd);
    double *o = (double *)malloc(sizeof(double) * n_rows * d);
    double *g = (double *)malloc(sizeof(double) * n_rows * c->d_ff);
    double *u = (double *)malloc(sizeof(double) * n_rows * c->d_ff);

    for (int r = 0; r < n_rows; ++r) rmsnorm(H + (size_t)r * d, w->attn_norm, dt, d, c->rms_eps, xn + (size_t)r * d);
    matmul(w->wq, dt, qd, d, xn, n_rows, q);
    matmul(w->wk, dt, kvd, d, xn, n_rows, k);
    matmul(w->wv, dt, kvd, d, xn, n_rows, v);
    double *kc = s->kcache + (size_t)l * s->max_seq * kvd, *vc = s->vcache + (size_t)l * s->max_seq * kvd;
    for (int r = 0; r < n_rows; ++r) {
        int pos = pos0 + r;
        for (int h = 0; h < nq; ++h) rope(q + (size_t)r * qd + h * hd, hd, pos, c->rope_base);
        for (int h = 0; h < nkv; ++h) rope(k + (size_t)r * kvd + h * hd, hd, pos, c->rope_base);
        if (c->kv_bf16) {
            for (int i = 0; i < kvd; ++i) { k[(size_t)r * kvd + i] = round_bf16(k[(size_t)r * kvd + i]); v[(size_t)r * kvd + i] = round_bf16(v[(size_t)r * kvd + i]); }
        }
        memcpy(kc + (size_t)pos * kvd, k + (size_t)r * kvd, sizeof(double) * kvd);
        memcpy(vc + (size_t)pos * kvd, v + (size_t)r * kvd, sizeof(double) * kvd);
    }
    s->kv_len[l] = pos0 + n_rows;

    const double scale = 1.0 / sqrt((double)hd);
#pragma omp parallel for schedule(static) collapse(2)
    for (int r = 0; r < n_rows; ++r) {
        for (int h = 0; h < nq; ++h) {
            int pos = pos0 + r, kvh = h / group;
            const double *qv = q + (size_t)r * qd + h * hd;
            double *sc = (double *)malloc(sizeof(double) * (pos + 1));
            double mx = -INFINITY;
            for (int t = 0; t <= pos; ++t) {
                const double *kt = kc + (size_t)t * kvd + kvh * hd;
                double a = 0.0;
                for (int i = 0; i < hd; ++i) a += qv[i] * kt[i];
                sc[t] = a * scale;
                if (sc[t] > mx) mx = sc[t];
            }
            double den = 0.0;
            for (int t = 0; t <= pos; ++t) { sc[t] = exp(sc[t] - mx); den += sc[t]; }
            double *out = att + (size_t)r * qd + h * hd;
            for (int i = 0; i < hd; ++i) out[i] = 0.0;
            for (int t = 0; t <= pos; ++t) {
                const double *vt = vc + (size_t)t * kvd + kvh * hd;
                double p = sc[t] / den;
                for (int i = 0; i < hd; ++i) out[i] += p * vt[i];
            }
            free(sc);
        }
    }
    matmul(w->wo, dt, d, qd, att, n_rows, o);
    for (size_t i = 0; i < (size_t)n_rows * d; ++i) H[i] += o[i];

    for (int r = 0; r < n_rows; ++r) rmsnorm(H + (size_t)r * d, w->ffn_norm, dt, d, c->rms_eps, xn + (size_t)r * d);
    matmul(w->w_gate, dt, c->d_ff, d, xn, n_rows, g);
    matmul(w->w_up, dt, c->d_ff, d, xn, n_rows, u);
    for (size_t i = 0; i < (size_t)n_rows * c->d_ff; ++i) g[i] = silu(g[i]) * u[i];
    matmul(w->w_down, dt, d, c->d_ff, g, n_rows, o);
    for (size_t i = 0; i < (size_t)n_rows * d; ++i) H[i] += o[i];

    free(xn); free(q); free(k); free(v); free(att); free(o); free(g); free(u);
    return 0;
}

static void embed(const orc_model *m, int tok, double *h) {
    for (int i = 0; i < m->c.d_model; ++i) h[i] = widen(m->tok_embed, m->c.wdtype, (size_t)tok * m->c.d_model + i);
}

/* Final-layer logits z = E* RMSNorm_f(h); returns argmax (lowest index among equal maxima). */
static int final_logits(const orc_model *m, const double *h, double *z) {
    const orc_config *c = &m->c;
    double *xn = (double *)malloc(sizeof(double) * c->d_model);
    rmsnorm(h, m->final_norm, c->wdtype, c->d_model, c->rms_eps, xn);
    matmul(m->lm_head, c->wdtype, c->vocab, c->d_model, xn, 1, z);
    free(xn);
    int best = 0;
    for (int t = 1; t < c->vocab; ++t) if (z[t] > z[best]) best = t;
    return best;
}

/* Intermediate head at 1-based layer (Section 2.1): p = softmax(s * E* T RMSNorm_f(h)).
   Greedy sampling (Appendix D: temperature zero): token = argmax, *p = its probability. */
static int head_eval(const orc_model *m, int layer, const double *h, double *p_out, double *z) {
    const orc_config *c = &m->c;
    const int d = c->d_model;
    double *xn = (double *)malloc(sizeof(double) * d), *tx = (double *)malloc(sizeof(double) * d);
    rmsnorm(h, m->final_norm, c->wdtype, d, c->rms_eps, xn);
    if (m->head_T[layer]) matmul(m->head_T[layer], c->wdtype, d, d, xn, 1, tx);
    else memcpy(tx, xn, sizeof(double) * d);
    matmul(m->lm_head, c->wdtype, c->vocab, d, tx, 1, z);
    int best = 0;
    for (int t = 0; t < c->vocab; ++t) { z[t] *= m->head_scale[layer]; }
    for (int t = 1; t < c->vocab; ++t) if (z[t] > z[best]) best = t;
    double den = 0.0;
    for (int t = 0; t < c->vocab; ++t) den += exp(z[t] - z[best]);
    *p_out = 1.0 / den;
    free(xn); free(tx);
    return best;
}

/* Exposed for tests: head distribution of an arbitrary hidden state (probs may be NULL). */
int orc_head_eval(const orc_model *m, int layer, const double *h, double *p_out, double *probs) {
    double *z = (double *)malloc(sizeof(double) * m->c.vocab);
    int tok = head_eval(m, layer, h, p_out, z);
    if (probs) {
        double den = 0.0;
        for (int t = 0; t < m->c.vocab; ++t) den += exp(z[t] - z[tok]);
        for (int t = 0; t < m->c.vocab; ++t) probs[t] = exp(z[t] - z[tok]) / den;
    }
    free(z);
    return tok;
}

static void record_logits(orc_session *s, const double *z) {
    if (s->logit_sink && s->logit_n < s->logit_cap) {
        memcpy(s->logit_sink + (size_t)s->logit_n * s->m->c.vocab, z, sizeof(double) * s->m->c.vocab);
    }
    if (s->logit_sink) s->logit_n++;
}

/* KV cache <- LM(x) (first line of Algorithm 1): all prompt tokens through all layers.
   The first generated token is the full-depth argmax at the last prompt token; it becomes the
   newest (pending) token.  No BOS is inserted after the prompt. */
int orc_prefill(orc_session *s, const int32_t *prompt, int n) {
    const orc_config *c = &s->m->c;
    if (n < 1 || n + 1 > s->max_seq) return -1;
    for (int i = 0; i < n; ++i) if (prompt[i] < 0 || prompt[i] >= c->vocab) return -2;
    memcpy(s->tokens, prompt, sizeof(int32_t) * n);
    for (int l = 0; l < c->n_layers; ++l) s->kv_len[l] = 0;
    s->n_inflight = 0;
    double *H = (double *)malloc(sizeof(double) * n * c->d_model);
    for (int i = 0; i < n; ++i) embed(s->m, prompt[i], H + (size_t)i * c->d_model);
    for (int l = 0; l < c->n_layers; ++l) {
        int rc = layer_forward(s, l, 0, n, H);
        if (rc) { free(H); return rc; }
    }
    double *z = (double *)malloc(sizeof(double) * c->vocab);
    int tok = final_logits(s->m, H + (size_t)(n - 1) * c->d_model, z);
    record_logits(s, z);
    s->tokens[n] = tok;
    s->len = n + 1;
    s->n_prompt = n;
    s->n_reported = 0;
    free(z); free(H);
    return 0;
}

/* Final-layer logits of every position of an arbitrary token sequence, computed from scratch
   (no incremental state): the plain definition of the model.  out is [n][V]. */
int orc_full_logits(const orc_model *m, const int32_t *tokens, int n, double *out) {
    orc_session *s = orc_session_create(m, n + 1);
    if (!s) return -1;
    const orc_config *c = &m->c;
    double *H = (double *)malloc(sizeof(double) * n * c->d_model);
    for (int i = 0; i < n; ++i) embed(m, tokens[i], H + (size_t)i * c->d_model);
    int rc = 0;
    for (int l = 0; l < c->n_layers && !rc; ++l) rc = layer_forward(s, l, 0, n, H);
    for (int i = 0; i < n && !rc; ++i) final_logits(m, H + (size_t)i * c->d_model, out + (size_t)i * c->vocab);
    free(H);
    orc_session_destroy(s);
    return rc;
}

/* Hidden state of the last token after `upto_layer` layers (1-based count), from scratch. */
int orc_hidden_after(const orc_model *m, const int32_t *tokens, int n, int upto_layer, double *h_out) {
    orc_session *s = orc_session_create(m, n + 1);
    if (!s) return -1;
    const orc_config *c = &m->c;
    double *H = (double *)malloc(sizeof(double) * n * c->d_model);
    for (int i = 0; i < n; ++i) embed(m, tokens[i], H + (size_t)i * c->d_model);
    int rc = 0;
    for (int l = 0; l < upto_layer && !rc; ++l) rc = layer_forward(s, l, 0, n, H);
    memcpy(h_out, H + (size_t)(n - 1) * c->d_model, sizeof(double) * c->d_model);
    free(H);
    orc_session_destroy(s);
    return rc;
}

/* Copy out the next n generated tokens (those not yet reported) and mark them reported. */
static void report(orc_session *s, int n, int32_t *out) {
    memcpy(out, s->tokens + s->n_prompt + s->n_reported, sizeof(int32_t) * n);
    s->n_reported += n;
}

/* Standard greedy autoregressive decoding: returns the next n generated tokens.  After the call
   every token before the last returned one has K/V at all layers and the last one is pending.
   eos_id >= 0: generation stops at the first end-of-sequence token ("while t_i != [EOS]" of
   Algorithm 1, which plain decoding shares): *n_out receives the number of tokens produced, the
   rest of `out` is filled with eos_id. */
int orc_plain_decode(orc_session *s, int n, int eos_id, int32_t *out, int32_t *n_out, orc_stats *st) {
    const orc_config *c = &s->m->c;
    if (s->n_inflight) return -3;
    int target_len = s->n_prompt + s->n_reported + n;
    if (target_len > s->max_seq) return -4;
    double *h = (double *)malloc(sizeof(double) * c->d_model);
    double *z = (double *)malloc(sizeof(double) * c->vocab);
    while (s->len < target_len && !(eos_id >= 0 && s->tokens[s->len - 1] == eos_id)) {
        int pos = s->len - 1;
        embed(s->m, s->tokens[pos], h);
        for (int l = 0; l < c->n_layers; ++l) {
            int rc = layer_forward(s, l, pos, 1, h);
            if (rc) { free(h); free(z); return rc; }
            if (st) st->row_layers++;
        }
        int tok = final_logits(s->m, h, z);
        record_logits(s, z);
        s->tokens[s->len++] = tok;
        if (st) { st->steps++; st->verify_steps++; }
    }
    {
        int got = s->len - (s->n_prompt + s->n_reported);
        if (got > n) got = n;
        report(s, got, out);
        for (int i = got; i < n; ++i) out[i] = eos_id;
        if (n_out) *n_out = got;
    }
    free(h); free(z);
    return 0;
}

/*
 * Algorithm 1.  Returns the next n verified generated tokens.
 *
 *   gamma        early-prediction threshold of Eq. 1 (strict: exit iff p > gamma)
 *   exit_layers  ascending 1-based layers carrying a registered head, each < L
 *   max_early    cap on early predictions in flight between verifications (Appendix D: 5)
 *   tape         optional forced decisions, one entry consumed per head evaluation:
 *                0 = do not exit, 1 = exit, anything else = follow Eq. 1; past the end: Eq. 1
 *   tape_tok     optional forced early tokens, consumed alongside `tape`: >= 0 replaces the
 *                head's argmax as the emitted early token (lets tests plant wrong predictions)
 *
 * Readings of the paper taken here: a token leaves P[l] once layer l has processed it (the
 * worked example of Figure 2 fixes this); heads exist only at intermediate layers, so layer L
 * always verifies; only the newest token t_i consults heads; the rejected token's own K/V is
 * dropped together with everything after it; with max_early predictions in flight, or when the
 * requested count is already reached by tentative tokens, the newest token runs to layer L.
 */
int orc_adaptive_decode(orc_session *s, int n, double gamma, const int32_t *exit_layers, int n_exit,
                        int max_early, const uint8_t *tape, const int32_t *tape_tok, int n_tape, int eos_id,
                        int32_t *out, int32_t *n_out, orc_stats *st) {
    const orc_config *c = &s->m->c;
    const int L = c->n_layers, d = c->d_model;
    if (max_early < 0 || max_early > ORC_MAX_INFLIGHT) return -5;
    if (s->n_inflight) return -3;
    for (int e = 0; e < n_exit; ++e) {
        if (exit_layers[e] < 1 || exit_layers[e] >= L || !s->m->has_head[exit_layers[e]]) return -6;
        if (e && exit_layers[e] <= exit_layers[e - 1]) return -6;
    }
    int target_len = s->n_prompt + s->n_reported + n;
    if (target_len + 1 > s->max_seq) return -4;
    /* while t_i != [EOS]: the pending token is verified; if it is the end-of-sequence token nothing more is generated */
    if (eos_id >= 0 && s->len >= 1 && s->len <= target_len && s->tokens[s->len - 1] == eos_id) target_len = s->len;

    /* P[l]: positions of tokens pending at layer l (1-based l), in sequence order */
    int32_t(*P)[ORC_MAX_INFLIGHT + 1] = calloc(L + 1, sizeof(*P));
    int32_t *Pn = (int32_t *)calloc(L + 1, sizeof(int32_t));
    double *H = (double *)malloc(sizeof(double) * (ORC_MAX_INFLIGHT + 1) * d);
    double *z = (double *)malloc(sizeof(double) * c->vocab);
    int32_t *argm = (int32_t *)malloc(sizeof(int32_t) * (ORC_MAX_INFLIGHT + 1));
    int tape_i = 0, rc = 0;
    int64_t step_no = st ? st->steps : 0;

    /* verified generated tokens so far: everything up to and including the pending token when
       nothing is in flight */
    while (!(s->n_inflight == 0 && s->len >= target_len)) {
        /* while t_i != EOS: the newest token t_i sits at position len-1, nothing computed yet */
        const int pos_new = s->len - 1;
        double *h_new = s->inflight_h + (size_t)s->n_inflight * d; /* slot after the in-flight ones */
        embed(s->m, s->tokens[pos_new], h_new);
        int exited = 0;
        for (int l = 1; l <= L && !exited; ++l) {
            /* P[l] <- P[l] (+) t_i */
            P[l][Pn[l]++] = pos_new;
            /* process all tokens in P[l] in parallel: gather their hidden states in order */
            int n_rows = Pn[l], pos0 = P[l][0];
            for (int r = 0; r < n_rows; ++r) {
                if (P[l][r] != pos0 + r) { rc = -20; goto done; }              /* contiguous suffix */
                int slot = P[l][r] == pos_new ? s->n_inflight : -1;
                for (int f = 0; f < s->n_inflight && slot < 0; ++f) if (s->inflight_pos[f] == P[l][r]) slot = f;
                if (slot < 0) { rc = -21; goto done; }
                if (slot < s->n_inflight && s->inflight_depth[slot] != l - 1) { rc = -22; goto done; }
                memcpy(H + (size_t)r * d, s->inflight_h + (size_t)slot * d, sizeof(double) * d);
            }
            rc = layer_forward(s, l - 1, pos0, n_rows, H);
            if (rc) goto done;
            for (int r = 0; r < n_rows; ++r) {
                int slot = P[l][r] == pos_new ? s->n_inflight : -1;
                for (int f = 0; f < s->n_inflight && slot < 0; ++f) if (s->inflight_pos[f] == P[l][r]) slot = f;
                memcpy(s->inflight_h + (size_t)slot * d, H + (size_t)r * d, sizeof(double) * d);
                if (slot < s->n_inflight) s->inflight_depth[slot] = l;
            }
            if (st) st->row_layers += n_rows;
            if (s->trace) {
                if (s->trace_n < s->trace_cap) {
                    int32_t *t = s->trace + 4 * (size_t)s->trace_n;
                    t[0] = (int32_t)step_no; t[1] = l; t[2] = pos0; t[3] = n_rows;
                }
                s->trace_n++;
            }
            if (l < L) Pn[l] = 0; /* processed tokens leave P[l] */

            /* intermediate head at l?  (only t_i consults it; cap and end-of-call rule) */
            int is_exit_layer = 0;
            for (int e = 0; e < n_exit; ++e) if (exit_layers[e] == l) is_exit_layer = 1;
            if (l < L && is_exit_layer && s->n_inflight < max_early && s->len < target_len) {
                double p;
                int tok = head_eval(s->m, l, h_new, &p, z);
                int decide = p > gamma;
                if (tape_i < n_tape) {
                    if (tape && tape[tape_i] == 0) decide = 0;
                    if (tape && tape[tape_i] == 1) decide = 1;
                    if (tape_tok && tape_tok[tape_i] >= 0) tok = tape_tok[tape_i];
                    tape_i++;
                }
                if (st) st->head_evals++;
                if (s->head_sink) {
                    if (s->head_n < s->head_cap) {
                        double *hs = s->head_sink + 4 * (size_t)s->head_n;
                        hs[0] = (double)step_no; hs[1] = l; hs[2] = tok; hs[3] = p;
                    }
                    s->head_n++;
                }
                if (decide) {
                    /* y <- y (+) t_{i+1};  P[l'] <- P[l'] (+) t_i for l < l' <= L;  break */
                    s->tokens[s->len++] = tok;
                    for (int l2 = l + 1; l2 <= L; ++l2) P[l2][Pn[l2]++] = pos_new;
                    s->inflight_pos[s->n_inflight] = pos_new;
                    s->inflight_depth[s->n_inflight] = l;
                    s->n_inflight++;
                    if (st) { st->early_exits++; st->exits_at_layer[l]++; }
                    exited = 1;
                }
            }
            if (l == L) {
                /* verify all tokens in P[L] in order (Eq. 2, greedy form): row r holds token at
                   position pos0+r; its full-depth argmax must equal the tentative token at
                   position pos0+r+1.  The last row (t_i) has no successor: its argmax is new. */
                for (int r = 0; r < n_rows; ++r) {
                    argm[r] = final_logits(s->m, H + (size_t)r * d, z);
                    /* logits are recorded below only for rows whose output is kept */
                    int keep = 1;
                    for (int q = 0; q < r; ++q) if (argm[q] != s->tokens[pos0 + q + 1]) keep = 0;
                    if (keep) record_logits(s, z);
                }
                int first_bad = -1;
                for (int r = 0; r + 1 < n_rows; ++r)
                    if (argm[r] != s->tokens[pos0 + r + 1]) { first_bad = r; break; }
                if (first_bad < 0) {
                    if (st) st->accepted += n_rows - 1;
                    s->tokens[s->len++] = argm[n_rows - 1]; /* the new token from the full model */
                } else {
                    /* reject the token at position pos0+first_bad+1: replace it by the full-depth
                       argmax, drop it and everything after it from the sequence and from the
                       K/V cache of every layer, resume from the replacement */
                    int bad_pos = pos0 + first_bad + 1;
                    if (st) {
                        st->accepted += first_bad;
                        st->rejected += 1;
                        st->discarded += (n_rows - 1) - first_bad - 1;
                    }
                    s->tokens[bad_pos] = argm[first_bad];
                    s->len = bad_pos + 1;
                    for (int l2 = 0; l2 < L; ++l2) if (s->kv_len[l2] > bad_pos) s->kv_len[l2] = bad_pos;
                }
                Pn[L] = 0;
                s->n_inflight = 0;
                if (st) st->verify_steps++;
                /* while t_i != [EOS]: every token after position pos0 is now verified (each equals the full
                   model's greedy choice); the first end-of-sequence token among them ends the sequence.  An
                   early-predicted end-of-sequence token has stopped nothing until this point. */
                if (eos_id >= 0)
                    for (int q = pos0 + 1; q < s->len; ++q)
                        if (s->tokens[q] == eos_id) { if (q + 1 < target_len) target_len = q + 1; break; }
            }
        }
        if (st) st->steps++;
        step_no++;
        /* invariant: fill levels are non-increasing with depth */
        for (int l2 = 1; l2 < L; ++l2) if (s->kv_len[l2] > s->kv_len[l2 - 1]) { rc = -23; goto done; }
    }
    /* end the call on exactly the requested count: verified tokens beyond it are dropped (they
       will be recomputed by the next call), leaving the same state plain decoding leaves */
    if (s->len > target_len) {
        if (st) st->truncated += s->len - target_len;
        s->len = target_len;
        for (int l2 = 0; l2 < L; ++l2) if (s->kv_len[l2] > target_len - 1) s->kv_len[l2] = target_len - 1;
    }
    {
        int got = s->len - (s->n_prompt + s->n_reported);
        if (got > n) got = n;
        report(s, got, out);
        for (int i = got; i < n; ++i) out[i] = eos_id;
        if (n_out) *n_out = got;
    }
done:
    free(P); free(Pn); free(H); free(z); free(argm);
    return rc;
}

/* ---------------------------------------------------------------- Algorithm 1 with sampling */

#define ORC_NU 8 /* uniforms per sequence position: [0] draw at the last layer, [1] acceptance test of Eq. 2,
                    [2] resampling after a rejection, [3 + e] draw at the e-th exit layer of the call (e < 5) */

/* softmax(z / temperature) into p */
static void softmax_t(const double *z, int V, double temperature, double *p) {
    double zmax = z[0], den = 0.0;
    for (int t = 1; t < V; ++t) if (z[t] > zmax) zmax = z[t];
    for (int t = 0; t < V; ++t) { p[t] = exp((z[t] - zmax) / temperature); den += p[t]; }
    for (int t = 0; t < V; ++t) p[t] /= den;
}

/* Inverse-CDF draw in vocabulary order from the non-negative weights w: the first token whose running
   sum exceeds u x (sum of all weights); the last token of non-zero weight if rounding leaves none. */
static int draw(const double *w, int V, double u, double *margin) {
    double total = 0.0, run = 0.0;
    int last = 0;
    for (int t = 0; t < V; ++t) total += w[t];
    for (int t = 0; t < V; ++t) {
        if (w[t] > 0.0) last = t;
        run += w[t];
        if (run > u * total) {
            /* how far u is from the two ends of the token's interval of the CDF: a caller comparing with a
               lower-precision implementation can tell a decision that rounding could flip */
            if (margin) {
                double lo = u - (run - w[t]) / total, hi = run / total - u;
                if (t > 0 && lo < *margin) *margin = lo;
                if (hi < *margin) *margin = hi;
            }
            return t;
        }
    }
    return last;
}

/*
 * Algorithm 1 with a sampled next token instead of the greedy one.
 *
 *   Eq. 1: at an exit layer the newest token's successor is DRAWN from the head's distribution
 *          q = softmax(head logits / temperature); the draw t is emitted early iff q(t) > gamma,
 *          otherwise it is thrown away and the token climbs on.
 *   Eq. 2: at the last layer every early-predicted token t (drawn from q at its exit layer) is accepted
 *          with probability min{1, p*(t) / q(t)}, p* = softmax(final logits / temperature) of the row
 *          before it, in sequence order; the first rejected one is replaced by a draw from
 *          Normalize(max(0, p* - q)), the K/V of everything from its position on is dropped and
 *          generation resumes from the replacement.  If all are accepted the next token is drawn from
 *          p* of the newest row.
 *
 * Every random number is an input: u[pos * ORC_NU + k] belongs to the token at sequence position pos.
 * A position that is drawn again after a rollback uses its numbers again: they are independent of the
 * event that caused the rollback (the acceptance test of an earlier position).
 *
 * gamma = 0 makes every consulted head emit its draw, which is speculative sampling with the head as
 * the draft distribution: the verified tokens are then distributed exactly as plain sampling from p*.
 * For gamma > 0 the draft is used only where q(t) > gamma and the law of a verified token is
 *   P(v) = sum_i prod_{j<i}(1 - Q_j) [ 1{q_i(v) > gamma} min(q_i(v), p*(v)) + R_i res_i(v) ] + prod_j (1 - Q_j) p*(v),
 * Q_i = sum_{q_i(t) > gamma} q_i(t), R_i = sum_{q_i(t) > gamma} max(0, q_i(t) - p*(t)), res_i = Normalize(max(0, p* - q_i)),
 * which the tests compute independently and compare with the frequencies this function produces.
 */
int orc_sampling_decode(orc_session *s, int n, double temperature, double gamma, const int32_t *exit_layers, int n_exit,
                        int max_early, const double *u, int eos_id, int32_t *out, int32_t *n_out, orc_stats *st,
                        double *min_margin /* nullable: smallest distance, in probability, of any decision from flipping */) {
    const orc_config *c = &s->m->c;
    const int L = c->n_layers, d = c->d_model, V = c->vocab;
    if (max_early < 0 || max_early > ORC_MAX_INFLIGHT) return -5;
    if (s->n_inflight) return -3;
    if (!(temperature > 0.0) || n_exit > ORC_NU - 3 || !u) return -7;
    for (int e = 0; e < n_exit; ++e) {
        if (exit_layers[e] < 1 || exit_layers[e] >= L || !s->m->has_head[exit_layers[e]]) return -6;
        if (e && exit_layers[e] <= exit_layers[e - 1]) return -6;
    }
    int target_len = s->n_prompt + s->n_reported + n;
    if (target_len + 1 > s->max_seq) return -4;
    if (eos_id >= 0 && s->len >= 1 && s->len <= target_len && s->tokens[s->len - 1] == eos_id) target_len = s->len;

    int32_t(*P)[ORC_MAX_INFLIGHT + 1] = calloc(L + 1, sizeof(*P));
    int32_t *Pn = (int32_t *)calloc(L + 1, sizeof(int32_t));
    double *H = (double *)malloc(sizeof(double) * (ORC_MAX_INFLIGHT + 1) * d);
    double *z = (double *)malloc(sizeof(double) * V);
    double *pstar = (double *)malloc(sizeof(double) * V), *res = (double *)malloc(sizeof(double) * V);
    double *Q = (double *)malloc(sizeof(double) * (size_t)(max_early + 1) * V); /* q of every early token in flight */
    int rc = 0;
    int64_t step_no = st ? st->steps : 0;
    double margin = 1.0;

    while (!(s->n_inflight == 0 && s->len >= target_len)) {
        const int pos_new = s->len - 1;
        double *h_new = s->inflight_h + (size_t)s->n_inflight * d;
        embed(s->m, s->tokens[pos_new], h_new);
        int exited = 0;
        for (int l = 1; l <= L && !exited; ++l) {
            P[l][Pn[l]++] = pos_new;
            int n_rows = Pn[l], pos0 = P[l][0];
            for (int r = 0; r < n_rows; ++r) {
                if (P[l][r] != pos0 + r) { rc = -20; goto done; }
                int slot = P[l][r] == pos_new ? s->n_inflight : P[l][r] - s->inflight_pos[0];
                if (slot < 0 || slot > s->n_inflight) { rc = -21; goto done; }
                if (slot < s->n_inflight && (s->inflight_pos[slot] != P[l][r] || s->inflight_depth[slot] != l - 1)) { rc = -22; goto done; }
                memcpy(H + (size_t)r * d, s->inflight_h + (size_t)slot * d, sizeof(double) * d);
            }
            rc = layer_forward(s, l - 1, pos0, n_rows, H);
            if (rc) goto done;
            for (int r = 0; r < n_rows; ++r) {
                int slot = P[l][r] == pos_new ? s->n_inflight : P[l][r] - s->inflight_pos[0];
                memcpy(s->inflight_h + (size_t)slot * d, H + (size_t)r * d, sizeof(double) * d);
                if (slot < s->n_inflight) s->inflight_depth[slot] = l;
            }
            if (st) st->row_layers += n_rows;
            if (l < L) Pn[l] = 0;

            int exit_idx = -1;
            for (int e = 0; e < n_exit; ++e) if (exit_layers[e] == l) exit_idx = e;
            if (l < L && exit_idx >= 0 && s->n_inflight < max_early && s->len < target_len) {
                /* Eq. 1: t ~ q, emitted iff q(t) > gamma */
                double pbest;
                double *q = Q + (size_t)s->n_inflight * V;
                head_eval(s->m, l, h_new, &pbest, z);
                softmax_t(z, V, temperature, q);
                const int tok = draw(q, V, u[(size_t)s->len * ORC_NU + 3 + exit_idx], &margin);
                if (fabs(q[tok] - gamma) < margin) margin = fabs(q[tok] - gamma);
                if (st) st->head_evals++;
                if (s->head_sink) {
                    if (s->head_n < s->head_cap) {
                        double *hs = s->head_sink + 4 * (size_t)s->head_n;
                        hs[0] = (double)step_no; hs[1] = l; hs[2] = tok; hs[3] = q[tok];
                    }
                    s->head_n++;
                }
                if (q[tok] > gamma) {
                    s->tokens[s->len++] = tok;
                    for (int l2 = l + 1; l2 <= L; ++l2) P[l2][Pn[l2]++] = pos_new;
                    s->inflight_pos[s->n_inflight] = pos_new;
                    s->inflight_depth[s->n_inflight] = l;
                    s->n_inflight++;
                    if (st) { st->early_exits++; st->exits_at_layer[l]++; }
                    exited = 1;
                }
            }
            if (l == L) {
                /* Eq. 2: row r holds the token at position pos0 + r; the token after it (position pos0 + r + 1) was
                   drawn from Q[r] when row r left at its exit layer */
                int first_bad = -1;
                for (int r = 0; r + 1 < n_rows && first_bad < 0; ++r) {
                    const int pos_t = pos0 + r + 1, t = s->tokens[pos_t];
                    const double *q = Q + (size_t)r * V;
                    final_logits(s->m, H + (size_t)r * d, z);
                    softmax_t(z, V, temperature, pstar);
                    record_logits(s, z);
                    {
                        const double gap = fabs(u[(size_t)pos_t * ORC_NU + 1] - pstar[t] / q[t]);
                        if (pstar[t] < q[t] && gap < margin) margin = gap;
                    }
                    if (u[(size_t)pos_t * ORC_NU + 1] * q[t] < pstar[t]) continue; /* accepted with probability min{1, p*(t)/q(t)} */
                    first_bad = r;
                    double mass = 0.0;
                    for (int v = 0; v < V; ++v) { res[v] = pstar[v] > q[v] ? pstar[v] - q[v] : 0.0; mass += res[v]; }
                    s->tokens[pos_t] = draw(mass > 0.0 ? res : pstar, V, u[(size_t)pos_t * ORC_NU + 2], &margin);
                    if (st) {
                        st->accepted += r;
                        st->rejected += 1;
                        st->discarded += (n_rows - 1) - r - 1;
                    }
                    s->len = pos_t + 1;
                    for (int l2 = 0; l2 < L; ++l2) if (s->kv_len[l2] > pos_t) s->kv_len[l2] = pos_t;
                }
                if (first_bad < 0) {
                    if (st) st->accepted += n_rows - 1;
                    final_logits(s->m, H + (size_t)(n_rows - 1) * d, z);
                    softmax_t(z, V, temperature, pstar);
                    record_logits(s, z);
                    s->tokens[s->len] = draw(pstar, V, u[(size_t)s->len * ORC_NU + 0], &margin);
                    s->len++;
                }
                Pn[L] = 0;
                s->n_inflight = 0;
                if (st) st->verify_steps++;
                if (eos_id >= 0)
                    for (int q2 = pos0 + 1; q2 < s->len; ++q2)
                        if (s->tokens[q2] == eos_id) { if (q2 + 1 < target_len) target_len = q2 + 1; break; }
            }
        }
        if (st) st->steps++;
        step_no++;
        for (int l2 = 1; l2 < L; ++l2) if (s->kv_len[l2] > s->kv_len[l2 - 1]) { rc = -23; goto done; }
    }
    if (s->len > target_len) {
        if (st) st->truncated += s->len - target_len;
        s->len = target_len;
        for (int l2 = 0; l2 < L; ++l2) if (s->kv_len[l2] > target_len - 1) s->kv_len[l2] = target_len - 1;
    }
    {
        int got = s->len - (s->n_prompt + s->n_reported);
        if (got > n) got = n;
        report(s, got, out);
        for (int i = got; i < n; ++i) out[i] = eos_id;
        if (n_out) *n_out = got;
    }
done:
    if (min_margin) *min_margin = margin;
    free(P); free(Pn); free(H); free(z); free(pstar); free(res); free(Q);
    return rc;
}
