/*
 * EESD decode-round oracle -- TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow CPU statement of what one round of Early-exiting Speculative Decoding
 * computes (Liu et al., "Speculative Decoding via Early-exiting for Faster LLM Inference
 * with Thompson Sampling Control Mechanism"): the draft model of Eq. 1 (first N layers of
 * the target, one early-exit decoder layer, RMSNorm, own vocabulary head), the target
 * model's verification pass (Algorithm 1, verification step), lossless speculative
 * acceptance, and the Beta-posterior Thompson-sampling controller (Eq. 3-4, Algorithm 2).
 *
 * Precision: weights and logits are fp32 values; every activation, dot product, norm and
 * attention softmax is carried in fp64.  Storage formats are part of a configuration: bf16
 * configurations hand this file bf16-rounded weight values and set kv_bf16, which rounds keys
 * and values to bfloat16 when they enter the cache.  The acceptance / sampling arithmetic is the one
 * place where fp32 is fixed, step by step (see "canonical sampling arithmetic" below), so
 * that an independent implementation can reproduce it bit for bit.
 *
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call this file.  It
 * shares no source, table or constant with the CUDA library.
 *
 * Parity pins live in tests/test_oracle_*.py.  Unpinned: behaviour on real LLaMA-2 weights
 * (acceptance rates of trained exit layers) -- "parity unpinned", no weights available.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int d, H, Hkv, D, F, V, L, N; /* L target layers, N early layers shared with the draft */
    int max_ctx;
    double eps, theta;
    int kv_bf16; /* 1: cached keys/values are stored rounded to bfloat16 (the storage format of
                    the bf16 configurations); arithmetic on them stays fp64 */
    int E;       /* early-exit layers of the draft model (the experiment on the number of exit layers;
                    Eq. 1 has one): a stack of E decoder layers on H^N, each with its own weights and
                    cache slot; 0 reads as 1 */
} orc_cfg;

typedef struct {
    const float *g_attn, *wqkv, *wo, *g_ffn, *wg, *wu, *wd;
} orc_layer;

typedef struct {
    orc_cfg c;
    const float *embed, *g_final, *lm_head, *g_exit, *exit_head;
    orc_layer *layers; /* L target layers; indices L .. L+E-1 are the early-exit layers */
    double *kc, *vc;   /* [(L+E)][max_ctx][Hkv*D] rotated keys / values */
} orc_model;

/* ------------------------------------------------------------------ model plumbing */
orc_model *orc_model_new(const orc_cfg *c) {
    orc_model *m = (orc_model *)calloc(1, sizeof(orc_model));
    m->c = *c;
    if (m->c.E < 1) m->c.E = 1;
    m->layers = (orc_layer *)calloc((size_t)c->L + m->c.E, sizeof(orc_layer));
    size_t n = (size_t)(c->L + m->c.E) * c->max_ctx * c->Hkv * c->D;
    m->kc = (double *)calloc(n, sizeof(double));
    m->vc = (double *)calloc(n, sizeof(double));
    return m;
}
void orc_model_free(orc_model *m) {
    if (!m) return;
    free(m->layers); free(m->kc); free(m->vc); free(m);
}
void orc_set_layer(orc_model *m, int idx, const float *g_attn, const float *wqkv, const float *wo,
                   const float *g_ffn, const float *wg, const float *wu, const float *wd) {
    orc_layer *l = &m->layers[idx];
    l->g_attn = g_attn; l->wqkv = wqkv; l->wo = wo; l->g_ffn = g_ffn; l->wg = wg; l->wu = wu; l->wd = wd;
}
void orc_set_globals(orc_model *m, const float *embed, const float *g_final, const float *lm_head,
                     const float *g_exit, const float *exit_head) {
    m->embed = embed; m->g_final = g_final; m->lm_head = lm_head; m->g_exit = g_exit; m->exit_head = exit_head;
}

/* ------------------------------------------------------------------ layer pieces */
/* RMSNorm (LLaMA form, named in Sec. 3.1): out = x * g / sqrt(mean(x^2) + eps) */
void orc_rmsnorm(const double *x, const float *g, int d, double eps, double *out) {
    double ss = 0.0;
    for (int i = 0; i < d; i++) ss += x[i] * x[i];
    double r = 1.0 / sqrt(ss / d + eps);
    for (int i = 0; i < d; i++) out[i] = x[i] * r * (double)g[i];
}

/* Rotary position embedding on one head vector: pair (2i, 2i+1) turns by pos * theta^(-2i/D) */
void orc_rope(double *v, int D, int pos, double theta) {
    for (int i = 0; i < D / 2; i++) {
        double ang = (double)pos * pow(theta, -2.0 * i / D);
        double c = cos(ang), s = sin(ang);
        double a = v[2 * i], b = v[2 * i + 1];
        v[2 * i] = a * c - b * s;
        v[2 * i + 1] = a * s + b * c;
    }
}

/* y[r] = sum_k W[r][k] * x[k], W fp32 [rows][cols] row-major */
static void matvec(const float *W, const double *x, int rows, int cols, double *y) {
#pragma omp parallel for schedule(static)
    for (int r = 0; r < rows; r++) {
        const float *w = W + (size_t)r * cols;
        double acc = 0.0;
        for (int k = 0; k < cols; k++) acc += (double)w[k] * x[k];
        y[r] = acc;
    }
}

/* value of x after storage as bfloat16: round to nearest even on the upper 16 bits of fp32 */
double orc_bf16_round(double x) {
    union { float f; uint32_t u; } v;
    v.f = (float)x;
    if ((v.u & 0x7F800000u) == 0x7F800000u) return (double)v.f; /* inf / nan unchanged */
    v.u += 0x7FFFu + ((v.u >> 16) & 1u);
    v.u &= 0xFFFF0000u;
    return (double)v.f;
}

static double *cache_row(double *base, const orc_cfg *c, int slot, int pos) {
    return base + ((size_t)slot * c->max_ctx + pos) * ((size_t)c->Hkv * c->D);
}

/* Keys/values of rows x[M][d] at positions pos0.. for cache slot `slot` using layer `lw`:
 * k = RoPE(Wk . RMSNorm(x)), v = Wv . RMSNorm(x).  Optionally returns q (rotated). */
static void project_qkv(orc_model *m, const orc_layer *lw, int slot, const double *x, int M, int pos0,
                        double *q_out /* [M][H*D] or NULL */) {
    const orc_cfg *c = &m->c;
    int qd = c->H * c->D, kvd = c->Hkv * c->D;
    double *n = (double *)malloc(sizeof(double) * c->d);
    double *qkv = (double *)malloc(sizeof(double) * (qd + 2 * kvd));
    for (int r = 0; r < M; r++) {
        int pos = pos0 + r;
        orc_rmsnorm(x + (size_t)r * c->d, lw->g_attn, c->d, c->eps, n);
        if (q_out) {
            matvec(lw->wqkv, n, qd + 2 * kvd, c->d, qkv);
            for (int h = 0; h < c->H; h++) orc_rope(qkv + h * c->D, c->D, pos, c->theta);
            memcpy(q_out + (size_t)r * qd, qkv, sizeof(double) * qd);
        } else {
            matvec(lw->wqkv + (size_t)qd * c->d, n, 2 * kvd, c->d, qkv + qd);
        }
        for (int h = 0; h < c->Hkv; h++) orc_rope(qkv + qd + h * c->D, c->D, pos, c->theta);
        if (c->kv_bf16)
            for (int i = 0; i < 2 * kvd; i++) qkv[qd + i] = orc_bf16_round(qkv[qd + i]);
        memcpy(cache_row(m->kc, c, slot, pos), qkv + qd, sizeof(double) * kvd);
        memcpy(cache_row(m->vc, c, slot, pos), qkv + qd + kvd, sizeof(double) * kvd);
    }
    free(n); free(qkv);
}

/* One decoder layer on M new rows at positions pos0..pos0+M-1 (x updated in place):
 *   x += Wo . Attn(q, K[0..pos], V[0..pos]);  x += Wd . (silu(Wg n) * (Wu n)),  n = RMSNorm(x)
 * `lidx` picks the weights, `slot` the KV cache (they differ only in tests). */
void orc_layer_fwd(orc_model *m, int lidx, int slot, double *x, int M, int pos0) {
    const orc_cfg *c = &m->c;
    const orc_layer *lw = &m->layers[lidx];
    int qd = c->H * c->D, grp = c->H / c->Hkv;
    double *q = (double *)malloc(sizeof(double) * (size_t)M * qd);
    double *att = (double *)malloc(sizeof(double) * qd);
    double *sc = (double *)malloc(sizeof(double) * c->max_ctx);
    double *o = (double *)malloc(sizeof(double) * c->d);
    double *n = (double *)malloc(sizeof(double) * c->d);
    double *g = (double *)malloc(sizeof(double) * c->F);
    double *u = (double *)malloc(sizeof(double) * c->F);
    project_qkv(m, lw, slot, x, M, pos0, q);
    double inv = 1.0 / sqrt((double)c->D);
    for (int r = 0; r < M; r++) {
        int pos = pos0 + r; /* attends to cache positions 0..pos (causal) */
        double *xr = x + (size_t)r * c->d;
        for (int h = 0; h < c->H; h++) {
            const double *qh = q + (size_t)r * qd + h * c->D;
            int kh = h / grp;
            double mx = -INFINITY;
            for (int j = 0; j <= pos; j++) {
                const double *kj = cache_row(m->kc, c, slot, j) + kh * c->D;
                double s = 0.0;
                for (int e = 0; e < c->D; e++) s += qh[e] * kj[e];
                sc[j] = s * inv;
                if (sc[j] > mx) mx = sc[j];
            }
            double z = 0.0;
            for (int j = 0; j <= pos; j++) { sc[j] = exp(sc[j] - mx); z += sc[j]; }
            double *ah = att + h * c->D;
            for (int e = 0; e < c->D; e++) ah[e] = 0.0;
            for (int j = 0; j <= pos; j++) {
                const double *vj = cache_row(m->vc, c, slot, j) + kh * c->D;
                double w = sc[j] / z;
                for (int e = 0; e < c->D; e++) ah[e] += w * vj[e];
            }
        }
        matvec(lw->wo, att, c->d, qd, o);
        for (int i = 0; i < c->d; i++) xr[i] += o[i];
        orc_rmsnorm(xr, lw->g_ffn, c->d, c->eps, n);
        matvec(lw->wg, n, c->F, c->d, g);
        matvec(lw->wu, n, c->F, c->d, u);
        for (int i = 0; i < c->F; i++) g[i] = g[i] / (1.0 + exp(-g[i])) * u[i];
        matvec(lw->wd, g, c->d, c->F, o);
        for (int i = 0; i < c->d; i++) xr[i] += o[i];
    }
    free(q); free(att); free(sc); free(o); free(n); free(g); free(u);
}

void orc_embed(const orc_model *m, const int32_t *tok, int M, double *x) {
    for (int r = 0; r < M; r++)
        for (int i = 0; i < m->c.d; i++) x[(size_t)r * m->c.d + i] = (double)m->embed[(size_t)tok[r] * m->c.d + i];
}

/* logits[r][v] = W[v] . RMSNorm(x[r]; g), rounded to fp32 */
void orc_head(const orc_model *m, const double *x, int M, const float *g, const float *W, float *logits) {
    const orc_cfg *c = &m->c;
    double *n = (double *)malloc(sizeof(double) * c->d);
    double *y = (double *)malloc(sizeof(double) * c->V);
    for (int r = 0; r < M; r++) {
        orc_rmsnorm(x + (size_t)r * c->d, g, c->d, c->eps, n);
        matvec(W, n, c->V, c->d, y);
        for (int v = 0; v < c->V; v++) logits[(size_t)r * c->V + v] = (float)y[v];
    }
    free(n); free(y);
}

/* Target model on M rows (tokens at positions pos0..): all L layers, KV rows written for
 * every layer, and the exit layers' k,v written for the same positions: those of the first exit
 * layer depend on H^N only; with E > 1 exit layers, those of exit layer e depend on the output of
 * exit layer e-1, so exit layers 1..E-1 run in full on a copy of H^N (the target's own residual
 * stream is not touched) and the last one contributes its key / value projection only.  hidden
 * (optional) receives the residual stream after the embedding and after every target layer:
 * [(L+1)][M][d].  logits (optional) [M][V]. */
void orc_target_rows(orc_model *m, const int32_t *tok, int M, int pos0, double *hidden, float *logits) {
    const orc_cfg *c = &m->c;
    size_t md = (size_t)M * c->d;
    double *x = (double *)malloc(sizeof(double) * md);
    orc_embed(m, tok, M, x);
    if (hidden) memcpy(hidden, x, sizeof(double) * md);
    for (int l = 0; l < c->L; l++) {
        orc_layer_fwd(m, l, l, x, M, pos0);
        if (hidden) memcpy(hidden + (size_t)(l + 1) * md, x, sizeof(double) * md);
        if (l == c->N - 1) {
            double *xe = (double *)malloc(sizeof(double) * md);
            memcpy(xe, x, sizeof(double) * md);
            for (int e = 0; e < c->E - 1; e++) orc_layer_fwd(m, c->L + e, c->L + e, xe, M, pos0);
            project_qkv(m, &m->layers[c->L + c->E - 1], c->L + c->E - 1, xe, M, pos0, NULL);
            free(xe);
        }
    }
    if (logits) orc_head(m, x, M, m->g_final, m->lm_head, logits);
    free(x);
}

/* Draft model (Eq. 1) on ONE row: first N layers (sharing the target's KV cache), the
 * early-exit layer(s) with their own weights and KV slots, RMSNorm, exit head W. */
void orc_draft_row(orc_model *m, int32_t tok, int pos, float *logits, double *hidden_exit /* [d] or NULL */) {
    const orc_cfg *c = &m->c;
    double *x = (double *)malloc(sizeof(double) * c->d);
    orc_embed(m, &tok, 1, x);
    for (int l = 0; l < c->N; l++) orc_layer_fwd(m, l, l, x, 1, pos);
    for (int e = 0; e < c->E; e++) orc_layer_fwd(m, c->L + e, c->L + e, x, 1, pos);
    if (hidden_exit) memcpy(hidden_exit, x, sizeof(double) * c->d);
    orc_head(m, x, 1, m->g_exit, m->exit_head, logits);
    free(x);
}

/* ------------------------------------------------------------------ canonical sampling arithmetic
 * The paper states no stochastic acceptance formula (its runs are greedy); the rule is the
 * standard lossless one it cites: accept x_i with probability min(1, p_i(x_i)/q_i(x_i)); at
 * the first rejection emit y ~ normalize(max(0, p_j - q_j)); with no rejection emit
 * y ~ p_{K+1}.  To make every decision a pure function of (logits, uniforms) independent of
 * summation order, the arithmetic is fixed as follows (all fp32 ops round to nearest even):
 *   m   = max_v logit_v                       t_v = (logit_v - m) / T
 *   e_v = exp_spec(t_v)                       (below)
 *   Z   = sum_v floor(e_v * 2^40)  in uint64  Zf = float(Z) * 2^-40
 *   prob_v = e_v / Zf
 *   inverse CDF of weights w: W = sum floor(w_v * 2^32) (uint64); u = m_u * 2^-24;
 *       tau = (m_u * W) >> 24; emit the smallest v whose inclusive prefix sum exceeds tau.
 *   accept test: fl(u * q(x)) < p(x).
 * exp_spec(t), t <= 0: 0 if t < -64; else n = rint(fl(t * log2e)); r = fma(-n, ln2_hi, t);
 *   r = fma(-n, ln2_lo, r); degree-6 Horner polynomial in r with fmaf; times 2^n. */
static float bits_f32(uint32_t b) { union { uint32_t u; float f; } s; s.u = b; return s.f; }
static float exp_spec(float t) {
    if (!(t >= -64.0f)) return 0.0f;
    const float LOG2E = bits_f32(0x3FB8AA3Bu);  /* fl(log2 e) */
    const float LN2_HI = bits_f32(0x3F317200u); /* ln 2 to 12 fewer bits, so n * LN2_HI is exact */
    const float LN2_LO = bits_f32(0x35BFBE8Eu); /* fl(ln 2 - LN2_HI) */
    float n = rintf(t * LOG2E);
    float r = fmaf(-n, LN2_HI, t);
    r = fmaf(-n, LN2_LO, r);
    float p = bits_f32(0x3AB60B61u);            /* 1/720 */
    p = fmaf(p, r, bits_f32(0x3C088889u));      /* 1/120 */
    p = fmaf(p, r, bits_f32(0x3D2AAAABu));      /* 1/24  */
    p = fmaf(p, r, bits_f32(0x3E2AAAABu));      /* 1/6   */
    p = fmaf(p, r, 0.5f);
    p = fmaf(p, r, 1.0f);
    p = fmaf(p, r, 1.0f);
    return p * bits_f32((uint32_t)((int)n + 127) << 23); /* times 2^n, n in [-93, 0] */
}
float orc_exp_spec(float t) { return exp_spec(t); }

/* prob[v] for one row of logits at temperature T (> 0) */
void orc_softmax_spec(const float *logits, int V, float T, float *prob) {
    float m = logits[0];
    for (int v = 1; v < V; v++) if (logits[v] > m) m = logits[v];
    uint64_t Z = 0;
    for (int v = 0; v < V; v++) {
        float e = exp_spec((logits[v] - m) / T);
        prob[v] = e;
        Z += (uint64_t)(e * 1099511627776.0f); /* floor(e * 2^40), exact product */
    }
    float Zf = (float)Z * (1.0f / 1099511627776.0f);
    for (int v = 0; v < V; v++) prob[v] = prob[v] / Zf;
}

/* inverse-CDF draw from non-negative weights w (fp32, each <= 1) with uniform u = m_u 2^-24.
 * Returns -1 when every weight floors to zero. */
int orc_sample_weights(const float *w, int V, float u) {
    uint64_t W = 0;
    for (int v = 0; v < V; v++) W += (uint64_t)(w[v] * 4294967296.0f);
    if (W == 0) return -1;
    uint64_t mu = (uint64_t)(u * 16777216.0f);
    uint64_t tau = (mu * W) >> 24;
    uint64_t acc = 0;
    for (int v = 0; v < V; v++) {
        acc += (uint64_t)(w[v] * 4294967296.0f);
        if (acc > tau) return v;
    }
    return V - 1; /* unreachable: tau < W */
}

int orc_argmax(const float *x, int V) {
    int b = 0;
    for (int v = 1; v < V; v++) if (x[v] > x[b]) b = v; /* lowest index wins ties */
    return b;
}

/* token from one row of logits: greedy if T == 0, else x ~ softmax(logits / T) */
int orc_sample_logits(const float *logits, int V, float T, float u) {
    if (T == 0.0f) return orc_argmax(logits, V);
    float *p = (float *)malloc(sizeof(float) * V);
    orc_softmax_spec(logits, V, T, p);
    int x = orc_sample_weights(p, V, u);
    free(p);
    return x;
}

/* Verification of K drafted tokens x[0..K-1] of one sequence.
 * p_logits [K+1][V]: target logits; row i is the target's distribution for draft token i,
 * row K for the bonus token.  q_logits [K][V]: draft logits the tokens were drawn from.
 * Returns the number of accepted tokens and the emitted correction / bonus token y. */
void orc_accept_resample(const float *p_logits, const float *q_logits, const int32_t *x,
                         const float *u_acc, float u_res, int K, int V, float T,
                         int *n_acc, int *y) {
    int j = 0;
    if (T == 0.0f) { /* greedy rule (footnote of Sec. 4.1): keep the prefix equal to the target's top-1 */
        while (j < K && x[j] == orc_argmax(p_logits + (size_t)j * V, V)) j++;
        *n_acc = j;
        *y = orc_argmax(p_logits + (size_t)j * V, V);
        return;
    }
    float *p = (float *)malloc(sizeof(float) * V);
    float *q = (float *)malloc(sizeof(float) * V);
    for (; j < K; j++) {
        orc_softmax_spec(p_logits + (size_t)j * V, V, T, p);
        orc_softmax_spec(q_logits + (size_t)j * V, V, T, q);
        float lhs = u_acc[j] * q[x[j]];
        if (!(lhs < p[x[j]])) break; /* rejected */
    }
    *n_acc = j;
    if (j == K) {
        orc_softmax_spec(p_logits + (size_t)K * V, V, T, p);
        *y = orc_sample_weights(p, V, u_res);
    } else {
        for (int v = 0; v < V; v++) { float r = p[v] - q[v]; q[v] = r > 0.0f ? r : 0.0f; }
        int t = orc_sample_weights(q, V, u_res);
        if (t < 0) t = orc_sample_weights(p, V, u_res); /* p == q to the last bit */
        *y = t;
    }
    free(p); free(q);
}

void orc_accept_resample_batch(const float *p_logits, const float *q_logits, const int32_t *x,
                               const float *u_acc, const float *u_res, int B, int K, int V, float T,
                               int *n_acc, int *y) {
#pragma omp parallel for schedule(dynamic)
    for (int b = 0; b < B; b++)
        orc_accept_resample(p_logits + (size_t)b * (K + 1) * V, q_logits + (size_t)b * K * V,
                            x + (size_t)b * K, u_acc + (size_t)b * K, u_res[b], K, V, T, &n_acc[b], &y[b]);
}

/* ------------------------------------------------------------------ Thompson-sampling controller
 * Beta posterior over the continue-probability theta (Sec. 3.3).  alpha, beta stay integers
 * (integer prior, integer updates), so theta ~ Beta(a, b) is drawn as X / (X + Y) with
 * X ~ Gamma(a, 1) = -sum_{a} ln u, Y ~ Gamma(b, 1) likewise.  Uniforms come from the
 * caller's stream u[*cursor...]; a zero uniform is replaced by 2^-25.  Returns chi in {0,1};
 * -1 when the stream is exhausted. */
static double neg_log_u(float u) { return -log(u > 0.0f ? (double)u : 2.98023223876953125e-08); }

int orc_ts_continue(long alpha, long beta, const float *u, long n_u, long *cursor, double *theta_out) {
    if (*cursor + alpha + beta + 1 > n_u) return -1;
    double X = 0.0, Y = 0.0;
    for (long i = 0; i < alpha; i++) X += neg_log_u(u[(*cursor)++]);
    for (long i = 0; i < beta; i++) Y += neg_log_u(u[(*cursor)++]);
    double theta = X / (X + Y);
    if (theta_out) *theta_out = theta;
    return (double)u[(*cursor)++] < theta ? 1 : 0;
}

/* Posterior update after a round that drafted n_draft tokens and added q_v tokens to the
 * output (Eq. 3-4; Algorithm 2, update steps): r = |Q_v| - 1, n = min(|Q_v| + 1, |Q_d|).
 * rule 0: as printed.  rule 1: n = min(|Q_v|, |Q_d|) (one failure at most). */
void orc_ts_update(long *alpha, long *beta, int q_v, int n_draft, int rule) {
    long r = q_v - 1;
    long n = rule == 0 ? (q_v + 1 < n_draft ? q_v + 1 : n_draft) : (q_v < n_draft ? q_v : n_draft);
    *alpha += r;
    *beta += n - r;
}

/* ------------------------------------------------------------------ generation (Algorithm 1) */
/* ------------------------------------------------------------------ Thompson sampling with calibration
 * (Sec. 3.3 "TS with Calibration", Eq. 5-8, Algorithm 3).  Readings where the text leaves a choice:
 *  - Eq. 5 applies "Sigmoid" to the output of a TWO-row W_p trained with cross-entropy: theta_M is
 *    read as the class-1 probability of the 2-class softmax, 1 / (1 + exp(l_0 - l_1)).
 *  - H_t^(T): the target's residual stream after its last layer (before the final norm) at the
 *    last position the target has processed; H_{t+i}^(D): the draft model's residual stream after
 *    the early-exit layer (before its norm) at the current draft step.
 *  - W^i: i is the number of the draft step within the round (1-based), capped at 10.
 *  - theta_hat: Eq. 8 read literally (with |Q_v| counting the token the target supplies) adds the
 *    same amount to numerator and denominator and can only rise towards 1; the text calls it the
 *    observed sample mean of chi, so it is kept as exactly that: with r successes in n verified
 *    drafts of a round (the r, n of Eq. 3-4), theta_hat <- (theta_hat * (N + 1) + r) / (N + n + 1),
 *    N = verified drafts so far, the initial theta_hat_0 weighing as one observation (the "+1"
 *    of Eq. 8). */
double orc_cali_theta_m(const float *Wi /* [d][d] */, const float *Wp /* [2][2d] */, const double *hT,
                        const double *hD, int d) {
    double *v = (double *)malloc(sizeof(double) * d);
    matvec(Wi, hT, d, d, v);
    double l[2];
    for (int c = 0; c < 2; c++) {
        double s = 0.0;
        for (int k = 0; k < d; k++) s += (double)Wp[(size_t)c * 2 * d + k] * v[k];
        for (int k = 0; k < d; k++) s += (double)Wp[(size_t)c * 2 * d + d + k] * hD[k];
        l[c] = s;
    }
    free(v);
    return 1.0 / (1.0 + exp(l[0] - l[1]));
}

/* Eq. 6 and Eq. 7: posterior of mu after n verifications */
void orc_cali_posterior(double theta_m, double theta_hat, long n, double sigma_m, double sigma_s, double *mu, double *var) {
    const double sm2 = sigma_m * sigma_m, ss2 = sigma_s * sigma_s;
    const double den = (double)n * sm2 + ss2;
    *mu = ss2 / den * theta_m + (double)n * sm2 / den * theta_hat;
    *var = sm2 * ss2 / (ss2 + (double)n * sm2);
}

double orc_cali_theta_hat(double prev, long trials_prev, int r, int n) {
    return (prev * (double)(trials_prev + 1) + (double)r) / (double)(trials_prev + n + 1);
}

/* theta ~ N(mu, var) by the Box-Muller transform of two uniforms, chi ~ Bernoulli(theta) from a
 * third (theta outside [0, 1] acts as 0 or 1).  Returns chi, or -1 when the stream is exhausted. */
int orc_cali_continue(double mu, double var, const float *u, long n_u, long *cursor, double *theta_out) {
    if (*cursor + 3 > n_u) return -1;
    const double r = sqrt(2.0 * neg_log_u(u[(*cursor)++]));
    const double z = r * cos(6.283185307179586476925286766559 * (double)u[(*cursor)++]);
    const double theta = mu + sqrt(var) * z;
    if (theta_out) *theta_out = theta;
    return (double)u[(*cursor)++] < theta ? 1 : 0;
}

typedef struct {
    int max_new;
    int k_cap;          /* upper bound on drafted tokens per round */
    float temperature;  /* 0 = greedy */
    int controller;     /* 0: K from k_schedule[round] (or fixed_k), 1: Beta-TS, 2: TS with calibration */
    int fixed_k;
    long alpha0, beta0;
    int ts_rule;
    const int *k_schedule; int n_schedule;
    const float *u_draft, *u_accept, *u_resample; /* indexed by absolute token position:
        u_draft / u_accept by the position the drafted token takes, u_resample by the position
        of the round's first drafted token */
    const float *u_ctrl; long n_ctrl;             /* consumed in order */
    /* TS with calibration: predictor weights W^1..W^10 ([10][d][d]) and W_p ([2][2d]), the
     * hyper-parameters sigma_M, sigma_S and the initial sample mean theta_hat_0 */
    const float *cali_w, *cali_wp;
    double sigma_m, sigma_s, theta_hat0;
} orc_gen_cfg;

typedef struct { int k, n_acc, y; } orc_round;

/* Prefill: prompt tokens 0..n-2 go through the target (and the exit layer's k,v); the last
 * prompt token stays pending.  Then rounds of {draft until the controller stops, verify,
 * accept, update} until max_new tokens exist.  |Q_v| = accepted drafts + the one token the
 * target itself supplies, so t always advances.  Returns the number of rounds. */
int orc_generate(orc_model *m, const int32_t *prompt, int n_prompt, const orc_gen_cfg *g,
                 int32_t *out /* [max_new] */, orc_round *trace, int trace_cap, long *alpha_out, long *beta_out) {
    const orc_cfg *c = &m->c;
    int V = c->V, K_cap = g->k_cap;
    int32_t *ctx = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n_prompt + g->max_new + K_cap + 2));
    memcpy(ctx, prompt, sizeof(int32_t) * n_prompt);
    int T = n_prompt;
    const int cali = g->controller == 2;
    const int d = c->d;
    double *hT = (double *)calloc((size_t)d, sizeof(double));   /* H^(T): zeros until the target has run */
    double *hD = (double *)malloc(sizeof(double) * d);
    double *hid = NULL;
    if (cali) hid = (double *)malloc(sizeof(double) * (size_t)(c->L + 1) * (n_prompt > K_cap + 1 ? n_prompt : K_cap + 1) * d);
    if (n_prompt > 1) {
        orc_target_rows(m, prompt, n_prompt - 1, 0, hid, NULL);
        if (cali) memcpy(hT, hid + ((size_t)c->L * (n_prompt - 1) + (n_prompt - 2)) * d, sizeof(double) * d);
    }
    double theta_hat = g->theta_hat0;
    long n_verify = 0, trials = 0;
    float *ql = (float *)malloc(sizeof(float) * (size_t)K_cap * V);
    float *pl = (float *)malloc(sizeof(float) * (size_t)(K_cap + 1) * V);
    int32_t *xs = (int32_t *)malloc(sizeof(int32_t) * (K_cap + 1));
    long alpha = g->alpha0, beta = g->beta0, cur = 0;
    int t = 0, rounds = 0;
    while (t < g->max_new) {
        /* draft loop: x_0 is the pending token ctx[T-1] */
        int k_force = -1;
        if (g->controller == 0) {
            k_force = (g->k_schedule && rounds < g->n_schedule) ? g->k_schedule[rounds] : g->fixed_k;
            if (k_force > K_cap) k_force = K_cap;
            if (k_force < 1) k_force = 1;
        }
        xs[0] = ctx[T - 1];
        int K = 0;
        while (1) {
            int pos = T - 1 + K; /* position of the token fed to the draft model */
            orc_draft_row(m, xs[K], pos, ql + (size_t)K * V, cali ? hD : NULL);
            xs[K + 1] = orc_sample_logits(ql + (size_t)K * V, V, g->temperature, g->u_draft ? g->u_draft[pos + 1] : 0.0f);
            K++;
            if (K >= K_cap || T + K >= c->max_ctx - 1) break;
            if (g->controller == 0) { if (K >= k_force) break; }
            else if (cali) {
                const int wi = (K < 10 ? K : 10) - 1;   /* K drafts done: this was draft step K */
                const double th_m = orc_cali_theta_m(g->cali_w + (size_t)wi * d * d, g->cali_wp, hT, hD, d);
                double mu, var;
                orc_cali_posterior(th_m, theta_hat, n_verify, g->sigma_m, g->sigma_s, &mu, &var);
                int chi = orc_cali_continue(mu, var, g->u_ctrl, g->n_ctrl, &cur, NULL);
                if (chi <= 0) break;
            } else {
                int chi = orc_ts_continue(alpha, beta, g->u_ctrl, g->n_ctrl, &cur, NULL);
                if (chi <= 0) break;
            }
        }
        /* verify: K+1 rows x_0..x_K at positions T-1..T-1+K */
        orc_target_rows(m, xs, K + 1, T - 1, hid, pl);
        int n_acc, y;
        orc_accept_resample(pl, ql, xs + 1, g->u_accept ? g->u_accept + T : NULL,
                            g->u_resample ? g->u_resample[T] : 0.0f, K, V, g->temperature, &n_acc, &y);
        for (int i = 0; i < n_acc; i++) ctx[T + i] = xs[1 + i];
        ctx[T + n_acc] = y;
        if (trace && rounds < trace_cap) { trace[rounds].k = K; trace[rounds].n_acc = n_acc; trace[rounds].y = y; }
        T += n_acc + 1;
        t += n_acc + 1;
        orc_ts_update(&alpha, &beta, n_acc + 1, K, g->ts_rule);
        if (cali) {
            /* the row whose logits gave the next token is row n_acc of this pass */
            memcpy(hT, hid + ((size_t)c->L * (K + 1) + n_acc) * d, sizeof(double) * d);
            long a0 = 0, b0 = 0;
            orc_ts_update(&a0, &b0, n_acc + 1, K, g->ts_rule);   /* r and n - r of this round (Eq. 3-4) */
            theta_hat = orc_cali_theta_hat(theta_hat, trials, (int)a0, (int)(a0 + b0));
            trials += a0 + b0;
            n_verify++;
        }
        rounds++;
    }
    memcpy(out, ctx + n_prompt, sizeof(int32_t) * g->max_new);
    if (alpha_out) *alpha_out = alpha;
    if (beta_out) *beta_out = beta;
    free(ctx); free(ql); free(pl); free(xs); free(hT); free(hD); free(hid);
    return rounds;
}
