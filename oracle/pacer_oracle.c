/*
 * CPU oracle for the Pacer hot path.  TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, double-precision restatement of what the speculative decoding
 * loop with blockwise pre-verification computes.  Only the test-suite, the smoke
 * check and the benchmark's cpu-baseline leg may call it.  It shares no code,
 * table or constant with the CUDA library, and neither includes the other.
 *
 * What follows the paper, and where:
 *   orc_forward           Eq. 1 / Eq. 2: a decoder run on n new rows against a KV
 *                         cache (the decoder itself is a Llama-style stack; the
 *                         paper fixes no architecture, the workload does).
 *   orc_preverify         Eq. 7 and Algorithm 1 (pre-verification of a block with
 *                         the past KV cache, position embeddings e_i, mean test,
 *                         threshold growth).
 *   orc_draft_block       Eq. 6: b autoregressive draft forwards with hidden states.
 *   orc_verify            Eq. 4: one parallel target forward over the drafts.
 *   orc_accept            Eq. 5 and Algorithm 1's acceptance part: rejection
 *                         sampling, residual resampling, bonus token; the greedy
 *                         case is the same rule with one-hot distributions.
 *   orc_generate_pacer    Algorithm 1 as a whole.
 *   orc_generate_sd       Section 2.2 (fixed window), written separately.
 *   orc_generate_sched    Section 2.2 with a window given per step; with the windows
 *                         L_A* of a large-window run it is the gamma* decoding of
 *                         Section 3.1 (the oracle-knowledge upper bound).
 *   orc_generate_ar       Eq. 1 on the target: the definition of the lossless output.
 *
 * Readings of the paper taken where it is silent (each also listed in the design
 * notes of the repository): stop test is "mean <= t" (Algorithm 1); t restarts
 * at t0 every draft-and-verify step and grows by repeated fp32 multiplication;
 * the failing block is still verified; h_i is the draft's final-norm output of
 * the forward that emitted y_i, so the draft cache lacks y_gamma and catches up
 * with a two-row forward after a fully accepted step; M_B is one decoder layer at
 * draft width with its own KV cache, RMSNorm and a 2-way linear head, alpha_hat =
 * softmax(.)[1]; rows of accepted history carry no position embedding; M_B's
 * cache is truncated together with the draft's.  The restricted attention
 * contexts of the ablation ("local draft", "local block") start at the first
 * draft row of the step / of the block; a history row then sees itself only.
 *
 * Parity pins live in tests/test_oracle_*.py.  Unpinned: the architecture of M_B
 * against the authors' trained module (no checkpoint exists here) - "parity
 * unpinned" for that one choice.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <stdio.h>

typedef double real;

typedef struct {
    int32_t n_layers, d_model, n_heads, n_kv_heads, d_ffn, vocab;
    float rope_theta, rms_eps;
    int32_t wdtype;     /* 0: float32 values, 1: bfloat16 bit patterns (uint16) */
    int32_t n_posemb;   /* rows of posemb (pre-verification layer only) */
    const void *embed, *wqkv, *wo, *wgate, *wup, *wdown, *norm1, *norm2, *normf, *head;
    const void *head_b, *posemb;
    const int32_t *succ; /* planted successor table or NULL */
    float succ_bias;
    int32_t pad_;
} orc_model;

typedef struct {
    real *k, *v;        /* [L][max_ctx][Hkv*hd] */
    int32_t max_ctx, len;
} orc_cache;

typedef struct {
    int32_t b, gamma_cap;
    float t0, rho;       /* t0 < 0: the block test always passes (fixed window) */
    int32_t criterion;   /* 0 mean, 1 any token, 2 last token */
    int32_t mode;        /* 0 greedy, 1 sampling at temperature 1 */
    uint64_t seed;
    int32_t seq_id;
    int32_t use_posemb;  /* 1: add e_i to draft rows (the method); 0: ablation */
    int32_t scope;       /* attention context of M_B: 0 full (the method), 1 local draft, 2 local block */
    int32_t pad_;
} orc_params;

typedef struct {
    int64_t n_draft_fwd, n_mb_calls, n_target_fwd, n_steps;
    double min_margin_target;  /* min top1-top2 gap over target rows that decided a token */
    double min_margin_draft;   /* same for draft rows */
    double min_margin_stop;    /* min |statistic - t_k| over block tests that compared */
    double min_margin_accept;  /* sampling: min |log r - log(p/q)| over accept tests */
} orc_stats;

typedef struct {
    const orc_model *T, *D, *B;
    orc_cache *cT, *cD, *cB;
    orc_params prm;
    int32_t *x;          /* accepted tokens, capacity max_ctx */
    int32_t P;           /* number of accepted tokens */
    /* per-step state */
    int32_t gamma;       /* drafts so far in this step */
    int32_t k_round;     /* pre-verification rounds passed in this step */
    float t_k;           /* current threshold (fp32, repeated multiply) */
    int32_t drafting;    /* 1 while the draft loop may continue */
    int32_t *y;          /* [gamma_cap] draft tokens */
    real *qlogits;       /* [gamma_cap][V] draft logits (bias included) */
    real *hpend;         /* [gamma_cap+1][d_D] hidden states not yet given to M_B */
    int32_t *hpend_e;    /* draft index (1-based) of each pending row, 0 = history row */
    int32_t n_pend;
    real *alpha;         /* [gamma_cap] alpha_hat of the drafts of this step */
    real *plogits;       /* [gamma_cap+1][V] target logits of the last verify */
    int32_t last_n, last_next;
    int32_t mb_start;    /* M_B cache position of the first draft row of this step (scope 1) */
    const real *alpha_override; int32_t n_alpha_override, alpha_override_pos; /* test hook */
    orc_stats st;
} orc_state;

/* ---------------------------------------------------------------- weights */

static inline real wget(const void *p, int dtype, size_t i) {
    if (dtype == 0) return (real)((const float *)p)[i];
    uint32_t bits = ((uint32_t)((const uint16_t *)p)[i]) << 16;
    float f;
    memcpy(&f, &bits, 4);
    return (real)f;
}

/* y[r][o] = sum_k W[off + o*K + k] * x[r][k] */
static void linear(const orc_model *m, const void *W, size_t off, int N, int K,
                   const real *x, int n, real *y, int ldy) {
#pragma omp parallel
    {
        real *row = (real *)malloc(sizeof(real) * (size_t)K);
#pragma omp for schedule(static)
        for (int o = 0; o < N; ++o) {
            size_t base = off + (size_t)o * (size_t)K;
            for (int k = 0; k < K; ++k) row[k] = wget(W, m->wdtype, base + k);
            for (int r = 0; r < n; ++r) {
                const real *xr = x + (size_t)r * K;
                real s = 0;
                for (int k = 0; k < K; ++k) s += row[k] * xr[k];
                y[(size_t)r * ldy + o] = s;
            }
        }
        free(row);
    }
}

static void rmsnorm(const orc_model *m, const void *g, size_t goff, const real *x, int n, int d, real *y) {
    for (int r = 0; r < n; ++r) {
        real ss = 0;
        for (int i = 0; i < d; ++i) ss += x[(size_t)r * d + i] * x[(size_t)r * d + i];
        real inv = 1.0 / sqrt(ss / d + (real)m->rms_eps);
        for (int i = 0; i < d; ++i) y[(size_t)r * d + i] = x[(size_t)r * d + i] * inv * wget(g, m->wdtype, goff + i);
    }
}

/* rotate-half rotary embedding of one head vector at absolute position pos */
static void rope(real *v, int hd, int pos, real theta) {
    int half = hd / 2;
    for (int i = 0; i < half; ++i) {
        real ang = (real)pos * pow(theta, -2.0 * i / hd);
        real c = cos(ang), s = sin(ang);
        real a = v[i], b = v[i + half];
        v[i] = a * c - b * s;
        v[i + half] = b * c + a * s;
    }
}

/* ---------------------------------------------------------------- cache */

orc_cache *orc_cache_new(const orc_model *m, int max_ctx) {
    orc_cache *c = (orc_cache *)calloc(1, sizeof(orc_cache));
    size_t kvd = (size_t)m->n_kv_heads * (m->d_model / m->n_heads);
    size_t n = (size_t)m->n_layers * max_ctx * kvd;
    c->k = (real *)calloc(n, sizeof(real));
    c->v = (real *)calloc(n, sizeof(real));
    c->max_ctx = max_ctx;
    c->len = 0;
    return c;
}
void orc_cache_free(orc_cache *c) { if (c) { free(c->k); free(c->v); free(c); } }
int orc_cache_len(const orc_cache *c) { return c->len; }
void orc_cache_truncate(orc_cache *c, int len) { c->len = len; }

/* ---------------------------------------------------------------- decoder forward */

/* Runs the decoder on n new rows at positions pos0..pos0+n-1 (Eq. 2; n = 1 is one
 * step of Eq. 1).  Input rows are embeddings of `tokens`, or `x_in` [n][d] when
 * tokens is NULL (the pre-verification layer).  K and V of the new rows are
 * written to the cache at their positions and the cache length becomes pos0+n.
 * hidden_out [n][d]: output of the final RMSNorm.  logits_out [n][V]: LM head,
 * plus succ_bias on token succ[tokens[j]] of row j when a table is present. */
static void forward_from(const orc_model *m, orc_cache *c, const int32_t *tokens, const real *x_in,
                         int n, int pos0, int key_start, real *hidden_out, real *logits_out);

void orc_forward(const orc_model *m, orc_cache *c, const int32_t *tokens, const real *x_in,
                 int n, int pos0, real *hidden_out, real *logits_out) {
    forward_from(m, c, tokens, x_in, n, pos0, 0, hidden_out, logits_out);
}

/* The same forward with a restricted attention context (the "attention context"
 * ablation of the pre-verification layer): the row at position pos attends to the
 * cache positions key_start..pos; a row that lies before key_start attends to
 * itself only.  key_start = 0 is ordinary causal attention. */
void orc_forward_scoped(const orc_model *m, orc_cache *c, const int32_t *tokens, const real *x_in,
                        int n, int pos0, int key_start, real *hidden_out, real *logits_out) {
    forward_from(m, c, tokens, x_in, n, pos0, key_start, hidden_out, logits_out);
}

static void forward_from(const orc_model *m, orc_cache *c, const int32_t *tokens, const real *x_in,
                         int n, int pos0, int key_start, real *hidden_out, real *logits_out) {
    const int d = m->d_model, H = m->n_heads, Hkv = m->n_kv_heads, hd = d / H, F = m->d_ffn;
    const int kvd = Hkv * hd, qrows = (H + 2 * Hkv) * hd, group = H / Hkv;
    real *x = (real *)malloc(sizeof(real) * (size_t)n * d);
    real *a = (real *)malloc(sizeof(real) * (size_t)n * d);
    real *qkv = (real *)malloc(sizeof(real) * (size_t)n * qrows);
    real *att = (real *)malloc(sizeof(real) * (size_t)n * H * hd);
    real *o = (real *)malloc(sizeof(real) * (size_t)n * d);
    real *g = (real *)malloc(sizeof(real) * (size_t)n * F);
    real *u = (real *)malloc(sizeof(real) * (size_t)n * F);
    real *sc = (real *)malloc(sizeof(real) * (size_t)(pos0 + n));
    if (tokens) {
        for (int r = 0; r < n; ++r)
            for (int i = 0; i < d; ++i) x[(size_t)r * d + i] = wget(m->embed, m->wdtype, (size_t)tokens[r] * d + i);
    } else {
        memcpy(x, x_in, sizeof(real) * (size_t)n * d);
    }
    for (int l = 0; l < m->n_layers; ++l) {
        rmsnorm(m, m->norm1, (size_t)l * d, x, n, d, a);
        linear(m, m->wqkv, (size_t)l * qrows * d, qrows, d, a, n, qkv, qrows);
        real *ck = c->k + (size_t)l * c->max_ctx * kvd, *cv = c->v + (size_t)l * c->max_ctx * kvd;
        for (int r = 0; r < n; ++r) {
            int pos = pos0 + r;
            real *q = qkv + (size_t)r * qrows, *kk = q + H * hd, *vv = kk + kvd;
            for (int h = 0; h < H; ++h) rope(q + h * hd, hd, pos, m->rope_theta);
            for (int h = 0; h < Hkv; ++h) rope(kk + h * hd, hd, pos, m->rope_theta);
            memcpy(ck + (size_t)pos * kvd, kk, sizeof(real) * kvd);
            memcpy(cv + (size_t)pos * kvd, vv, sizeof(real) * kvd);
        }
        for (int r = 0; r < n; ++r) {
            int pos = pos0 + r;               /* causal: keys first..pos (first = 0 unless the context is restricted) */
            int first = key_start < pos ? key_start : pos;
            for (int h = 0; h < H; ++h) {
                const real *q = qkv + (size_t)r * qrows + h * hd;
                int kh = h / group;
                real mx = -INFINITY;
                for (int p = first; p <= pos; ++p) {
                    const real *kp = ck + (size_t)p * kvd + kh * hd;
                    real s = 0;
                    for (int i = 0; i < hd; ++i) s += q[i] * kp[i];
                    sc[p] = s / sqrt((real)hd);
                    if (sc[p] > mx) mx = sc[p];
                }
                real den = 0;
                for (int p = first; p <= pos; ++p) { sc[p] = exp(sc[p] - mx); den += sc[p]; }
                real *out = att + (size_t)r * H * hd + h * hd;
                for (int i = 0; i < hd; ++i) out[i] = 0;
                for (int p = first; p <= pos; ++p) {
                    const real *vp = cv + (size_t)p * kvd + kh * hd;
                    real w = sc[p] / den;
                    for (int i = 0; i < hd; ++i) out[i] += w * vp[i];
                }
            }
        }
        linear(m, m->wo, (size_t)l * d * H * hd, d, H * hd, att, n, o, d);
        for (size_t i = 0; i < (size_t)n * d; ++i) x[i] += o[i];
        rmsnorm(m, m->norm2, (size_t)l * d, x, n, d, a);
        linear(m, m->wgate, (size_t)l * F * d, F, d, a, n, g, F);
        linear(m, m->wup, (size_t)l * F * d, F, d, a, n, u, F);
        for (size_t i = 0; i < (size_t)n * F; ++i) g[i] = g[i] / (1.0 + exp(-g[i])) * u[i];
        linear(m, m->wdown, (size_t)l * d * F, d, F, g, n, o, d);
        for (size_t i = 0; i < (size_t)n * d; ++i) x[i] += o[i];
    }
    c->len = pos0 + n;
    rmsnorm(m, m->normf, 0, x, n, d, a);
    if (hidden_out) memcpy(hidden_out, a, sizeof(real) * (size_t)n * d);
    if (logits_out) {
        linear(m, m->head, 0, m->vocab, d, a, n, logits_out, m->vocab);
        if (m->succ && tokens)
            for (int r = 0; r < n; ++r) logits_out[(size_t)r * m->vocab + m->succ[tokens[r]]] += (real)m->succ_bias;
    }
    free(x); free(a); free(qkv); free(att); free(o); free(g); free(u); free(sc);
}

/* One plain matrix product y[r][o] = sum_k W[o][k] x[r][k] with the oracle's
 * weight decoding; used to check single GEMM kernels at full width. */
void orc_linear(const void *W, int wdtype, int N, int K, const real *x, int n, real *y) {
    orc_model m; memset(&m, 0, sizeof m); m.wdtype = wdtype;
    linear(&m, W, 0, N, K, x, n, y, N);
}

/* ---------------------------------------------------------------- small helpers */

static int argmax_margin(const real *v, int n, real *margin) {
    int best = 0; real b1 = v[0], b2 = -INFINITY;
    for (int i = 1; i < n; ++i) {
        if (v[i] > b1) { b2 = b1; b1 = v[i]; best = i; }   /* ties keep the lowest index */
        else if (v[i] > b2) b2 = v[i];
    }
    if (margin) *margin = b1 - b2;
    return best;
}

static real logsumexp(const real *v, int n) {
    real mx = v[0];
    for (int i = 1; i < n; ++i) if (v[i] > mx) mx = v[i];
    real s = 0;
    for (int i = 0; i < n; ++i) s += exp(v[i] - mx);
    return mx + log(s);
}

/* Philox4x32-10 (Salmon et al., "Parallel random numbers: as easy as 1, 2, 3"). */
void orc_philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2], uint32_t out[4]) {
    uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
    uint32_t k0 = key_in[0], k1 = key_in[1];
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0, p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0, n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1, n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

enum { TAG_DRAFT = 1, TAG_ACCEPT = 2, TAG_NEXT = 3 };

/* uniform in (0,1) attached to (vocabulary index, absolute position, sequence, tag) */
double orc_uniform(uint64_t seed, uint32_t v, uint32_t pos, uint32_t seq, uint32_t tag) {
    uint32_t ctr[4] = { v >> 2, pos, seq, tag }, key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) }, o[4];
    orc_philox4x32_10(ctr, key, o);
    return ((double)(o[v & 3] >> 8) + 0.5) * (1.0 / 16777216.0);
}

static real gumbel(uint64_t seed, int v, int pos, int seq, int tag) {
    return -log(-log(orc_uniform(seed, (uint32_t)v, (uint32_t)pos, (uint32_t)seq, (uint32_t)tag)));
}

/* Draw from softmax(logits) by the Gumbel-max rule; the margin is the gap
 * between the two largest perturbed logits. */
static int sample_gumbel(const real *logits, int V, uint64_t seed, int pos, int seq, int tag, real *margin) {
    int best = -1; real b1 = -INFINITY, b2 = -INFINITY;
    for (int v = 0; v < V; ++v) {
        real s = logits[v] + gumbel(seed, v, pos, seq, tag);
        if (s > b1) { b2 = b1; b1 = s; best = v; } else if (s > b2) b2 = s;
    }
    if (margin) *margin = b1 - b2;
    return best;
}

/* ---------------------------------------------------------------- acceptance (Eq. 5) */

/* Decides how many of the gamma drafts y are accepted and which token follows.
 * plog [gamma+1][V] target logits (row j is the distribution p_{j+1}), qlog
 * [gamma][V] draft logits.  pos_first = absolute position of y_1.
 * Greedy: accept while y_i equals the target's argmax; next = argmax of row n.
 * Sampling: accept while r_i <= p_i(y_i)/q_i(y_i); on a rejection next is drawn
 * from norm(max(0, p_{n+1} - q_{n+1})), else from p_{gamma+1}. */
int orc_accept_rule(const real *plog, const real *qlog, const int32_t *y, int gamma, int V,
                    int mode, uint64_t seed, int pos_first, int seq, int32_t *next_out,
                    double *margin_target, double *margin_accept) {
    int n = 0;
    double mt = INFINITY, ma = INFINITY;
    if (mode == 0) {
        for (; n < gamma; ++n) {
            real mg; int top = argmax_margin(plog + (size_t)n * V, V, &mg);
            if (mg < mt) mt = mg;
            if (top != y[n]) break;
        }
        if (n == gamma) {
            real mg; *next_out = argmax_margin(plog + (size_t)gamma * V, V, &mg);
            if (mg < mt) mt = mg;
        } else {
            *next_out = argmax_margin(plog + (size_t)n * V, V, NULL);
        }
    } else {
        for (; n < gamma; ++n) {
            const real *p = plog + (size_t)n * V, *q = qlog + (size_t)n * V;
            real lp = p[y[n]] - logsumexp(p, V), lq = q[y[n]] - logsumexp(q, V);
            real lr = log(orc_uniform(seed, 0, (uint32_t)(pos_first + n), (uint32_t)seq, TAG_ACCEPT));
            real gap = fabs(lr - (lp - lq));
            if (lp < lq && gap < ma) ma = gap;       /* alpha_i < 1: the draw matters */
            if (lr > lp - lq) break;                 /* r > p/q : reject */
        }
        if (n == gamma) {
            real mg; *next_out = sample_gumbel(plog + (size_t)gamma * V, V, seed, pos_first + gamma, seq, TAG_NEXT, &mg);
            if (mg < mt) mt = mg;
        } else {
            const real *p = plog + (size_t)n * V, *q = qlog + (size_t)n * V;
            real lsp = logsumexp(p, V), lsq = logsumexp(q, V);
            int best = -1; real b1 = -INFINITY, b2 = -INFINITY;
            for (int v = 0; v < V; ++v) {
                real res = exp(p[v] - lsp) - exp(q[v] - lsq);
                if (!(res > 0)) continue;
                real s = log(res) + gumbel(seed, v, pos_first + n, seq, TAG_NEXT);
                if (s > b1) { b2 = b1; b1 = s; best = v; } else if (s > b2) b2 = s;
            }
            if (best < 0) best = argmax_margin(p, V, NULL);  /* p == q exactly: cannot be rejected in exact arithmetic */
            if (b1 - b2 < mt) mt = b1 - b2;
            *next_out = best;
        }
    }
    if (margin_target) *margin_target = mt;
    if (margin_accept) *margin_accept = ma;
    return n;
}

/* ---------------------------------------------------------------- loop state */

static void stats_reset(orc_stats *s) {
    memset(s, 0, sizeof *s);
    s->min_margin_target = s->min_margin_draft = s->min_margin_stop = s->min_margin_accept = INFINITY;
}

orc_state *orc_new(const orc_model *T, const orc_model *D, const orc_model *B, int max_ctx, const orc_params *prm) {
    orc_state *s = (orc_state *)calloc(1, sizeof(orc_state));
    s->T = T; s->D = D; s->B = B; s->prm = *prm;
    s->cT = orc_cache_new(T, max_ctx);
    s->cD = orc_cache_new(D, max_ctx);
    if (B) s->cB = orc_cache_new(B, max_ctx);
    s->x = (int32_t *)calloc(max_ctx, sizeof(int32_t));
    int gc = prm->gamma_cap, V = T->vocab, dD = D->d_model;
    s->y = (int32_t *)calloc(gc, sizeof(int32_t));
    s->qlogits = (real *)calloc((size_t)gc * V, sizeof(real));
    s->hpend = (real *)calloc((size_t)(gc + 1) * dD, sizeof(real));
    s->hpend_e = (int32_t *)calloc(gc + 1, sizeof(int32_t));
    s->alpha = (real *)calloc(gc, sizeof(real));
    s->plogits = (real *)calloc((size_t)(gc + 1) * V, sizeof(real));
    stats_reset(&s->st);
    return s;
}

void orc_free(orc_state *s) {
    if (!s) return;
    orc_cache_free(s->cT); orc_cache_free(s->cD); orc_cache_free(s->cB);
    free(s->x); free(s->y); free(s->qlogits); free(s->hpend); free(s->hpend_e); free(s->alpha); free(s->plogits);
    free(s);
}

static void step_reset(orc_state *s) {
    s->gamma = 0; s->k_round = 0; s->t_k = s->prm.t0; s->drafting = 1; s->n_pend = 0;
}

/* Fills the three caches with prompt tokens 0..n-2; the last prompt token is the
 * first step's input row.  M_B sees the draft's hidden states of those rows
 * without position embedding (they are accepted history, h_x in Eq. 7). */
void orc_prefill(orc_state *s, const int32_t *prompt, int n_prompt) {
    memcpy(s->x, prompt, sizeof(int32_t) * n_prompt);
    s->P = n_prompt;
    int m = n_prompt - 1;
    s->cT->len = s->cD->len = 0; if (s->cB) s->cB->len = 0;
    if (m > 0) {
        orc_forward(s->T, s->cT, prompt, NULL, m, 0, NULL, NULL);
        real *h = (real *)malloc(sizeof(real) * (size_t)m * s->D->d_model);
        orc_forward(s->D, s->cD, prompt, NULL, m, 0, h, NULL);
        if (s->B) orc_forward(s->B, s->cB, NULL, h, m, 0, NULL, NULL);
        free(h);
    }
    step_reset(s);
    stats_reset(&s->st);
}

/* Eq. 6: b autoregressive draft forwards.  The i-th forward of the step takes
 * y_{i-1} (the last accepted token for i = 1) and emits y_i, q_i and h_i.  When
 * the draft cache is one row short (previous step fully accepted) the first
 * forward takes two rows; its first row is history for M_B. */
void orc_draft_block(orc_state *s) {
    const orc_model *D = s->D;
    const int V = D->vocab, d = D->d_model;
    real *hid = (real *)malloc(sizeof(real) * 2 * d), *lg = (real *)malloc(sizeof(real) * 2 * (size_t)V);
    for (int j = 0; j < s->prm.b; ++j) {
        int32_t in[2]; int n_in, pos0 = s->cD->len;
        if (s->gamma == 0) {                       /* first forward of the step */
            int missing = (s->P - 1) - s->cD->len; /* 0 normally, 1 after a fully accepted step */
            n_in = missing + 1;
            for (int r = 0; r < n_in; ++r) in[r] = s->x[pos0 + r];
        } else { n_in = 1; in[0] = s->y[s->gamma - 1]; }
        orc_forward(D, s->cD, in, NULL, n_in, pos0, hid, lg);
        s->st.n_draft_fwd += 1;
        const real *lrow = lg + (size_t)(n_in - 1) * V;
        real mg; int tok;
        int pos_tok = s->P + s->gamma;            /* absolute position of the token being drafted */
        if (s->prm.mode == 0) tok = argmax_margin(lrow, V, &mg);
        else tok = sample_gumbel(lrow, V, s->prm.seed, pos_tok, s->prm.seq_id, TAG_DRAFT, &mg);
        if (mg < s->st.min_margin_draft) s->st.min_margin_draft = mg;
        memcpy(s->qlogits + (size_t)s->gamma * V, lrow, sizeof(real) * V);
        for (int r = 0; r < n_in; ++r) {
            memcpy(s->hpend + (size_t)s->n_pend * d, hid + (size_t)r * d, sizeof(real) * d);
            s->hpend_e[s->n_pend] = (r == n_in - 1) ? s->gamma + 1 : 0;
            s->n_pend += 1;
        }
        s->y[s->gamma] = tok;
        s->gamma += 1;
    }
    free(hid); free(lg);
}

/* Eq. 7 + the stop test of Algorithm 1.  Runs M_B on the rows the draft has
 * produced since the last call, with e_i added to draft rows, against M_B's own
 * KV cache; then decides whether drafting continues.  Returns the block
 * statistic that was compared (or would have been). */
double orc_preverify(orc_state *s) {
    const orc_model *B = s->B;
    const int d = B->d_model, n = s->n_pend, b = s->prm.b;
    real *xin = (real *)malloc(sizeof(real) * (size_t)n * d), *hid = (real *)malloc(sizeof(real) * (size_t)n * d);
    for (int r = 0; r < n; ++r) {
        int e = s->hpend_e[r];
        for (int i = 0; i < d; ++i) {
            real v = s->hpend[(size_t)r * d + i];
            if (e > 0 && s->prm.use_posemb) v += wget(B->posemb, B->wdtype, (size_t)(e - 1) * d + i);
            xin[(size_t)r * d + i] = v;
        }
    }
    /* attention context (Section 5, "attention context" ablation): full = the whole cache (the method);
     * local draft = the drafts of this step; local block = the drafts of this block.  History rows
     * (a catch-up row comes first in the step's first call) are never part of a restricted context. */
    int n_hist = 0;
    while (n_hist < n && s->hpend_e[n_hist] == 0) n_hist += 1;
    if (s->gamma == b) s->mb_start = s->cB->len + n_hist;      /* first call of the step */
    int key_start = s->prm.scope == 2 ? s->cB->len + n_hist : s->prm.scope == 1 ? s->mb_start : 0;
    forward_from(B, s->cB, NULL, xin, n, s->cB->len, key_start, hid, NULL);
    s->st.n_mb_calls += 1;
    for (int r = 0; r < n; ++r) {
        int e = s->hpend_e[r];
        if (e == 0) continue;
        real z[2];
        linear(B, B->head_b, 0, 2, d, hid + (size_t)r * d, 1, z, 2);
        real a = 1.0 / (1.0 + exp(z[0] - z[1]));          /* softmax(z)[1] */
        if (s->alpha_override && s->alpha_override_pos < s->n_alpha_override) a = s->alpha_override[s->alpha_override_pos++];
        s->alpha[e - 1] = a;
    }
    s->n_pend = 0;
    /* block statistic over the b newest drafts */
    real stat;
    const real *ab = s->alpha + (s->gamma - b);
    if (s->prm.criterion == 1) { stat = ab[0]; for (int i = 1; i < b; ++i) if (ab[i] < stat) stat = ab[i]; }
    else if (s->prm.criterion == 2) stat = ab[b - 1];
    else { stat = 0; for (int i = 0; i < b; ++i) stat += ab[i]; stat /= b; }
    int stop = 0;
    if (s->prm.t0 >= 0) {
        real gap = fabs(stat - (real)s->t_k);
        if (gap < s->st.min_margin_stop) s->st.min_margin_stop = gap;
        if (stat <= (real)s->t_k) stop = 1;
    }
    if (s->gamma + b > s->prm.gamma_cap) stop = 1;
    if (stop) s->drafting = 0;
    else { s->t_k = s->t_k * s->prm.rho; s->k_round += 1; }
    free(xin); free(hid);
    return stat;
}

/* Eq. 4: one target forward over [last accepted token, y_1..y_gamma]. */
void orc_verify(orc_state *s) {
    int n = s->gamma + 1;
    int32_t *in = (int32_t *)malloc(sizeof(int32_t) * n);
    in[0] = s->x[s->P - 1];
    for (int i = 0; i < s->gamma; ++i) in[i + 1] = s->y[i];
    orc_forward(s->T, s->cT, in, NULL, n, s->P - 1, NULL, s->plogits);
    s->st.n_target_fwd += 1;
    free(in);
}

/* Acceptance (Eq. 5), commit of [y_1..y_n, next], rollback of the three caches. */
int orc_accept(orc_state *s) {
    double mt, ma; int32_t next;
    int gamma = s->gamma;
    int n = orc_accept_rule(s->plogits, s->qlogits, s->y, gamma, s->T->vocab, s->prm.mode, s->prm.seed,
                            s->P, s->prm.seq_id, &next, &mt, &ma);
    if (mt < s->st.min_margin_target) s->st.min_margin_target = mt;
    if (ma < s->st.min_margin_accept) s->st.min_margin_accept = ma;
    int P = s->P;
    for (int i = 0; i < n; ++i) s->x[P + i] = s->y[i];
    s->x[P + n] = next;
    s->P = P + n + 1;
    s->cT->len = P + n;                                   /* rows P-1 .. P-1+n stay */
    int keepD = P - 1 + (n + 1 < gamma ? n + 1 : gamma);  /* the draft never saw y_gamma */
    s->cD->len = keepD;
    if (s->cB) s->cB->len = keepD;
    s->last_n = n; s->last_next = next;
    s->st.n_steps += 1;
    step_reset(s);
    return n;
}

/* ---------------------------------------------------------------- whole loops */

/* Algorithm 1.  Returns the number of draft-and-verify steps; out_tokens gets the
 * first max_new generated tokens; draft_len/accept_len [max_new] get gamma and n
 * of every step (untruncated). */
int orc_generate_pacer(orc_state *s, const int32_t *prompt, int n_prompt, int max_new,
                       int32_t *out_tokens, int32_t *draft_len, int32_t *accept_len, orc_stats *stats) {
    orc_prefill(s, prompt, n_prompt);
    int steps = 0;
    while (s->P - n_prompt < max_new) {
        while (s->drafting) {
            orc_draft_block(s);
            orc_preverify(s);
        }
        orc_verify(s);
        int gamma = s->gamma;
        int n = orc_accept(s);
        draft_len[steps] = gamma; accept_len[steps] = n;
        steps += 1;
    }
    for (int i = 0; i < max_new; ++i) out_tokens[i] = s->x[n_prompt + i];
    if (stats) *stats = s->st;
    return steps;
}

/* Section 2.2: speculative decoding with a fixed window gamma.  Written on its
 * own (no block loop, no pre-verification layer) so that Algorithm 1 with a test
 * that always passes can be compared against it. */
int orc_generate_sd(const orc_model *T, const orc_model *D, const int32_t *prompt, int n_prompt, int max_new,
                    int gamma, int mode, uint64_t seed, int seq, int max_ctx,
                    int32_t *out_tokens, int32_t *draft_len, int32_t *accept_len, orc_stats *stats) {
    const int V = T->vocab;
    orc_cache *cT = orc_cache_new(T, max_ctx), *cD = orc_cache_new(D, max_ctx);
    int32_t *x = (int32_t *)calloc(max_ctx, sizeof(int32_t)), *y = (int32_t *)calloc(gamma, sizeof(int32_t));
    int32_t *in = (int32_t *)calloc(gamma + 1, sizeof(int32_t));
    real *ql = (real *)malloc(sizeof(real) * (size_t)gamma * V), *pl = (real *)malloc(sizeof(real) * (size_t)(gamma + 1) * V);
    real *lg = (real *)malloc(sizeof(real) * 2 * (size_t)V);
    orc_stats st; stats_reset(&st);
    memcpy(x, prompt, sizeof(int32_t) * n_prompt);
    int P = n_prompt, steps = 0;
    if (P > 1) { orc_forward(T, cT, x, NULL, P - 1, 0, NULL, NULL); orc_forward(D, cD, x, NULL, P - 1, 0, NULL, NULL); }
    while (P - n_prompt < max_new) {
        for (int i = 0; i < gamma; ++i) {
            int pos0 = cD->len, n_in = (i == 0) ? (P - pos0) : 1;   /* 1 row, or 2 when catching up */
            const int32_t *src = (i == 0) ? (x + pos0) : (y + i - 1);
            orc_forward(D, cD, src, NULL, n_in, pos0, NULL, lg);
            st.n_draft_fwd += 1;
            const real *lrow = lg + (size_t)(n_in - 1) * V;
            real mg;
            y[i] = (mode == 0) ? argmax_margin(lrow, V, &mg) : sample_gumbel(lrow, V, seed, P + i, seq, TAG_DRAFT, &mg);
            if (mg < st.min_margin_draft) st.min_margin_draft = mg;
            memcpy(ql + (size_t)i * V, lrow, sizeof(real) * V);
        }
        in[0] = x[P - 1];
        for (int i = 0; i < gamma; ++i) in[i + 1] = y[i];
        orc_forward(T, cT, in, NULL, gamma + 1, P - 1, NULL, pl);
        st.n_target_fwd += 1;
        int32_t next; double mt, ma;
        int n = orc_accept_rule(pl, ql, y, gamma, V, mode, seed, P, seq, &next, &mt, &ma);
        if (mt < st.min_margin_target) st.min_margin_target = mt;
        if (ma < st.min_margin_accept) st.min_margin_accept = ma;
        for (int i = 0; i < n; ++i) x[P + i] = y[i];
        x[P + n] = next;
        cT->len = P + n;
        cD->len = (n < gamma) ? P + n : P + gamma - 1;
        P += n + 1;
        draft_len[steps] = gamma; accept_len[steps] = n;
        steps += 1; st.n_steps += 1;
    }
    for (int i = 0; i < max_new; ++i) out_tokens[i] = x[n_prompt + i];
    if (stats) *stats = st;
    orc_cache_free(cT); orc_cache_free(cD); free(x); free(y); free(in); free(ql); free(pl); free(lg);
    return steps;
}

/* Speculative decoding (Section 2.2) whose window is prescribed per step: step s
 * drafts windows[s] tokens (0 = a plain target step), steps past n_windows reuse
 * the last entry.  With windows[s] = the accepted length L_A* of step s of a
 * large-window run this is decoding with the optimal draft length gamma* of
 * Section 3.1 (every draft is accepted, no forward is wasted).  The draft model
 * catches up on the rows it has not seen (one forward) when it next drafts. */
int orc_generate_sched(const orc_model *T, const orc_model *D, const int32_t *prompt, int n_prompt, int max_new,
                       const int32_t *windows, int n_windows, int mode, uint64_t seed, int seq, int max_ctx,
                       int32_t *out_tokens, int32_t *draft_len, int32_t *accept_len, orc_stats *stats) {
    const int V = T->vocab;
    int gmax = 1;
    for (int i = 0; i < n_windows; ++i) if (windows[i] > gmax) gmax = windows[i];
    orc_cache *cT = orc_cache_new(T, max_ctx), *cD = orc_cache_new(D, max_ctx);
    int32_t *x = (int32_t *)calloc(max_ctx, sizeof(int32_t)), *y = (int32_t *)calloc(gmax, sizeof(int32_t));
    int32_t *in = (int32_t *)calloc(gmax + 1, sizeof(int32_t));
    real *ql = (real *)malloc(sizeof(real) * (size_t)gmax * V), *pl = (real *)malloc(sizeof(real) * (size_t)(gmax + 1) * V);
    orc_stats st; stats_reset(&st);
    memcpy(x, prompt, sizeof(int32_t) * n_prompt);
    int P = n_prompt, steps = 0;
    if (P > 1) { orc_forward(T, cT, x, NULL, P - 1, 0, NULL, NULL); orc_forward(D, cD, x, NULL, P - 1, 0, NULL, NULL); }
    while (P - n_prompt < max_new) {
        const int gamma = windows[steps < n_windows ? steps : n_windows - 1];
        for (int i = 0; i < gamma; ++i) {
            int pos0 = cD->len, n_in = (i == 0) ? (P - pos0) : 1;   /* all rows the draft has not seen yet */
            const int32_t *src = (i == 0) ? (x + pos0) : (y + i - 1);
            real *lg = (real *)malloc(sizeof(real) * (size_t)n_in * V);
            orc_forward(D, cD, src, NULL, n_in, pos0, NULL, lg);
            st.n_draft_fwd += 1;
            const real *lrow = lg + (size_t)(n_in - 1) * V;
            real mg;
            y[i] = (mode == 0) ? argmax_margin(lrow, V, &mg) : sample_gumbel(lrow, V, seed, P + i, seq, TAG_DRAFT, &mg);
            if (mg < st.min_margin_draft) st.min_margin_draft = mg;
            memcpy(ql + (size_t)i * V, lrow, sizeof(real) * V);
            free(lg);
        }
        in[0] = x[P - 1];
        for (int i = 0; i < gamma; ++i) in[i + 1] = y[i];
        orc_forward(T, cT, in, NULL, gamma + 1, P - 1, NULL, pl);
        st.n_target_fwd += 1;
        int32_t next; double mt, ma;
        int n = orc_accept_rule(pl, ql, y, gamma, V, mode, seed, P, seq, &next, &mt, &ma);
        if (mt < st.min_margin_target) st.min_margin_target = mt;
        if (ma < st.min_margin_accept) st.min_margin_accept = ma;
        for (int i = 0; i < n; ++i) x[P + i] = y[i];
        x[P + n] = next;
        cT->len = P + n;
        if (gamma > 0) cD->len = (n < gamma) ? P + n : P + gamma - 1;   /* a step without drafts leaves the draft cache alone */
        P += n + 1;
        draft_len[steps] = gamma; accept_len[steps] = n;
        steps += 1; st.n_steps += 1;
    }
    for (int i = 0; i < max_new; ++i) out_tokens[i] = x[n_prompt + i];
    if (stats) *stats = st;
    orc_cache_free(cT); orc_cache_free(cD); free(x); free(y); free(in); free(ql); free(pl);
    return steps;
}

/* Eq. 1 on the target alone: max_new sequential forwards.  Greedy output is the
 * sequence every lossless speculative variant must reproduce. */
void orc_generate_ar(const orc_model *T, const int32_t *prompt, int n_prompt, int max_new, int mode,
                     uint64_t seed, int seq, int max_ctx, int32_t *out_tokens, double *min_margin) {
    const int V = T->vocab;
    orc_cache *c = orc_cache_new(T, max_ctx);
    real *lg = (real *)malloc(sizeof(real) * (size_t)V);
    double mm = INFINITY;
    if (n_prompt > 1) orc_forward(T, c, prompt, NULL, n_prompt - 1, 0, NULL, NULL);
    int32_t tok = prompt[n_prompt - 1];
    for (int i = 0; i < max_new; ++i) {
        orc_forward(T, c, &tok, NULL, 1, n_prompt - 1 + i, NULL, lg);
        real mg;
        tok = (mode == 0) ? argmax_margin(lg, V, &mg) : sample_gumbel(lg, V, seed, n_prompt + i, seq, TAG_NEXT, &mg);
        if (mg < mm) mm = mg;
        out_tokens[i] = tok;
    }
    if (min_margin) *min_margin = mm;
    orc_cache_free(c); free(lg);
}

/* ---------------------------------------------------------------- accessors for the tests */

int orc_get_P(const orc_state *s) { return s->P; }
int orc_get_gamma(const orc_state *s) { return s->gamma; }
int orc_get_drafting(const orc_state *s) { return s->drafting; }
float orc_get_t_k(const orc_state *s) { return s->t_k; }
int orc_get_last_n(const orc_state *s) { return s->last_n; }
int orc_get_last_next(const orc_state *s) { return s->last_next; }
int orc_get_len(const orc_state *s, int which) { return which == 0 ? s->cT->len : which == 1 ? s->cD->len : s->cB->len; }
const int32_t *orc_get_x(const orc_state *s) { return s->x; }
const int32_t *orc_get_y(const orc_state *s) { return s->y; }
const real *orc_get_alpha(const orc_state *s) { return s->alpha; }
const real *orc_get_plogits(const orc_state *s) { return s->plogits; }
const real *orc_get_qlogits(const orc_state *s) { return s->qlogits; }
const real *orc_get_hpend(const orc_state *s) { return s->hpend; }
int orc_get_n_pend(const orc_state *s) { return s->n_pend; }
void orc_get_stats(const orc_state *s, orc_stats *out) { *out = s->st; }
void orc_set_seed(orc_state *s, uint64_t seed, int seq_id) { s->prm.seed = seed; s->prm.seq_id = seq_id; }
void orc_set_alpha_override(orc_state *s, const real *a, int n) { s->alpha_override = a; s->n_alpha_override = n; s->alpha_override_pos = 0; }
orc_cache *orc_get_cache(orc_state *s, int which) { return which == 0 ? s->cT : which == 1 ? s->cD : s->cB; }
const real *orc_cache_k(const orc_cache *c) { return c->k; }
const real *orc_cache_v(const orc_cache *c) { return c->v; }
