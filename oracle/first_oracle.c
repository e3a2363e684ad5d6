/*
 * first_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, host-only statement of the FiRST routed decoder (arXiv 2410.12513):
 * per-layer routers score the prompt, a per-sequence layer-skip mask is fixed, and
 * every decode step applies a transformer layer only to the sequences that keep it.
 * It exists so that the CUDA library can be checked against something written
 * straight from the paper.  It shares no source, header, table or helper with the
 * CUDA tree; nothing in the product path may call it.
 *
 * Arithmetic: every tensor is held in IEEE float32 (the paper runs "full precision",
 * App. "Training and Inference Setup"); every reduction (dot products, norms,
 * softmax sums, router means) is accumulated in float64 and rounded to float32 once,
 * so the oracle's own rounding is far below the tolerances it is used to judge.
 * Weight matrices may be handed in as float32 or as bfloat16 bit patterns (uint16,
 * the upper half of the float32 word); bfloat16 values are widened exactly.
 * The KV cache has a storage format too (kv_dtype): float32, or bfloat16, in which case a
 * key/value is rounded to bfloat16 once, when it enters the cache, and attention reads the
 * rounded value -- the same contract as for weights: both sides agree on the stored values,
 * all arithmetic on them stays float32/float64.
 *
 * What follows the paper, and where:
 *   - layer recursion  H_i = H_{i-1} + phi_i(H^1..H^j)             Eq. 1 (Problem Statement)
 *   - skip recursion   H_i = H_k            if phi_i not selected   Eq. 3 (Proposed Solution)
 *   - inference rule   H_i = H_{i-1} + round(rho_i) * phi_i(..)     Sec. "Proposed Solution", unnumbered
 *     with round(rho) = 1 iff rho >= 0.5
 *   - router: bias-free linear D->1, per-token sigmoid, mean over   Sec. "Adaptive Router Module"
 *     the sequence's tokens
 *   - no skipping during prefill; decisions fixed for all decode    Sec. "Inference for FiRST", items 1-2
 *     steps; kept layers see the K/V of every earlier token
 * The paper names the LLaMA family but not the block's internals; phi_i is the
 * public LLaMA block: RMSNorm -> q,k,v projections -> rotary embedding (half-split
 * pairing) -> causal softmax attention with grouped KV heads -> output projection
 * -> residual; RMSNorm -> SwiGLU feed-forward -> residual.  No linear biases.
 *
 * Pins (tests/test_oracle_*.py): Hugging Face LlamaForCausalLM on the same random
 * weights (all-keep special case), hand-computed router values, the closed form for
 * an all-skip mask, bit-identity of skipped rows and their caches, cached decode
 * against the cache-free recompute below, batch-permutation invariance, and the
 * router parameter fraction the paper prints.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define FO_OK 0
#define FO_E_ARG (-1)
#define FO_E_CAPACITY (-2)
#define FO_E_ALLOC (-3)

typedef struct {
    int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, ffn_dim, vocab;
    int32_t weight_dtype; /* 0 = float32, 1 = bfloat16 bit patterns (uint16) */
    double rope_base, rms_eps;
    int32_t kv_dtype;     /* storage format of cached keys/values: 0 = float32, 1 = values rounded to
                             bfloat16 (nearest even) when stored, still held in float32 words */
} fo_model;

typedef struct {
    const void *embed;   /* [V][D] */
    const void *lm_head; /* [V][D] */
    const float *final_norm;       /* [D] */
    const float *const *attn_norm; /* L x [D] */
    const float *const *ffn_norm;  /* L x [D] */
    const void *const *wq;         /* L x [Hq*hd][D]  */
    const void *const *wk;         /* L x [Hkv*hd][D] */
    const void *const *wv;         /* L x [Hkv*hd][D] */
    const void *const *wo;         /* L x [D][Hq*hd]  */
    const void *const *wg;         /* L x [F][D] */
    const void *const *wu;         /* L x [F][D] */
    const void *const *wd;         /* L x [D][F] */
} fo_weights;

/* Host KV cache, float32, token-major: layer l, sequence b, token t lives at row
 * slab_off[b] + t of k[l] / v[l]; a row is [Hkv][hd]. */
typedef struct {
    float *const *k;
    float *const *v;
    const int64_t *slab_off; /* [B] */
    const int32_t *slab_cap; /* [B] */
    int32_t *len;            /* [L][B] tokens present */
    int32_t *pos;            /* [B] absolute index of the next token */
} fo_kv;

/* float32 -> nearest bfloat16 (ties to even), returned widened back to float32 */
static inline float bf16_round(float f) {
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7f800000u) == 0x7f800000u) return f; /* inf / nan unchanged */
    u += 0x7fffu + ((u >> 16) & 1u);
    u &= 0xffff0000u;
    memcpy(&f, &u, sizeof f);
    return f;
}

static void store_round(float *v, size_t n, int kv_dtype) {
    if (kv_dtype == 1)
        for (size_t i = 0; i < n; ++i) v[i] = bf16_round(v[i]);
}

static inline float bf16_widen(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* one weight row (length K) dotted with x, float64 accumulation */
static double row_dot(const void *w, int dtype, size_t row, int K, const float *x) {
    double acc = 0.0;
    if (dtype == 0) {
        const float *p = (const float *)w + row * (size_t)K;
#pragma omp simd reduction(+ : acc)
        for (int k = 0; k < K; ++k) acc += (double)p[k] * (double)x[k];
    } else {
        const uint16_t *p = (const uint16_t *)w + row * (size_t)K;
#pragma omp simd reduction(+ : acc)
        for (int k = 0; k < K; ++k) acc += (double)bf16_widen(p[k]) * (double)x[k];
    }
    return acc;
}

/* Y[r][o] = sum_k W[o][k] X[r][k]  for r < R (rows have strides ldx, ldy) */
static void linear(const void *w, int dtype, int out, int in, const float *X, size_t ldx, float *Y,
                   size_t ldy, int R) {
#pragma omp parallel for schedule(static)
    for (int o = 0; o < out; ++o)
        for (int r = 0; r < R; ++r) Y[(size_t)r * ldy + o] = (float)row_dot(w, dtype, (size_t)o, in, X + (size_t)r * ldx);
}

static void load_row(const void *w, int dtype, size_t row, int K, float *dst) {
    if (dtype == 0)
        memcpy(dst, (const float *)w + row * (size_t)K, (size_t)K * sizeof(float));
    else {
        const uint16_t *p = (const uint16_t *)w + row * (size_t)K;
        for (int k = 0; k < K; ++k) dst[k] = bf16_widen(p[k]);
    }
}

/* y = x / sqrt(mean(x^2) + eps) * gain */
static void rmsnorm(const float *x, const float *gain, int D, double eps, float *y) {
    double ss = 0.0;
    for (int i = 0; i < D; ++i) ss += (double)x[i] * (double)x[i];
    double inv = 1.0 / sqrt(ss / (double)D + eps);
    for (int i = 0; i < D; ++i) y[i] = (float)((double)x[i] * inv * (double)gain[i]);
}

/* rotary embedding, half-split pairing (i, i + hd/2), angle = pos * base^(-2i/hd) */
static void rope(float *vec, int n_heads, int hd, int pos, double base) {
    int half = hd / 2;
    for (int h = 0; h < n_heads; ++h) {
        float *p = vec + (size_t)h * hd;
        for (int i = 0; i < half; ++i) {
            double ang = (double)pos * pow(base, -2.0 * (double)i / (double)hd);
            double c = cos(ang), s = sin(ang);
            double a = p[i], b = p[i + half];
            p[i] = (float)(a * c - b * s);
            p[i + half] = (float)(b * c + a * s);
        }
    }
}

/* softmax attention of one query token over T cached tokens (rows of Kc/Vc are
 * [Hkv][hd]); query head h reads KV head h / (Hq/Hkv). */
static void attend(const fo_model *m, const float *q, const float *Kc, const float *Vc, int T, float *out,
                   double *score) {
    int Hq = m->n_q_heads, Hkv = m->n_kv_heads, hd = m->head_dim, grp = Hq / Hkv;
    size_t row = (size_t)Hkv * hd;
    double scale = 1.0 / sqrt((double)hd);
    for (int h = 0; h < Hq; ++h) {
        int g = h / grp;
        const float *qh = q + (size_t)h * hd;
        double mx = -INFINITY;
        for (int t = 0; t < T; ++t) {
            const float *kr = Kc + (size_t)t * row + (size_t)g * hd;
            double s = 0.0;
            for (int d = 0; d < hd; ++d) s += (double)qh[d] * (double)kr[d];
            s *= scale;
            score[t] = s;
            if (s > mx) mx = s;
        }
        double den = 0.0;
        for (int t = 0; t < T; ++t) {
            score[t] = exp(score[t] - mx);
            den += score[t];
        }
        for (int d = 0; d < hd; ++d) {
            double acc = 0.0;
            for (int t = 0; t < T; ++t) acc += score[t] * (double)Vc[(size_t)t * row + (size_t)g * hd + d];
            out[(size_t)h * hd + d] = (float)(acc / den);
        }
    }
}

static void swiglu_ffn(const fo_model *m, const fo_weights *w, int l, const float *u, int R, float *gate,
                       float *up, float *down) {
    int D = m->d_model, F = m->ffn_dim, dt = m->weight_dtype;
    linear(w->wg[l], dt, F, D, u, (size_t)D, gate, (size_t)F, R);
    linear(w->wu[l], dt, F, D, u, (size_t)D, up, (size_t)F, R);
    for (size_t i = 0; i < (size_t)R * F; ++i) {
        double g = gate[i];
        gate[i] = (float)(g / (1.0 + exp(-g)) * (double)up[i]);
    }
    linear(w->wd[l], dt, D, F, gate, (size_t)F, down, (size_t)D, R);
}

/* ---------------------------------------------------------------------------------
 * Router (Sec. "Adaptive Router Module"; rounding rule of Sec. "Proposed Solution").
 * z_j = w . hidden[j] (+ bias if given).
 *   mode 0 (the paper's order): rho = mean_j sigmoid(z_j)
 *   mode 1 (pooled variant)   : rho = sigmoid(mean_j z_j)
 * keep = (rho >= tau); the paper's tau is 0.5 and equality keeps the layer.
 * -------------------------------------------------------------------------------*/
int fo_route(const float *hidden, int32_t n, int32_t D, const float *w, const float *bias, double tau,
             int32_t mode, double *rho_out, uint8_t *keep_out) {
    if (!hidden || !w || n <= 0 || D <= 0 || (mode != 0 && mode != 1)) return FO_E_ARG;
    double sum = 0.0;
    for (int j = 0; j < n; ++j) {
        double z = bias ? (double)bias[0] : 0.0;
        const float *h = hidden + (size_t)j * D;
        for (int d = 0; d < D; ++d) z += (double)w[d] * (double)h[d];
        sum += (mode == 0) ? 1.0 / (1.0 + exp(-z)) : z;
    }
    double mean = sum / (double)n;
    double rho = (mode == 0) ? mean : 1.0 / (1.0 + exp(-mean));
    if (rho_out) *rho_out = rho;
    if (keep_out) *keep_out = (uint8_t)(rho >= tau ? 1 : 0);
    return FO_OK;
}

/* ---------------------------------------------------------------------------------
 * One routed decode step for a batch (inference rule; "Inference for FiRST" item 2).
 * For sequence b and layer l: mask[b][l] == 0 leaves the residual row, the cache
 * rows and len[l][b] untouched; otherwise the new token's k,v are appended at row
 * len[l][b] and x_b += phi_l(x_b | cache).  The rotary position is pos[b], the
 * absolute index of the token, whatever was skipped.  Afterwards pos[b] += 1.
 * layer_inputs (optional, [L][B][D]) receives the residual entering each layer --
 * what router l reads when the step is used to prefill token by token.
 * -------------------------------------------------------------------------------*/
int fo_decode_step(const fo_model *m, const fo_weights *w, int32_t B, const int32_t *tokens,
                   const uint8_t *mask, fo_kv *kv, float *logits, float *layer_inputs) {
    if (!m || !w || !tokens || !mask || !kv || B <= 0) return FO_E_ARG;
    int L = m->n_layers, D = m->d_model, Hq = m->n_q_heads, Hkv = m->n_kv_heads, hd = m->head_dim;
    int F = m->ffn_dim, V = m->vocab, dt = m->weight_dtype;
    size_t qd = (size_t)Hq * hd, kvd = (size_t)Hkv * hd;
    for (int b = 0; b < B; ++b) {
        if (tokens[b] < 0 || tokens[b] >= V) return FO_E_ARG;
        for (int l = 0; l < L; ++l) {
            if (mask[(size_t)b * L + l] > 1) return FO_E_ARG;
            if (mask[(size_t)b * L + l] && kv->len[(size_t)l * B + b] >= kv->slab_cap[b]) return FO_E_CAPACITY;
        }
    }
    int maxT = 0;
    for (int b = 0; b < B; ++b)
        if (kv->slab_cap[b] > maxT) maxT = kv->slab_cap[b];
    float *x = malloc((size_t)B * D * sizeof(float));
    float *xn = malloc((size_t)D * sizeof(float));
    float *q = malloc(qd * sizeof(float));
    float *att = malloc(qd * sizeof(float));
    float *proj = malloc((size_t)D * sizeof(float));
    float *gate = malloc((size_t)F * sizeof(float));
    float *up = malloc((size_t)F * sizeof(float));
    double *score = malloc((size_t)(maxT + 1) * sizeof(double));
    if (!x || !xn || !q || !att || !proj || !gate || !up || !score) return FO_E_ALLOC;

    for (int b = 0; b < B; ++b) load_row(w->embed, dt, (size_t)tokens[b], D, x + (size_t)b * D);

    for (int l = 0; l < L; ++l) {
        if (layer_inputs) memcpy(layer_inputs + (size_t)l * B * D, x, (size_t)B * D * sizeof(float));
        for (int b = 0; b < B; ++b) {
            if (!mask[(size_t)b * L + l]) continue; /* skipped: identity on the residual */
            float *xb = x + (size_t)b * D;
            int T = kv->len[(size_t)l * B + b];
            float *Kc = kv->k[l] + (size_t)kv->slab_off[b] * kvd;
            float *Vc = kv->v[l] + (size_t)kv->slab_off[b] * kvd;
            rmsnorm(xb, w->attn_norm[l], D, m->rms_eps, xn);
            linear(w->wq[l], dt, (int)qd, D, xn, (size_t)D, q, qd, 1);
            linear(w->wk[l], dt, (int)kvd, D, xn, (size_t)D, Kc + (size_t)T * kvd, kvd, 1);
            linear(w->wv[l], dt, (int)kvd, D, xn, (size_t)D, Vc + (size_t)T * kvd, kvd, 1);
            rope(q, Hq, hd, kv->pos[b], m->rope_base);
            rope(Kc + (size_t)T * kvd, Hkv, hd, kv->pos[b], m->rope_base);
            store_round(Kc + (size_t)T * kvd, kvd, m->kv_dtype); /* the cache's storage format */
            store_round(Vc + (size_t)T * kvd, kvd, m->kv_dtype);
            kv->len[(size_t)l * B + b] = T + 1;
            attend(m, q, Kc, Vc, T + 1, att, score);
            linear(w->wo[l], dt, D, (int)qd, att, qd, proj, (size_t)D, 1);
            for (int d = 0; d < D; ++d) xb[d] += proj[d];
            rmsnorm(xb, w->ffn_norm[l], D, m->rms_eps, xn);
            swiglu_ffn(m, w, l, xn, 1, gate, up, proj);
            for (int d = 0; d < D; ++d) xb[d] += proj[d];
        }
    }
    if (logits) {
        for (int b = 0; b < B; ++b) {
            rmsnorm(x + (size_t)b * D, w->final_norm, D, m->rms_eps, x + (size_t)b * D);
        }
        linear(w->lm_head, dt, V, D, x, (size_t)D, logits, (size_t)V, B);
    }
    for (int b = 0; b < B; ++b) kv->pos[b] += 1;
    free(x); free(xn); free(q); free(att); free(proj); free(gate); free(up); free(score);
    return FO_OK;
}

/* ---------------------------------------------------------------------------------
 * Cache-free forward of one sequence of n_total tokens, of which the first n_prompt
 * are the prompt.  Prompt positions run every layer ("Inference for FiRST" item 1:
 * no skipping in prefill); positions j >= n_prompt run layer l only if keep[l] != 0
 * (item 2) and otherwise carry their residual through (Eq. 3).  At a layer the
 * positions that run it attend causally over the earlier positions that ran it too.
 *   n_prompt == n_total  -> plain prefill of the prompt (keep is ignored, may be NULL)
 *   n_prompt <  n_total  -> what a KV-cached routed decode must reproduce.
 * Outputs (each optional):
 *   k_out[l], v_out[l]   [n_total][Hkv*hd]  rotated keys / values of positions that ran l
 *   router_in            [L][n_total][D]    residual entering layer l (the router's input)
 *   logits               [n_total-logits_from][V] for positions >= logits_from
 * -------------------------------------------------------------------------------*/
int fo_forward_full(const fo_model *m, const fo_weights *w, int32_t n_total, const int32_t *tokens,
                    int32_t n_prompt, const uint8_t *keep, float *const *k_out, float *const *v_out,
                    float *router_in, int32_t logits_from, float *logits) {
    if (!m || !w || !tokens || n_total <= 0 || n_prompt <= 0 || n_prompt > n_total) return FO_E_ARG;
    if (n_prompt < n_total && !keep) return FO_E_ARG;
    int L = m->n_layers, D = m->d_model, Hq = m->n_q_heads, Hkv = m->n_kv_heads, hd = m->head_dim;
    int F = m->ffn_dim, V = m->vocab, dt = m->weight_dtype, n = n_total;
    size_t qd = (size_t)Hq * hd, kvd = (size_t)Hkv * hd;
    for (int j = 0; j < n; ++j)
        if (tokens[j] < 0 || tokens[j] >= V) return FO_E_ARG;
    float *H = malloc((size_t)n * D * sizeof(float));
    float *U = malloc((size_t)n * D * sizeof(float));
    float *Q = malloc((size_t)n * qd * sizeof(float));
    float *K = malloc((size_t)n * kvd * sizeof(float));
    float *Vv = malloc((size_t)n * kvd * sizeof(float));
    float *A = malloc((size_t)n * qd * sizeof(float));
    float *P = malloc((size_t)n * D * sizeof(float));
    float *G = malloc((size_t)n * F * sizeof(float));
    float *Up = malloc((size_t)n * F * sizeof(float));
    if (!H || !U || !Q || !K || !Vv || !A || !P || !G || !Up) return FO_E_ALLOC;

    for (int j = 0; j < n; ++j) load_row(w->embed, dt, (size_t)tokens[j], D, H + (size_t)j * D);

    for (int l = 0; l < L; ++l) {
        if (router_in) memcpy(router_in + (size_t)l * n * D, H, (size_t)n * D * sizeof(float));
        /* positions [0, r) run this layer: everyone if kept, the prompt only if not */
        int r = (n_prompt == n || keep[l]) ? n : n_prompt;
        for (int j = 0; j < r; ++j) rmsnorm(H + (size_t)j * D, w->attn_norm[l], D, m->rms_eps, U + (size_t)j * D);
        linear(w->wq[l], dt, (int)qd, D, U, (size_t)D, Q, qd, r);
        linear(w->wk[l], dt, (int)kvd, D, U, (size_t)D, K, kvd, r);
        linear(w->wv[l], dt, (int)kvd, D, U, (size_t)D, Vv, kvd, r);
        for (int j = 0; j < r; ++j) {
            rope(Q + (size_t)j * qd, Hq, hd, j, m->rope_base);
            rope(K + (size_t)j * kvd, Hkv, hd, j, m->rope_base);
        }
        store_round(K, (size_t)r * kvd, m->kv_dtype); /* attention reads what the cache would hold */
        store_round(Vv, (size_t)r * kvd, m->kv_dtype);
        if (k_out && k_out[l]) memcpy(k_out[l], K, (size_t)r * kvd * sizeof(float));
        if (v_out && v_out[l]) memcpy(v_out[l], Vv, (size_t)r * kvd * sizeof(float));
#pragma omp parallel
        {
            double *score = malloc((size_t)n * sizeof(double));
#pragma omp for schedule(dynamic, 4)
            for (int j = 0; j < r; ++j) attend(m, Q + (size_t)j * qd, K, Vv, j + 1, A + (size_t)j * qd, score);
            free(score);
        }
        linear(w->wo[l], dt, D, (int)qd, A, qd, P, (size_t)D, r);
        for (size_t i = 0; i < (size_t)r * D; ++i) H[i] += P[i];
        for (int j = 0; j < r; ++j) rmsnorm(H + (size_t)j * D, w->ffn_norm[l], D, m->rms_eps, U + (size_t)j * D);
        swiglu_ffn(m, w, l, U, r, G, Up, P);
        for (size_t i = 0; i < (size_t)r * D; ++i) H[i] += P[i];
    }
    if (logits) {
        if (logits_from < 0 || logits_from >= n) return FO_E_ARG;
        int cnt = n - logits_from;
        for (int j = logits_from; j < n; ++j) rmsnorm(H + (size_t)j * D, w->final_norm, D, m->rms_eps, U + (size_t)j * D);
        linear(w->lm_head, dt, V, D, U + (size_t)logits_from * D, (size_t)D, logits, (size_t)V, cnt);
    }
    free(H); free(U); free(Q); free(K); free(Vv); free(A); free(P); free(G); free(Up);
    return FO_OK;
}

/* lowest index of the maximum (greedy decoding; ties -> lowest index) */
int32_t fo_argmax(const float *v, int32_t n) {
    int32_t best = 0;
    for (int32_t i = 1; i < n; ++i)
        if (v[i] > v[best]) best = i;
    return best;
}

/* Temperature + top-k sampling of one row of logits (App. "Training and Inference Setup",
 * inference settings: temperature 0.8, top-k over 10 tokens).  The candidates are the k largest
 * logits, taken one by one (among equal values the lowest index first); their probabilities are
 * the softmax of logit/T over the candidates only; the token is the first candidate, in that
 * order, whose cumulative probability exceeds the uniform draw u in [0,1), which is an input.
 * k = 1 or T = 0 is greedy decoding.  cand[k] and prob[k] (optional) receive the ordered
 * candidates and their probabilities.  Returns the token, or FO_E_ARG. */
int32_t fo_sample_topk(const float *v, int32_t n, int32_t k, double T, double u, int32_t *cand, double *prob) {
    if (!v || n <= 0 || k <= 0 || k > n || T < 0.0 || !(u >= 0.0 && u < 1.0)) return FO_E_ARG;
    int32_t *c = (int32_t *)malloc(sizeof(int32_t) * (size_t)k);
    double *p = (double *)malloc(sizeof(double) * (size_t)k);
    uint8_t *taken = (uint8_t *)calloc((size_t)n, 1);
    if (!c || !p || !taken) { free(c); free(p); free(taken); return FO_E_ARG; }
    for (int32_t j = 0; j < k; ++j) {
        int32_t best = -1;
        for (int32_t i = 0; i < n; ++i)
            if (!taken[i] && (best < 0 || v[i] > v[best])) best = i;
        taken[best] = 1;
        c[j] = best;
    }
    int32_t token = c[0];
    if (k == 1 || T == 0.0) {
        for (int32_t j = 0; j < k; ++j) p[j] = j == 0 ? 1.0 : 0.0;
    } else {
        double sum = 0.0;
        for (int32_t j = 0; j < k; ++j) { p[j] = exp(((double)v[c[j]] - (double)v[c[0]]) / T); sum += p[j]; }
        double cum = 0.0;
        token = c[k - 1];
        for (int32_t j = 0; j < k; ++j) p[j] /= sum;
        for (int32_t j = 0; j < k; ++j) {
            cum += p[j];
            if (u < cum) { token = c[j]; break; }
        }
    }
    for (int32_t j = 0; j < k; ++j) { if (cand) cand[j] = c[j]; if (prob) prob[j] = p[j]; }
    free(c); free(p); free(taken);
    return token;
}

/* Active-row lists of a mask: for each layer the ascending sequence indices that keep
 * it (Sec. "Adaptive Router Module": one decision per sequence per layer). */
int fo_plan(const uint8_t *mask, int32_t B, int32_t L, int32_t *idx, int32_t *cnt, int32_t *slot) {
    if (!mask || !idx || !cnt || B <= 0 || L <= 0) return FO_E_ARG;
    for (int l = 0; l < L; ++l) {
        int c = 0;
        for (int b = 0; b < B; ++b) {
            uint8_t mk = mask[(size_t)b * L + l];
            if (mk > 1) return FO_E_ARG;
            if (slot) slot[(size_t)l * B + b] = mk ? c : -1;
            if (mk) idx[(size_t)l * B + c++] = b;
        }
        for (int i = c; i < B; ++i) idx[(size_t)l * B + i] = -1;
        cnt[l] = c;
    }
    return FO_OK;
}
