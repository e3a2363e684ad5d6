// C ABI of the routed decode step: context, argument checks, launch sequence.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "attn_simple.cuh"
#include "common.cuh"
#include "first.h"
#include "gemv.cuh"
#include "router.cuh"
#include "step.cuh"

using namespace first;

#define CU_TRY(expr)                                                                                   \
    do {                                                                                               \
        cudaError_t e_ = (expr);                                                                       \
        if (e_ != cudaSuccess) {                                                                       \
            std::snprintf(g_last_cuda_error, sizeof g_last_cuda_error, "%s: %s", #expr, cudaGetErrorString(e_)); \
            return FIRST_E_CUDA;                                                                       \
        }                                                                                              \
    } while (0)

static thread_local char g_last_cuda_error[256] = "";

enum KernelClass { kClsStepBegin = 0, kClsRmsnorm, kClsGemv, kClsGemmTc, kClsRopeAppend, kClsAttn, kClsAttnCombine,
                   kClsSiluMul, kClsStepEnd, kClsRouterScores, kClsRouterFinalize, kClsPlan, kNumClasses };
static const char* const kClassNames[kNumClasses] = {"step_begin", "rmsnorm_rows", "gemv_rows", "gemm_tc",
                                                     "rope_append", "attn_split", "attn_combine", "silu_mul",
                                                     "step_end", "router_token_scores", "router_finalize",
                                                     "plan_compact"};

struct first_ctx {
    first_model_desc d{};
    const void *embed = nullptr, *lm_head = nullptr;
    const float* final_norm = nullptr;
    std::vector<const float*> attn_norm, ffn_norm;
    std::vector<const void*> wqkv, wo, w_gate_up, w_down;
    int qd = 0, kvd = 0, qkvd = 0, group = 0;
    int n_sm = 148;
    // scratch (device)
    float *x = nullptr, *xn = nullptr, *qkv = nullptr, *q = nullptr, *att = nullptr, *gu = nullptr, *act = nullptr;
    float *o_part = nullptr, *logits_int = nullptr, *tokscore = nullptr;
    float2 *ml_part = nullptr, *cs = nullptr;
    double* inv_freq = nullptr;
    int32_t *idx = nullptr, *cnt = nullptr, *slot = nullptr;
    uint32_t* flags = nullptr;
    int64_t tok_cap = 0;
    int max_splits = 16;
    // plan (host side)
    std::vector<int32_t> cnt_h;
    int B = 0;
    bool has_mask = false;
    int64_t launches = 0;
    // per-kernel-class timing (off unless first_profile enables it)
    bool profiling = false;
    std::vector<cudaEvent_t> ev_pool;
    std::vector<int> ev_cls;  // class of event pair i (events 2i, 2i+1)
    double prof_ms[kNumClasses] = {};
    int64_t prof_launches[kNumClasses] = {};
    // options
    int max_gemv_rows = -1;
    int attn_simple = -1;
};

namespace {

template <typename T>
int dev_alloc(T** p, size_t n) {
    CU_TRY(cudaMalloc(reinterpret_cast<void**>(p), n * sizeof(T)));
    return FIRST_OK;
}

// Brackets one kernel launch: counts it and, when profiling, records an event pair around it.
struct Launch {
    first_ctx* c;
    cudaStream_t st;
    bool on;
    Launch(first_ctx* c_, cudaStream_t st_, int cls) : c(c_), st(st_), on(c_->profiling) {
        c->launches += 1;
        if (on) {
            const size_t i = c->ev_cls.size();
            while (c->ev_pool.size() < 2 * (i + 1)) {
                cudaEvent_t e;
                if (cudaEventCreate(&e) != cudaSuccess) { on = false; return; }
                c->ev_pool.push_back(e);
            }
            c->ev_cls.push_back(cls);
            cudaEventRecord(c->ev_pool[2 * i], st);
        }
    }
    ~Launch() {
        if (on) cudaEventRecord(c->ev_pool[2 * (c->ev_cls.size() - 1) + 1], st);
    }
};

#define FIRST_LAUNCH(cls, ...)      \
    do {                            \
        Launch guard_(c, st, cls);  \
        __VA_ARGS__;                \
    } while (0)

int check_launch(first_ctx*) {
    CU_TRY(cudaGetLastError());
    return FIRST_OK;
}

template <typename WT, int EPI>
int launch_gemv(first_ctx* c, cudaStream_t st, const void* W, int n_out, int K, const float* X, int m, float* Y,
                int64_t ldy, const int32_t* idx) {
    const int blocks = std::min((n_out + 7) / 8, c->n_sm * 8);
    for (int r0 = 0; r0 < m; r0 += 8) {
        const int rv = std::min(8, m - r0);
        const WT* w = static_cast<const WT*>(W);
        if (rv == 1) FIRST_LAUNCH(kClsGemv, (gemv_rows<WT, 1, EPI><<<blocks, 256, 0, st>>>(w, n_out, K, X, r0, rv, Y, ldy, idx)));
        else if (rv == 2) FIRST_LAUNCH(kClsGemv, (gemv_rows<WT, 2, EPI><<<blocks, 256, 0, st>>>(w, n_out, K, X, r0, rv, Y, ldy, idx)));
        else if (rv <= 4) FIRST_LAUNCH(kClsGemv, (gemv_rows<WT, 4, EPI><<<blocks, 256, 0, st>>>(w, n_out, K, X, r0, rv, Y, ldy, idx)));
        else FIRST_LAUNCH(kClsGemv, (gemv_rows<WT, 8, EPI><<<blocks, 256, 0, st>>>(w, n_out, K, X, r0, rv, Y, ldy, idx)));
        int rc = check_launch(c);
        if (rc) return rc;
    }
    return FIRST_OK;
}

template <typename KT, int HD>
int launch_attn_simple_g(first_ctx* c, cudaStream_t st, int S, int m, const KT* kc, const KT* vc,
                         const first_kv_cache* kv, const int32_t* len_l, const int32_t* idx) {
    dim3 grid(S, c->d.n_kv_heads, m);
#define FIRST_ATTN_CASE(G)                                                                                   \
    case G:                                                                                                  \
        FIRST_LAUNCH(kClsAttn, (attn_split_simple<KT, HD, G><<<grid, 128, 0, st>>>(                          \
                                   c->q, kc, vc, kv->cap_total, kv->slab_off, len_l, idx, c->d.n_q_heads,    \
                                   c->o_part, c->ml_part)));                                                 \
        break;
    switch (c->group) {
        FIRST_ATTN_CASE(1)
        FIRST_ATTN_CASE(2)
        FIRST_ATTN_CASE(4)
        FIRST_ATTN_CASE(8)
        default: return FIRST_E_UNSUPPORTED;
    }
#undef FIRST_ATTN_CASE
    return check_launch(c);
}

template <typename KT>
int launch_attn_simple(first_ctx* c, cudaStream_t st, int S, int m, const void* kc, const void* vc,
                       const first_kv_cache* kv, const int32_t* len_l, const int32_t* idx) {
    const KT *k = static_cast<const KT*>(kc), *v = static_cast<const KT*>(vc);
    switch (c->d.head_dim) {
        case 32: return launch_attn_simple_g<KT, 32>(c, st, S, m, k, v, kv, len_l, idx);
        case 64: return launch_attn_simple_g<KT, 64>(c, st, S, m, k, v, kv, len_l, idx);
        case 128: return launch_attn_simple_g<KT, 128>(c, st, S, m, k, v, kv, len_l, idx);
        default: return FIRST_E_UNSUPPORTED;
    }
}

// The whole step, for one weight/cache element type.
template <typename WT>
int decode_step_impl(first_ctx* c, const int32_t* tokens, const first_kv_cache* kv, float* logits,
                     int32_t* next_tokens, float* layer_inputs, cudaStream_t st) {
    const first_model_desc& d = c->d;
    const int B = c->B, D = d.d_model, F = d.ffn_dim, V = d.vocab, L = d.n_layers, hd = d.head_dim;
    int rc;
    FIRST_LAUNCH(kClsStepBegin, (step_begin<WT><<<B, 256, 0, st>>>(tokens, static_cast<const WT*>(c->embed), D, V, kv->pos, c->inv_freq, hd / 2,
                                      c->x, c->cs, c->flags)));
    if ((rc = check_launch(c))) return rc;

    int S = (d.max_tokens_per_seq + 255) / 256;
    S = std::max(1, std::min(S, c->max_splits));
    const float qscale = 1.0f / std::sqrt((float)hd);

    for (int l = 0; l < L; ++l) {
        if (layer_inputs)
            CU_TRY(cudaMemcpyAsync(layer_inputs + (size_t)l * B * D, c->x, (size_t)B * D * sizeof(float),
                                   cudaMemcpyDeviceToDevice, st));
        const int m = c->cnt_h[l];
        if (m == 0) continue;  // every sequence skips this layer: no launch at all
        const int32_t* idx = c->idx + (size_t)l * B;
        int32_t* len_l = kv->len + (size_t)l * B;
        // attention half
        FIRST_LAUNCH(kClsRmsnorm, (rmsnorm_rows<<<m, 256, 0, st>>>(c->x, idx, D, c->attn_norm[l], d.rms_eps, c->xn, nullptr, nullptr)));
        if ((rc = check_launch(c))) return rc;
        if ((rc = launch_gemv<WT, kStore>(c, st, c->wqkv[l], c->qkvd, D, c->xn, m, c->qkv, c->qkvd, nullptr))) return rc;
        FIRST_LAUNCH(kClsRopeAppend, (rope_append<WT><<<m, 256, 0, st>>>(c->qkv, idx, d.n_q_heads, d.n_kv_heads, hd, c->cs, qscale, c->q,
                                           static_cast<WT*>(kv->k[l]), static_cast<WT*>(kv->v[l]), kv->cap_total,
                                           kv->slab_off, kv->slab_cap, len_l, c->flags)));
        if ((rc = check_launch(c))) return rc;
        if ((rc = launch_attn_simple<WT>(c, st, S, m, kv->k[l], kv->v[l], kv, len_l, idx))) return rc;
        FIRST_LAUNCH(kClsAttnCombine, (attn_combine<<<m * d.n_q_heads, 128, 0, st>>>(c->o_part, c->ml_part, S, hd, c->att, nullptr, nullptr)));
        if ((rc = check_launch(c))) return rc;
        if ((rc = launch_gemv<WT, kScatterAdd>(c, st, c->wo[l], D, c->qd, c->att, m, c->x, D, idx))) return rc;
        // feed-forward half
        FIRST_LAUNCH(kClsRmsnorm, (rmsnorm_rows<<<m, 256, 0, st>>>(c->x, idx, D, c->ffn_norm[l], d.rms_eps, c->xn, nullptr, nullptr)));
        if ((rc = check_launch(c))) return rc;
        if ((rc = launch_gemv<WT, kStore>(c, st, c->w_gate_up[l], 2 * F, D, c->xn, m, c->gu, 2 * F, nullptr))) return rc;
        FIRST_LAUNCH(kClsSiluMul, (silu_mul<<<std::min((m * F + 255) / 256, c->n_sm * 8), 256, 0, st>>>(c->gu, m, F, c->act, nullptr, nullptr)));
        if ((rc = check_launch(c))) return rc;
        if ((rc = launch_gemv<WT, kScatterAdd>(c, st, c->w_down[l], D, F, c->act, m, c->x, D, idx))) return rc;
    }
    float* lg = logits;
    if (!lg && next_tokens) {
        if (!c->logits_int && (rc = dev_alloc(&c->logits_int, (size_t)d.max_batch * V))) return rc;
        lg = c->logits_int;
    }
    if (lg) {
        FIRST_LAUNCH(kClsRmsnorm, (rmsnorm_rows<<<B, 256, 0, st>>>(c->x, nullptr, D, c->final_norm, d.rms_eps, c->xn, nullptr, nullptr)));
        if ((rc = check_launch(c))) return rc;
        if ((rc = launch_gemv<WT, kStore>(c, st, c->lm_head, V, D, c->xn, B, lg, V, nullptr))) return rc;
    }
    FIRST_LAUNCH(kClsStepEnd, (step_end<<<B, 256, 0, st>>>(lg, V, next_tokens, kv->pos)));
    return check_launch(c);
}

}  // namespace

extern "C" {

const char* first_status_string(int status) {
    switch (status) {
        case FIRST_OK: return "ok";
        case FIRST_E_ARG: return "bad argument";
        case FIRST_E_SHAPE: return "inconsistent shape";
        case FIRST_E_UNSUPPORTED: return "unsupported shape or dtype";
        case FIRST_E_CAPACITY: return "capacity exceeded";
        case FIRST_E_CUDA: return g_last_cuda_error[0] ? g_last_cuda_error : "CUDA error";
        case FIRST_E_DEVICE_FLAG: return "device flag set";
        case FIRST_E_STATE: return "call out of order";
        default: return "unknown status";
    }
}

int first_create(const first_model_desc* desc, const first_weights* w, first_ctx** out) {
    if (!desc || !w || !out) return FIRST_E_ARG;
    *out = nullptr;
    const first_model_desc& d = *desc;
    if (d.n_layers <= 0 || d.d_model <= 0 || d.n_q_heads <= 0 || d.n_kv_heads <= 0 || d.head_dim <= 0 ||
        d.ffn_dim <= 0 || d.vocab <= 0 || d.max_batch <= 0 || d.max_tokens_per_seq <= 0 || !(d.rope_base > 0.f) ||
        !(d.rms_eps >= 0.f))
        return FIRST_E_ARG;
    if (d.dtype != FIRST_DTYPE_F32 && d.dtype != FIRST_DTYPE_BF16) return FIRST_E_ARG;
    if (d.n_q_heads % d.n_kv_heads) return FIRST_E_SHAPE;
    const int group = d.n_q_heads / d.n_kv_heads;
    if (d.head_dim != 32 && d.head_dim != 64 && d.head_dim != 128) return FIRST_E_UNSUPPORTED;
    if (group != 1 && group != 2 && group != 4 && group != 8) return FIRST_E_UNSUPPORTED;
    if (d.d_model % 8 || d.ffn_dim % 8) return FIRST_E_UNSUPPORTED;
    if (!w->embed || !w->lm_head || !w->final_norm || !w->attn_norm || !w->wqkv || !w->wo || !w->ffn_norm ||
        !w->w_gate_up || !w->w_down)
        return FIRST_E_ARG;
    for (int l = 0; l < d.n_layers; ++l)
        if (!w->attn_norm[l] || !w->wqkv[l] || !w->wo[l] || !w->ffn_norm[l] || !w->w_gate_up[l] || !w->w_down[l])
            return FIRST_E_ARG;

    first_ctx* c = new (std::nothrow) first_ctx();
    if (!c) return FIRST_E_ARG;
    c->d = d;
    c->embed = w->embed;
    c->lm_head = w->lm_head;
    c->final_norm = w->final_norm;
    c->attn_norm.assign(w->attn_norm, w->attn_norm + d.n_layers);
    c->ffn_norm.assign(w->ffn_norm, w->ffn_norm + d.n_layers);
    c->wqkv.assign(w->wqkv, w->wqkv + d.n_layers);
    c->wo.assign(w->wo, w->wo + d.n_layers);
    c->w_gate_up.assign(w->w_gate_up, w->w_gate_up + d.n_layers);
    c->w_down.assign(w->w_down, w->w_down + d.n_layers);
    c->group = group;
    c->qd = d.n_q_heads * d.head_dim;
    c->kvd = d.n_kv_heads * d.head_dim;
    c->qkvd = c->qd + 2 * c->kvd;
    c->cnt_h.assign(d.n_layers, 0);

    int dev = 0, rc = FIRST_OK;
    auto fail = [&](int code) { first_destroy(c); return code; };
    if (cudaGetDevice(&dev) != cudaSuccess) return fail(FIRST_E_CUDA);
    cudaDeviceGetAttribute(&c->n_sm, cudaDevAttrMultiProcessorCount, dev);
    const size_t MB = d.max_batch;
    const int xw = std::max(d.d_model, c->qd);
    if ((rc = dev_alloc(&c->x, MB * d.d_model)) || (rc = dev_alloc(&c->xn, MB * xw)) ||
        (rc = dev_alloc(&c->qkv, MB * c->qkvd)) || (rc = dev_alloc(&c->q, MB * c->qd)) ||
        (rc = dev_alloc(&c->att, MB * c->qd)) || (rc = dev_alloc(&c->gu, MB * 2 * d.ffn_dim)) ||
        (rc = dev_alloc(&c->act, MB * d.ffn_dim)) ||
        (rc = dev_alloc(&c->o_part, MB * d.n_q_heads * c->max_splits * d.head_dim)) ||
        (rc = dev_alloc(&c->ml_part, MB * d.n_q_heads * c->max_splits)) ||
        (rc = dev_alloc(&c->cs, MB * (d.head_dim / 2))) || (rc = dev_alloc(&c->inv_freq, (size_t)d.head_dim / 2)) ||
        (rc = dev_alloc(&c->idx, MB * d.n_layers)) || (rc = dev_alloc(&c->cnt, (size_t)d.n_layers)) ||
        (rc = dev_alloc(&c->slot, MB * d.n_layers)) || (rc = dev_alloc(&c->flags, (size_t)1)))
        return fail(rc);
    c->tok_cap = (int64_t)d.max_batch * d.max_tokens_per_seq;
    if ((rc = dev_alloc(&c->tokscore, (size_t)c->tok_cap))) return fail(rc);
    std::vector<double> inv(d.head_dim / 2);
    for (int i = 0; i < d.head_dim / 2; ++i) inv[i] = std::pow((double)d.rope_base, -2.0 * i / (double)d.head_dim);
    if (cudaMemcpy(c->inv_freq, inv.data(), inv.size() * sizeof(double), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemset(c->flags, 0, sizeof(uint32_t)) != cudaSuccess)
        return fail(FIRST_E_CUDA);
    *out = c;
    return FIRST_OK;
}

int first_destroy(first_ctx* c) {
    if (!c) return FIRST_OK;
    void* ptrs[] = {c->x, c->xn, c->qkv, c->q, c->att, c->gu, c->act, c->o_part, c->logits_int, c->tokscore,
                    c->ml_part, c->cs, c->inv_freq, c->idx, c->cnt, c->slot, c->flags};
    for (void* p : ptrs)
        if (p) cudaFree(p);
    for (cudaEvent_t e : c->ev_pool) cudaEventDestroy(e);
    delete c;
    return FIRST_OK;
}

int first_prefill_route(first_ctx* c, int32_t layer, const void* hidden, int32_t hidden_dtype,
                        const int32_t* cu_seqlens, int32_t B, int64_t total_tokens, const float* router_w,
                        const float* router_b, float tau, int32_t mode, uint8_t* mask, float* scores, void* stream) {
    if (!c || !hidden || !cu_seqlens || !router_w || !mask) return FIRST_E_ARG;
    if (layer < 0 || layer >= c->d.n_layers || B <= 0 || total_tokens <= 0) return FIRST_E_ARG;
    if (hidden_dtype != FIRST_DTYPE_F32 && hidden_dtype != FIRST_DTYPE_BF16) return FIRST_E_ARG;
    if (mode != FIRST_ROUTER_MEAN_OF_SIGMOID && mode != FIRST_ROUTER_SIGMOID_OF_MEAN) return FIRST_E_ARG;
    if (!(tau > 0.f && tau < 1.f)) return FIRST_E_ARG;
    if (total_tokens > c->tok_cap || total_tokens > 0x7fffffffLL) return FIRST_E_CAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int D = c->d.d_model;
    const int64_t want = (total_tokens + 7) / 8;
    const int blocks = (int)std::min<int64_t>(want, (int64_t)c->n_sm * 8);
    const size_t smem = (size_t)D * sizeof(float);
    if (hidden_dtype == FIRST_DTYPE_BF16)
        FIRST_LAUNCH(kClsRouterScores, (router_token_scores<__nv_bfloat16><<<blocks, 256, smem, st>>>(static_cast<const __nv_bfloat16*>(hidden),
                                                                      total_tokens, D, router_w, router_b, mode,
                                                                      c->tokscore)));
    else
        FIRST_LAUNCH(kClsRouterScores, (router_token_scores<float><<<blocks, 256, smem, st>>>(static_cast<const float*>(hidden), total_tokens, D,
                                                              router_w, router_b, mode, c->tokscore)));
    int rc = check_launch(c);
    if (rc) return rc;
    FIRST_LAUNCH(kClsRouterFinalize, (router_finalize<<<B, 256, 0, st>>>(c->tokscore, cu_seqlens, c->d.n_layers, layer, mode, tau, mask, scores,
                                       c->flags)));
    return check_launch(c);
}

int first_set_mask(first_ctx* c, const uint8_t* mask, int32_t B, void* stream) {
    if (!c || !mask || B <= 0) return FIRST_E_ARG;
    if (B > c->d.max_batch) return FIRST_E_CAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    c->has_mask = false;
    FIRST_LAUNCH(kClsPlan, (plan_compact<<<c->d.n_layers, 32, 0, st>>>(mask, B, c->d.n_layers, c->idx, c->cnt, c->slot, c->flags)));
    int rc = check_launch(c);
    if (rc) return rc;
    uint32_t fl = 0;
    CU_TRY(cudaMemcpyAsync(c->cnt_h.data(), c->cnt, sizeof(int32_t) * c->d.n_layers, cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaMemcpyAsync(&fl, c->flags, sizeof fl, cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaStreamSynchronize(st));
    if (fl & FIRST_FLAG_BAD_MASK) return FIRST_E_DEVICE_FLAG;
    c->B = B;
    c->has_mask = true;
    return FIRST_OK;
}

int first_get_plan(first_ctx* c, int32_t* idx, int32_t* cnt, int32_t* slot) {
    if (!c || !idx || !cnt) return FIRST_E_ARG;
    if (!c->has_mask) return FIRST_E_STATE;
    const size_t n = (size_t)c->d.n_layers * c->B;
    CU_TRY(cudaMemcpy(idx, c->idx, n * sizeof(int32_t), cudaMemcpyDeviceToHost));
    CU_TRY(cudaMemcpy(cnt, c->cnt, (size_t)c->d.n_layers * sizeof(int32_t), cudaMemcpyDeviceToHost));
    if (slot) CU_TRY(cudaMemcpy(slot, c->slot, n * sizeof(int32_t), cudaMemcpyDeviceToHost));
    return FIRST_OK;
}

int first_decode_step(first_ctx* c, const int32_t* tokens, const first_kv_cache* kv, float* logits,
                      int32_t* next_tokens, float* layer_inputs, void* stream) {
    if (!c || !tokens || !kv) return FIRST_E_ARG;
    if (!c->has_mask) return FIRST_E_STATE;
    if (!kv->k || !kv->v || !kv->slab_off || !kv->slab_cap || !kv->len || !kv->pos || kv->cap_total <= 0)
        return FIRST_E_ARG;
    for (int l = 0; l < c->d.n_layers; ++l)
        if (c->cnt_h[l] > 0 && (!kv->k[l] || !kv->v[l])) return FIRST_E_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (c->d.dtype == FIRST_DTYPE_BF16)
        return decode_step_impl<__nv_bfloat16>(c, tokens, kv, logits, next_tokens, layer_inputs, st);
    return decode_step_impl<float>(c, tokens, kv, logits, next_tokens, layer_inputs, st);
}

int first_last_device_flags(first_ctx* c, uint32_t* flags, void* stream) {
    if (!c || !flags) return FIRST_E_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CU_TRY(cudaMemcpyAsync(flags, c->flags, sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaMemsetAsync(c->flags, 0, sizeof(uint32_t), st));
    CU_TRY(cudaStreamSynchronize(st));
    return *flags ? FIRST_E_DEVICE_FLAG : FIRST_OK;
}

int64_t first_launch_count(const first_ctx* c) { return c ? c->launches : 0; }

int first_profile(first_ctx* c, int32_t enable) {
    if (!c) return FIRST_E_ARG;
    c->profiling = enable != 0;
    c->ev_cls.clear();
    for (int k = 0; k < kNumClasses; ++k) { c->prof_ms[k] = 0.0; c->prof_launches[k] = 0; }
    return FIRST_OK;
}

int first_profile_read(first_ctx* c, int32_t n, double* ms, int64_t* launches, void* stream) {
    if (!c || !ms || !launches || n < kNumClasses) return FIRST_E_ARG;
    CU_TRY(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    for (size_t i = 0; i < c->ev_cls.size(); ++i) {
        float t = 0.f;
        CU_TRY(cudaEventElapsedTime(&t, c->ev_pool[2 * i], c->ev_pool[2 * i + 1]));
        c->prof_ms[c->ev_cls[i]] += t;
        c->prof_launches[c->ev_cls[i]] += 1;
    }
    c->ev_cls.clear();
    for (int k = 0; k < n; ++k) {
        ms[k] = k < kNumClasses ? c->prof_ms[k] : 0.0;
        launches[k] = k < kNumClasses ? c->prof_launches[k] : 0;
    }
    return FIRST_OK;
}

int32_t first_kernel_class_count(void) { return kNumClasses; }
const char* first_kernel_class_name(int32_t k) { return (k >= 0 && k < kNumClasses) ? kClassNames[k] : ""; }

int first_set_option(first_ctx* c, const char* name, int64_t value) {
    if (!c || !name) return FIRST_E_ARG;
    if (!std::strcmp(name, "max_gemv_rows")) c->max_gemv_rows = (int)value;
    else if (!std::strcmp(name, "attn_simple")) c->attn_simple = (int)value;
    else return FIRST_E_ARG;
    return FIRST_OK;
}

}  // extern "C"
