// Router scoring for callers that must not allocate device memory.
//
// Same two kernels as first_prefill_route, but the per-token score scratch lives in a
// fixed array inside this library's device image instead of a context's cudaMalloc'd
// buffer.  See first_prefill_route_static in first.h for who needs this and the limits.
#include <mutex>

#include "first.h"
#include "router.cuh"

using namespace first;

namespace {

constexpr int64_t kStaticMaxTokens = FIRST_STATIC_ROUTE_MAX_TOKENS;
constexpr int kMaxDevices = 64;

// Word 0 of the header is the flag word used when the caller passes none; the token
// scores follow.  Every process that loads the library holds this on each GPU it touches.
struct StaticRouteScratch {
    uint32_t header[64];
    float tok[kStaticMaxTokens];
};
static __device__ __align__(256) StaticRouteScratch g_route_scratch;

// In host code `g_route_scratch` is only a handle for the runtime, not an address a kernel
// can use; the real device address is looked up once per device and kept here.
std::mutex g_mu;
StaticRouteScratch* g_dev_ptr[kMaxDevices] = {};

int scratch_for_current_device(StaticRouteScratch** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return FIRST_E_CUDA;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_dev_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_route_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return FIRST_E_CUDA;
        }
        g_dev_ptr[dev] = static_cast<StaticRouteScratch*>(p);
    }
    *out = g_dev_ptr[dev];
    return FIRST_OK;
}

}  // namespace

extern "C" int first_prefill_route_static(int32_t layer, int32_t n_layers, int32_t d_model, const void* hidden,
                                          int32_t hidden_dtype, const int32_t* cu_seqlens, int32_t B,
                                          int64_t total_tokens, const float* router_w, const float* router_b,
                                          float tau, int32_t mode, uint8_t* mask, float* scores, uint32_t* flags,
                                          void* stream) {
    if (!hidden || !cu_seqlens || !router_w || !mask) return FIRST_E_ARG;
    if (n_layers <= 0 || layer < 0 || layer >= n_layers || B <= 0 || total_tokens <= 0) return FIRST_E_ARG;
    if (d_model <= 0 || d_model % 8) return FIRST_E_UNSUPPORTED;
    if ((size_t)d_model * sizeof(float) > 48 * 1024) return FIRST_E_UNSUPPORTED;  // router weights sit in shared memory
    if (hidden_dtype != FIRST_DTYPE_F32 && hidden_dtype != FIRST_DTYPE_BF16) return FIRST_E_ARG;
    if (mode != FIRST_ROUTER_MEAN_OF_SIGMOID && mode != FIRST_ROUTER_SIGMOID_OF_MEAN) return FIRST_E_ARG;
    if (!(tau > 0.f && tau < 1.f)) return FIRST_E_ARG;
    if (total_tokens > kStaticMaxTokens) return FIRST_E_CAPACITY;  // beyond the built-in scratch

    StaticRouteScratch* s = nullptr;
    int rc = scratch_for_current_device(&s);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t* fl = flags;
    if (!fl) {
        // the built-in flag word keeps the previous call's bits: start it from zero
        fl = &s->header[0];
        if (cudaMemsetAsync(fl, 0, sizeof(uint32_t), st) != cudaSuccess) return FIRST_E_CUDA;
    }
    int n_sm = 148;
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    const int64_t want = (total_tokens + 7) / 8;
    const int blocks = (int)(want < (int64_t)n_sm * 8 ? want : (int64_t)n_sm * 8);
    const size_t smem = (size_t)d_model * sizeof(float);
    if (hidden_dtype == FIRST_DTYPE_BF16)
        router_token_scores<__nv_bfloat16><<<blocks, 256, smem, st>>>(static_cast<const __nv_bfloat16*>(hidden),
                                                                      total_tokens, d_model, router_w, router_b, mode,
                                                                      s->tok);
    else
        router_token_scores<float><<<blocks, 256, smem, st>>>(static_cast<const float*>(hidden), total_tokens, d_model,
                                                              router_w, router_b, mode, s->tok);
    if (cudaGetLastError() != cudaSuccess) return FIRST_E_CUDA;
    router_finalize<<<B, 256, 0, st>>>(s->tok, cu_seqlens, total_tokens, n_layers, layer, mode, tau, mask, scores, fl);
    if (cudaGetLastError() != cudaSuccess) return FIRST_E_CUDA;
    return FIRST_OK;
}
