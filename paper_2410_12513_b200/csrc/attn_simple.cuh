// Grouped-query decode attention over the active rows' caches, general version
// (any cache dtype, head_dim 32/64/128): plain coalesced loads, one warp per token,
// warp-shuffle dot products, online softmax.  Split along the token axis; a second
// kernel merges the splits.
#pragma once
#include "common.cuh"

namespace first {

// grid (S, Hkv, m), 128 threads.  Work item = (active row i, kv head h, split s): tokens
// [s*C, min(T,(s+1)*C)) with C = ceil(T/S), T = len[b]+1 (the new token is already written at row len[b]).
// q: [m][Hq][HD] float32, pre-scaled.  Partials: o_part [m][Hq][S][HD], ml_part [m][Hq][S] = (max, sum).
template <typename KT, int HD, int G>
__global__ void __launch_bounds__(128) attn_split_simple(const float* q, const KT* kc,
                                                         const KT* vc, int64_t cap_total,
                                                         const int64_t* __restrict__ slab_off,
                                                         const int32_t* len_l,
                                                         const int32_t* __restrict__ slab_cap,
                                                         const int32_t* __restrict__ idx,
                                                         const int32_t* __restrict__ m_dev, int Hq,
                                                         float* __restrict__ o_part, float2* __restrict__ ml_part,
                                                         int cap_max, uint64_t* stamp) {
    const Stamp stamp_guard(stamp);
    pdl_trigger();
    pdl_wait();
    if (m_dev && (int)blockIdx.z >= __ldg(m_dev)) return;  // beyond the layer's active rows (grid sized from a bound)
    constexpr int EPL = HD / 32;
    const int S = gridDim.x, s = blockIdx.x, h = blockIdx.y, i = blockIdx.z;
    const int b = idx[i];
    const int T = min(len_l[b] + 1, min(slab_cap[b], cap_max));  // the new token sits at row len (len itself advances later)
    const int C = (T + S - 1) / S;
    const int t0 = s * C, t1 = min(T, t0 + C);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    __shared__ float q_s[G][HD];
    __shared__ float acc_s[4][G][HD];
    __shared__ float m_s[4][G], l_s[4][G];
    for (int e = threadIdx.x; e < G * HD; e += 128) q_s[e / HD][e % HD] = q[((size_t)i * Hq + (size_t)h * G) * HD + e];
    __syncthreads();

    float qr[G][EPL], acc[G][EPL], mx[G], ls[G];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        mx[g] = -INFINITY;
        ls[g] = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) { qr[g][e] = q_s[g][lane * EPL + e]; acc[g][e] = 0.f; }
    }
    const KT* kbase = kc + ((size_t)h * cap_total + (size_t)slab_off[b]) * HD;
    const KT* vbase = vc + ((size_t)h * cap_total + (size_t)slab_off[b]) * HD;
    for (int t = t0 + warp; t < t1; t += 4) {
        float kv[EPL], vv[EPL];
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
            kv[e] = to_f32<KT>(kbase[(size_t)t * HD + lane * EPL + e]);
            vv[e] = to_f32<KT>(vbase[(size_t)t * HD + lane * EPL + e]);
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float d = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) d = fmaf(qr[g][e], kv[e], d);
            d = warp_sum(d);
            const float mn = fmaxf(mx[g], d);
            const float sc = __expf(mx[g] - mn), p = __expf(d - mn);
            ls[g] = ls[g] * sc + p;
#pragma unroll
            for (int e = 0; e < EPL; ++e) acc[g][e] = acc[g][e] * sc + p * vv[e];
            mx[g] = mn;
        }
    }
#pragma unroll
    for (int g = 0; g < G; ++g) {
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc_s[warp][g][lane * EPL + e] = acc[g][e];
        if (lane == 0) { m_s[warp][g] = mx[g]; l_s[warp][g] = ls[g]; }
    }
    __syncthreads();
    for (int e = threadIdx.x; e < G * HD; e += 128) {
        const int g = e / HD, d = e % HD;
        const float M = fmaxf(fmaxf(m_s[0][g], m_s[1][g]), fmaxf(m_s[2][g], m_s[3][g]));
        float o = 0.f, l = 0.f;
        if (M > -INFINITY) {
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                if (m_s[w][g] > -INFINITY) {
                    const float sc = __expf(m_s[w][g] - M);
                    o += acc_s[w][g][d] * sc;
                    l += l_s[w][g] * sc;
                }
            }
        }
        const size_t hq = (size_t)i * Hq + (size_t)h * G + g;
        o_part[(hq * S + s) * HD + d] = o;
        if (d == 0) ml_part[hq * S + s] = make_float2(M, l);
    }
}

// Merge the S partial results of each (row, query head): out[i][hq*HD + d] (float32) and,
// optionally, its bfloat16 hi/lo split for the tensor-core O-projection.
__global__ void __launch_bounds__(128) attn_combine(const float* o_part, const float2* ml_part,
                                                    const int32_t* __restrict__ m_dev, int Hq,
                                                    int S, int HD, float* __restrict__ out,
                                                    __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo,
                                                    uint64_t* stamp) {
    const Stamp stamp_guard(stamp);
    pdl_trigger();
    pdl_wait();
    if (m_dev && (int)(blockIdx.x / Hq) >= __ldg(m_dev)) return;
    const size_t hq = blockIdx.x;  // flat (row, query head)
    float M = -INFINITY;
    for (int s = 0; s < S; ++s) M = fmaxf(M, ml_part[hq * S + s].x);
    float den = 0.f;
    for (int s = 0; s < S; ++s) {
        const float2 ml = ml_part[hq * S + s];
        if (ml.x > -INFINITY) den += ml.y * __expf(ml.x - M);
    }
    for (int d = threadIdx.x; d < HD; d += blockDim.x) {
        float o = 0.f;
        for (int s = 0; s < S; ++s) {
            const float mx = ml_part[hq * S + s].x;
            if (mx > -INFINITY) o += o_part[(hq * S + s) * HD + d] * __expf(mx - M);
        }
        const float y = o / den;
        if (out) out[hq * HD + d] = y;
        if (hi) {
            const __nv_bfloat16 hh = __float2bfloat16_rn(y);
            hi[hq * HD + d] = hh;
            lo[hq * HD + d] = __float2bfloat16_rn(y - __bfloat162float(hh));
        }
    }
}

}  // namespace first
