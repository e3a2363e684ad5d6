// Per-step kernels around the projections: embedding gather, RMSNorm of the compacted
// active rows, rotary embedding + KV append, SwiGLU activation, greedy argmax.
#pragma once
#include "common.cuh"
#include "first.h"

namespace first {

// Start of a step: residual rows from the embedding table, and the rotary cos/sin of
// every sequence's position (same for all layers, so computed once, in float64:
// angle = pos * base^(-2i/hd), half-split pairing).
template <typename WT>
__global__ void __launch_bounds__(256) step_begin(const int32_t* __restrict__ tokens, const WT* __restrict__ embed,
                                                  int D, int V, const int32_t* __restrict__ pos,
                                                  const double* __restrict__ inv_freq, int half,
                                                  float* __restrict__ x, float2* __restrict__ cs,
                                                  uint32_t* __restrict__ flags, uint64_t* stamp) {
    const Stamp stamp_guard(stamp);
    pdl_trigger();
    pdl_wait();
    const int b = blockIdx.x;
    int tok = tokens[b];
    if (tok < 0 || tok >= V) {
        if (threadIdx.x == 0) atomicOr(flags, FIRST_FLAG_BAD_TOKEN);
        tok = 0;
    }
    const WT* e = embed + (size_t)tok * D;
    for (int k = threadIdx.x * 8; k < D; k += blockDim.x * 8) {
        float f[8];
        Load8<WT>::ld(e + k, f);
        float4* o = reinterpret_cast<float4*>(x + (size_t)b * D + k);
        o[0] = make_float4(f[0], f[1], f[2], f[3]);
        o[1] = make_float4(f[4], f[5], f[6], f[7]);
    }
    const double p = (double)pos[b];
    for (int i = threadIdx.x; i < half; i += blockDim.x) {
        double s, c;
        sincos(p * inv_freq[i], &s, &c);
        cs[(size_t)b * half + i] = make_float2((float)c, (float)s);
    }
}

__device__ __forceinline__ void split_store4(const float (&y)[4], __nv_bfloat16* hi, __nv_bfloat16* lo) {
    __nv_bfloat16 h[4], l[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        h[e] = __float2bfloat16_rn(y[e]);
        l[e] = __float2bfloat16_rn(y[e] - __bfloat162float(h[e]));
    }
    *reinterpret_cast<uint2*>(hi) = *reinterpret_cast<uint2*>(h);
    *reinterpret_cast<uint2*>(lo) = *reinterpret_cast<uint2*>(l);
}

// RMSNorm of the rows a layer keeps, written compactly: out[i] = norm(x[idx[i]]) * gain.
// Also emits the bfloat16 hi/lo split (v = hi + lo up to 2^-17 relative) that the
// tensor-core projections consume, when asked.  One block per active row.
// Two small jobs ride along so that they need no launch of their own:
//   zero_row: row i of a float32 accumulator (zero_cols wide) is cleared for a split-K projection;
//   len_inc:  the row's cache length is advanced by one (unless its slab is full) -- done here,
//             after the layer's attention, so no attention block can see a half-updated length.
//   rowinfo:  (attention side) what the attention kernel needs to know about row i, in one 16-byte
//             word: x = tokens to attend over (cache length + the new token, at most the slab's
//             capacity) | batch row << 32;  y = first slab row | (1 << 62 when the new token's key
//             and value are to be appended).  A full slab raises FIRST_FLAG_KV_FULL.
//   router:   (prompt processing) the row is also what the layer's router reads: its score
//             z = router_w . x[b] (+ bias) goes to tok_out[i], as sigmoid(z) in the paper's order
//             (mean of per-token sigmoids) or as z in the pooled order, like router_token_scores.
// m_dev (all the per-layer kernels have it): the layer's active-row count in device memory.  The grid is sized
// from a host-side upper bound of it (so that a recorded launch sequence survives small changes of the batch);
// work items beyond the count leave at once.  NULL = every row of the grid is live.
__global__ void __launch_bounds__(1024) rmsnorm_rows(const float* x, const int32_t* __restrict__ idx,
                                                     const int32_t* __restrict__ m_dev, int D,
                                                     const float* __restrict__ gain, float eps, float* __restrict__ out,
                                                     __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo,
                                                     float* __restrict__ zero_row, int zero_cols,
                                                     int32_t* __restrict__ len_inc, const int32_t* __restrict__ slab_cap,
                                                     longlong2* __restrict__ rowinfo,
                                                     const int32_t* len_ro,
                                                     const int64_t* __restrict__ slab_off,
                                                     uint32_t* __restrict__ flags,
                                                     const float* __restrict__ router_w,
                                                     const float* __restrict__ router_b, int router_mode,
                                                     float* __restrict__ tok_out, int cap_max, uint64_t* stamp) {
    const Stamp stamp_guard(stamp);
    // One pass: the row stays in registers between the sum of squares and the scaling
    // (up to kMaxV float4 per thread; longer rows re-read the tail from L1/L2).
    constexpr int kMaxV = 4;
    pdl_trigger();
    const int i = blockIdx.x, nt = blockDim.x;
    if (m_dev && i >= __ldg(m_dev)) {  // (the plan is fixed between first_set_mask calls)
        pdl_wait();  // a grid must not complete before its predecessor has: later kernels rely on that chain
        return;
    }
    float4 g[kMaxV];
    const int nv = D / 4;
#pragma unroll
    for (int v = 0; v < kMaxV; ++v) {  // gains do not depend on the previous kernel: fetch them before the wait
        const int k = threadIdx.x + v * nt;
        if (k < nv) g[v] = __ldg(reinterpret_cast<const float4*>(gain) + k);
    }
    const int b = idx ? idx[i] : i;  // the plan is fixed between first_set_mask calls: no need to wait for it
    pdl_wait();
    __shared__ float red[32];
    __shared__ float red_r[32];
    // cap_max: the context was sized for slabs of at most this many tokens (the attention grid covers no more);
    // a longer slab is used up to there and then counts as full
    if (len_inc && threadIdx.x == 0) {
        const int T = len_inc[b];
        if (T < min(slab_cap[b], cap_max)) len_inc[b] = T + 1;
    }
    if (rowinfo && threadIdx.x == (blockDim.x > 32 ? 32 : 0)) {
        const int T = len_ro[b], cap = min(slab_cap[b], cap_max);
        const bool room = T < cap;
        rowinfo[i] = make_longlong2((long long)min(T + 1, cap) | ((long long)b << 32),
                                    (long long)slab_off[b] | (room ? (1ll << 62) : 0ll));
        if (!room) atomicOr(flags, FIRST_FLAG_KV_FULL);
    }
    const float4* xr = reinterpret_cast<const float4*>(x + (size_t)b * D);
    float4 r[kMaxV];
    float ss = 0.f, rd = 0.f;
    const float4* rw4 = reinterpret_cast<const float4*>(router_w);
#pragma unroll
    for (int v = 0; v < kMaxV; ++v) {
        const int k = threadIdx.x + v * nt;
        if (k < nv) {
            r[v] = xr[k];
            ss += r[v].x * r[v].x + r[v].y * r[v].y + r[v].z * r[v].z + r[v].w * r[v].w;
            if (router_w) {
                const float4 w = __ldg(rw4 + k);
                rd += r[v].x * w.x + r[v].y * w.y + r[v].z * w.z + r[v].w * w.w;
            }
        }
    }
    for (int k = threadIdx.x + kMaxV * nt; k < nv; k += nt) {
        const float4 v = xr[k];
        ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        if (router_w) {
            const float4 w = __ldg(rw4 + k);
            rd += v.x * w.x + v.y * w.y + v.z * w.z + v.w * w.w;
        }
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    if (router_w) {
        rd = warp_sum(rd);
        if ((threadIdx.x & 31) == 0) red_r[threadIdx.x >> 5] = rd;
    }
    if (zero_row) {
        float4* z = reinterpret_cast<float4*>(zero_row + (size_t)i * zero_cols);
        for (int k = threadIdx.x; k < zero_cols / 4; k += nt) z[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    __syncthreads();
    float tot = 0.f;
    for (int w = 0; w < (nt >> 5); ++w) tot += red[w];
    if (router_w && threadIdx.x == 0) {
        float z = router_b ? router_b[0] : 0.f;
        for (int w = 0; w < (nt >> 5); ++w) z += red_r[w];
        tok_out[i] = (router_mode == FIRST_ROUTER_MEAN_OF_SIGMOID) ? 1.f / (1.f + expf(-z)) : z;
    }
    const float inv = rsqrtf(tot / (float)D + eps);
    auto emit = [&](int k, const float4& v, const float4& gg) {
        const float y[4] = {v.x * inv * gg.x, v.y * inv * gg.y, v.z * inv * gg.z, v.w * inv * gg.w};
        if (out) *reinterpret_cast<float4*>(out + (size_t)i * D + 4 * k) = make_float4(y[0], y[1], y[2], y[3]);
        if (hi) split_store4(y, hi + (size_t)i * D + 4 * k, lo + (size_t)i * D + 4 * k);
    };
#pragma unroll
    for (int v = 0; v < kMaxV; ++v) {
        const int k = threadIdx.x + v * nt;
        if (k < nv) emit(k, r[v], g[v]);
    }
    for (int k = threadIdx.x + kMaxV * nt; k < nv; k += nt) emit(k, xr[k], __ldg(reinterpret_cast<const float4*>(gain) + k));
}

// After the QKV projection: rotate q and k at the sequence's position, scale q by
// 1/sqrt(hd), write k and v at row len[l][b] of the sequence's slab.
// qkv: [m][(Hq+2Hkv)*hd] float32 (q heads, k heads, v heads).  grid (ceil((Hq+2*Hkv)/8), m), block
// (hd/2, 8): eight heads of a row per block; thread (d, .) handles the rotary pair (d, d+hd/2) of its head.
// len is only read here (the FFN-side rmsnorm_rows advances it once attention is done).
// rowinfo[i] = (tokens to attend over, first slab row) saves the attention CTAs two dependent loads.
// pair: 0 = every row has work items of its own; 1 = mark pairs of consecutive tokens (attn_split_mma's pair form);
// 2 = mark groups of up to eight consecutive tokens (attn_group_mma).
// A full slab sets FIRST_FLAG_KV_FULL and leaves the cache alone.
template <typename KT>
__global__ void __launch_bounds__(512) rope_append(const float* qkv, const int32_t* __restrict__ idx,
                                                  const int32_t* __restrict__ m_dev,
                                                  int Hq, int Hkv, int hd, const float2* cs,
                                                  float qscale, float* __restrict__ q_out, KT* __restrict__ kc,
                                                  KT* __restrict__ vc, int64_t cap_total,
                                                  const int64_t* __restrict__ slab_off,
                                                  const int32_t* __restrict__ slab_cap,
                                                  const int32_t* len_l, uint32_t* __restrict__ flags,
                                                  longlong2* __restrict__ rowinfo, int pair, int cap_max,
                                                  uint64_t* stamp) {
    const Stamp stamp_guard(stamp);
    pdl_trigger();
    const int m = m_dev ? min((int)gridDim.y, __ldg(m_dev)) : (int)gridDim.y;
    pdl_wait();
    if ((int)blockIdx.y >= m) return;
    const int i = blockIdx.y, head = blockIdx.x * blockDim.y + threadIdx.y, d = threadIdx.x, b = idx[i];
    if (head >= Hq + 2 * Hkv) return;
    if (rowinfo && head == 0 && d < 32) {  // what attention needs to know about this row, in one 16-byte word
        long long y = (long long)slab_off[b];
        if (pair == 1 && d == 0) {
            // Prompt processing: rows i0, i0+1 that are consecutive tokens of one slab (the first at an even
            // position, both with room) share attention work items: bit 61 marks the first, bit 60 the second.
            auto is_pair = [&](int i0) {
                if (i0 < 0 || i0 + 1 >= m) return false;
                const int b0 = idx[i0], b1 = idx[i0 + 1];
                const int t0 = len_l[b0];
                return slab_off[b0] == slab_off[b1] && slab_cap[b0] == slab_cap[b1] && len_l[b1] == t0 + 1 &&
                       t0 + 1 < min(slab_cap[b1], cap_max) && !(t0 & 1);
            };
            if (is_pair(i - 1)) y |= 1ll << 60;
            else if (is_pair(i)) y |= 1ll << 61;
        } else if (pair == 2) {
            // Groups (attn_group_mma): up to eight consecutive tokens of one slab inside one block of eight
            // positions.  A row leads a group unless it continues its predecessor's (again a local rule): bit 60
            // = served by the leader; a leader carries its member count - 1 in bits 56..59.  Lane d of the first
            // warp looks at rows i+d-1, i+d (the eight pairs are independent, so they are looked at side by side).
            auto consec = [&](int a) {  // rows a, a+1: consecutive tokens of one slab, the second with room
                if (a < 0 || a + 1 >= m) return false;
                const int b0 = idx[a], b1 = idx[a + 1];
                return slab_off[b0] == slab_off[b1] && slab_cap[b0] == slab_cap[b1] && len_l[b1] == len_l[b0] + 1 &&
                       len_l[b1] < min(slab_cap[b1], cap_max);
            };
            const int p = len_l[b];
            const bool link = d < 8 && consec(i + d - 1) && ((p + d) & 7) != 0;  // row i+d continues row i+d-1's group
            const unsigned links = __ballot_sync(__activemask(), link);
            if (links & 1u) y |= 1ll << 60;
            else y |= (long long)(__ffs(~((links >> 1) & 0x7fu)) - 1) << 56;  // members after the leader: leading links
        }
        if (d == 0)
            rowinfo[i] = make_longlong2((long long)min(len_l[b] + 1, min(slab_cap[b], cap_max)) | ((long long)b << 32), y);
    }
    const int half = hd >> 1;
    const int qd = Hq * hd, kvd = Hkv * hd;
    const float* row = qkv + (size_t)i * (qd + 2 * kvd) + (size_t)head * hd;
    const float a = row[d], bb = row[d + half];
    if (head < Hq) {
        const float2 c = cs[(size_t)b * half + d];
        float* dst = q_out + (size_t)i * qd + (size_t)head * hd;
        dst[d] = (a * c.x - bb * c.y) * qscale;
        dst[d + half] = (bb * c.x + a * c.y) * qscale;
        return;
    }
    const int T = len_l[b];
    if (T >= min(slab_cap[b], cap_max)) {  // (a slab longer than the context was sized for is full at that size)
        if (head == Hq && d == 0) atomicOr(flags, FIRST_FLAG_KV_FULL);
        return;
    }
    const size_t trow = (size_t)slab_off[b] + T;
    if (head < Hq + Hkv) {
        const float2 c = cs[(size_t)b * half + d];
        KT* dst = kc + ((size_t)(head - Hq) * cap_total + trow) * hd;
        dst[d] = from_f32<KT>(a * c.x - bb * c.y);
        dst[d + half] = from_f32<KT>(bb * c.x + a * c.y);
    } else {
        KT* dst = vc + ((size_t)(head - Hq - Hkv) * cap_total + trow) * hd;
        dst[d] = from_f32<KT>(a);
        dst[d + half] = from_f32<KT>(bb);
    }
}

// act[i][f] = silu(gate) * up from gu[i] = [gate(F) | up(F)]; optional bf16 hi/lo split.
__global__ void __launch_bounds__(256) silu_mul(const float* gu, int m, const int32_t* __restrict__ m_dev, int F,
                                                float* __restrict__ act,
                                                __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo,
                                                uint64_t* stamp) {
    const Stamp stamp_guard(stamp);
    pdl_trigger();
    if (m_dev) m = min(m, __ldg(m_dev));
    pdl_wait();
    const size_t n = (size_t)m * F;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        const size_t i = e / F, f = e - i * F;
        const float g = gu[i * 2 * F + f], u = gu[i * 2 * F + F + f];
        const float y = g / (1.f + expf(-g)) * u;
        if (act) act[e] = y;
        if (hi) {
            const __nv_bfloat16 h = __float2bfloat16_rn(y);
            hi[e] = h;
            lo[e] = __float2bfloat16_rn(y - __bfloat162float(h));
        }
    }
}

// End of a step: greedy next token per row (lowest index among equal maxima) and pos += 1.
// One block of 1024 threads per row; 16-byte loads when the row allows it.
__global__ void __launch_bounds__(1024) step_end(const float* logits, int V, int32_t* __restrict__ next,
                                                 int32_t* __restrict__ pos, uint64_t* stamp) {
    const Stamp stamp_guard(stamp);
    pdl_trigger();
    pdl_wait();
    const int b = blockIdx.x;
    if (next && logits) {
        __shared__ float bv[32];
        __shared__ int bi[32];
        const float* row = logits + (size_t)b * V;
        float best = -INFINITY;
        int besti = 0x7fffffff;
        auto consider = [&](float v, int i) {
            if (v > best || (v == best && i < besti)) { best = v; besti = i; }
        };
        if ((V & 3) == 0) {
            const float4* r4 = reinterpret_cast<const float4*>(row);
#pragma unroll 4
            for (int i = threadIdx.x; i < V / 4; i += 1024) {
                const float4 v = r4[i];
                consider(v.x, 4 * i); consider(v.y, 4 * i + 1); consider(v.z, 4 * i + 2); consider(v.w, 4 * i + 3);
            }
        } else {
            for (int i = threadIdx.x; i < V; i += 1024) consider(row[i], i);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float v = __shfl_xor_sync(0xffffffffu, best, o);
            const int j = __shfl_xor_sync(0xffffffffu, besti, o);
            consider(v, j);
        }
        if ((threadIdx.x & 31) == 0) { bv[threadIdx.x >> 5] = best; bi[threadIdx.x >> 5] = besti; }
        __syncthreads();
        if (threadIdx.x < 32) {
            best = bv[threadIdx.x];
            besti = bi[threadIdx.x];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float v = __shfl_xor_sync(0xffffffffu, best, o);
                const int j = __shfl_xor_sync(0xffffffffu, besti, o);
                consider(v, j);
            }
            if (threadIdx.x == 0) next[b] = besti == 0x7fffffff ? 0 : besti;
        }
    }
    if (threadIdx.x == 0) pos[b] += 1;
}

// End of a step with sampling: next token per row by temperature + top-k sampling (the paper's
// inference settings, appendix on training and inference set-up).  The candidates are the k
// largest logits (equal values: lowest index first); token = first candidate whose cumulative
// softmax(logit / T) mass over the candidates exceeds the row's uniform draw u.  One block of
// 1024 threads per row: every thread keeps the kSampleKMax best of the elements it reads, sorted,
// in registers; k rounds of a block-wide argmax over the threads' list heads then pop the row's k
// best in order; thread 0 walks the cumulative weights (u * sum < cum, so no division).
constexpr int kSampleKMax = 16;

__device__ __forceinline__ bool sample_before(float v, int i, float w, int j) { return v > w || (v == w && i < j); }

__global__ void __launch_bounds__(1024) step_end_sample(const float* logits, int V, int k, float inv_T,
                                                        const float* __restrict__ uniforms,
                                                        int32_t* __restrict__ next, int32_t* __restrict__ pos,
                                                        uint64_t* stamp) {
    const Stamp stamp_guard(stamp);
    pdl_trigger();
    pdl_wait();
    const int b = blockIdx.x;
    __shared__ float bv[2][32];
    __shared__ int bi[2][32];
    __shared__ float cand_v[kSampleKMax];
    __shared__ int cand_i[kSampleKMax];
    const float* row = logits + (size_t)b * V;
    float tv[kSampleKMax];
    int ti[kSampleKMax];
#pragma unroll
    for (int j = 0; j < kSampleKMax; ++j) { tv[j] = -INFINITY; ti[j] = 0x7fffffff; }
    auto consider = [&](float v, int i) {
        if (sample_before(v, i, tv[kSampleKMax - 1], ti[kSampleKMax - 1])) {
            tv[kSampleKMax - 1] = v;
            ti[kSampleKMax - 1] = i;
#pragma unroll
            for (int j = kSampleKMax - 1; j > 0; --j) {
                if (sample_before(tv[j], ti[j], tv[j - 1], ti[j - 1])) {
                    const float fv = tv[j]; tv[j] = tv[j - 1]; tv[j - 1] = fv;
                    const int fi = ti[j]; ti[j] = ti[j - 1]; ti[j - 1] = fi;
                }
            }
        }
    };
    if ((V & 3) == 0 && (reinterpret_cast<uintptr_t>(logits) & 15) == 0) {
        const float4* r4 = reinterpret_cast<const float4*>(row);
        for (int i = threadIdx.x; i < V / 4; i += 1024) {
            const float4 v = r4[i];
            consider(v.x, 4 * i); consider(v.y, 4 * i + 1); consider(v.z, 4 * i + 2); consider(v.w, 4 * i + 3);
        }
    } else {
        for (int i = threadIdx.x; i < V; i += 1024) consider(row[i], i);
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int r = 0; r < k; ++r) {
        float best = tv[0];
        int besti = ti[0];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float v = __shfl_xor_sync(0xffffffffu, best, o);
            const int j = __shfl_xor_sync(0xffffffffu, besti, o);
            if (sample_before(v, j, best, besti)) { best = v; besti = j; }
        }
        if (lane == 0) { bv[r & 1][warp] = best; bi[r & 1][warp] = besti; }
        __syncthreads();
        best = bv[r & 1][lane];
        besti = bi[r & 1][lane];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float v = __shfl_xor_sync(0xffffffffu, best, o);
            const int j = __shfl_xor_sync(0xffffffffu, besti, o);
            if (sample_before(v, j, best, besti)) { best = v; besti = j; }
        }
        if (threadIdx.x == 0) { cand_v[r] = best; cand_i[r] = besti; }
        if (ti[0] == besti) {  // the owner of the winner moves on to its next best
#pragma unroll
            for (int j = 0; j + 1 < kSampleKMax; ++j) { tv[j] = tv[j + 1]; ti[j] = ti[j + 1]; }
            tv[kSampleKMax - 1] = -INFINITY;
            ti[kSampleKMax - 1] = 0x7fffffff;
        }
    }
    if (threadIdx.x == 0) {
        const float z0 = cand_v[0];
        float sum = 0.f;
        for (int j = 0; j < k; ++j) {
            const float w = j == 0 ? 1.f : expf((cand_v[j] - z0) * inv_T);
            cand_v[j] = w;
            sum += w;
        }
        const float target = uniforms[b] * sum;
        int pick = cand_i[k - 1];
        float cum = 0.f;
        for (int j = 0; j < k; ++j) {
            cum += cand_v[j];
            if (target < cum) { pick = cand_i[j]; break; }
        }
        next[b] = pick == 0x7fffffff ? 0 : pick;
        if (pos) pos[b] += 1;
    }
}

}  // namespace first
