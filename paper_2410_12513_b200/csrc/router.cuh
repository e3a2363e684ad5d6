// Router scoring (Sec. "Adaptive Router Module") and the per-layer active-row plan.
#pragma once
#include "common.cuh"
#include "first.h"

namespace first {

// Pass 1: one float per prompt token.  z = w . h (+ bias); mode 0 stores sigmoid(z),
// mode 1 stores z.  HBM-bound: every hidden element is read exactly once, 16 bytes per
// lane per load; one warp per token, grid-stride over tokens.  Dynamic smem: D floats.
template <typename HT>
__global__ void __launch_bounds__(256) router_token_scores(const HT* __restrict__ hidden, int64_t n_tokens, int D,
                                                           const float* __restrict__ w, const float* __restrict__ bias,
                                                           int mode, float* __restrict__ tok) {
    extern __shared__ float w_s[];
    for (int i = threadIdx.x; i < D; i += blockDim.x) w_s[i] = w[i];
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, wpb = blockDim.x >> 5;
    const float b = bias ? bias[0] : 0.f;
    for (int64_t t = (int64_t)blockIdx.x * wpb + warp; t < n_tokens; t += (int64_t)gridDim.x * wpb) {
        const HT* h = hidden + t * D;
        float acc = 0.f;
#pragma unroll 4
        for (int k = lane * 8; k < D; k += 256) {
            float f[8];
            Load8<HT>::ld_stream(h + k, f);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc = fmaf(f[e], w_s[k + e], acc);
        }
        acc = warp_sum(acc);
        if (lane == 0) {
            const float z = acc + b;
            tok[t] = (mode == FIRST_ROUTER_MEAN_OF_SIGMOID) ? 1.f / (1.f + expf(-z)) : z;
        }
    }
}

// Pass 2: one block per sequence; float64 mean in a fixed order (strided partial sums
// then a fixed tree), sigmoid for mode 1, threshold with ">=".
// The sequence table comes from the caller: a row range that leaves [0, n_tokens] (the token
// scores pass 1 wrote), or runs backwards, is never followed -- the block raises
// FIRST_FLAG_BAD_SEQ_TABLE and writes nothing; an empty range raises FIRST_FLAG_EMPTY_SEQ.
static __global__ void __launch_bounds__(256) router_finalize(const float* __restrict__ tok, const int32_t* __restrict__ cu,
                                                       int64_t n_tokens, int L, int layer, int mode, float tau,
                                                       uint8_t* __restrict__ mask, float* __restrict__ scores,
                                                       uint32_t* __restrict__ flags) {
    __shared__ double part[256];
    const int b = blockIdx.x;
    const int lo = cu[b], hi = cu[b + 1];
    if (lo < 0 || hi < lo || (int64_t)hi > n_tokens) {  // uniform over the block
        if (threadIdx.x == 0) atomicOr(flags, FIRST_FLAG_BAD_SEQ_TABLE);
        return;
    }
    double s = 0.0;
    for (int j = lo + threadIdx.x; j < hi; j += 256) s += (double)tok[j];
    part[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) part[threadIdx.x] += part[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        if (hi == lo) {
            atomicOr(flags, FIRST_FLAG_EMPTY_SEQ);
            return;
        }
        const double mean = part[0] / (double)(hi - lo);
        const double rho = (mode == FIRST_ROUTER_MEAN_OF_SIGMOID) ? mean : 1.0 / (1.0 + exp(-mean));
        mask[(size_t)b * L + layer] = (rho >= (double)tau) ? 1 : 0;
        if (scores) scores[(size_t)b * L + layer] = (float)rho;
    }
}

// Active-row compaction: one warp per layer walks the batch 32 rows at a time; a ballot
// gives the keep bits, popc of the lower lanes the position inside the chunk, a running
// base the position in the list.  idx[l] = ascending active rows (rest -1), cnt[l],
// slot[l][b] = position of b in idx[l] or -1.
static __global__ void __launch_bounds__(32) plan_compact(const uint8_t* __restrict__ mask, int B, int L,
                                                   int32_t* __restrict__ idx, int32_t* __restrict__ cnt,
                                                   int32_t* __restrict__ slot, uint32_t* __restrict__ flags) {
    const int l = blockIdx.x, lane = threadIdx.x;
    int base = 0;
    for (int b0 = 0; b0 < B; b0 += 32) {
        const int b = b0 + lane;
        const uint8_t mk = (b < B) ? mask[(size_t)b * L + l] : 0;
        if (mk > 1) atomicOr(flags, FIRST_FLAG_BAD_MASK);
        const bool keep = mk == 1;
        const uint32_t bal = __ballot_sync(0xffffffffu, keep);
        const int p = base + __popc(bal & ((1u << lane) - 1u));
        if (b < B) {
            slot[(size_t)l * B + b] = keep ? p : -1;
            if (keep) idx[(size_t)l * B + p] = b;
        }
        base += __popc(bal);
    }
    for (int i = base + lane; i < B; i += 32) idx[(size_t)l * B + i] = -1;
    if (lane == 0) cnt[l] = base;
}

}  // namespace first
