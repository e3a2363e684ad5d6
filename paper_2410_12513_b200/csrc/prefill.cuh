// Batched prompt processing ("Inference for FiRST", item 1: no layer is skipped on the prompt;
// "Adaptive Router Module": router i reads the hidden states entering layer i for every prompt
// token).  The prompt tokens of a ragged batch go through the step kernels a chunk at a time,
// every token as a row of its own: row r of a chunk is (sequence b, position p), its cache
// slab is the slab of b, its cache length is p.  These kernels build those per-row tables,
// keep the last prompt token's residual of every sequence, and set len/pos at the end.
#pragma once
#include "common.cuh"
#include "first.h"

namespace first {

// Sequence that owns flat token g: the largest b with cu[b] <= g (cu strictly increasing).
__device__ __forceinline__ int seq_of_token(const int32_t* __restrict__ cu, int B, int g) {
    int lo = 0, hi = B;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (cu[mid] <= g) lo = mid; else hi = mid;
    }
    return lo;
}

// Row tables of the chunk that holds flat tokens g0 .. g0+rows-1.  v_len is [L][rows].
static __global__ void __launch_bounds__(128) prefill_rows(const int32_t* __restrict__ tokens, const int32_t* __restrict__ cu,
                                                           int B, int g0, int rows, int L,
                                                           const int64_t* __restrict__ slab_off,
                                                           const int32_t* __restrict__ slab_cap,
                                                           int32_t* __restrict__ v_tok, int64_t* __restrict__ v_off,
                                                           int32_t* __restrict__ v_cap, int32_t* __restrict__ v_pos,
                                                           int32_t* __restrict__ v_len) {
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= rows) return;
    const int g = g0 + r, b = seq_of_token(cu, B, g), p = g - cu[b];
    v_tok[r] = tokens[g];
    v_off[r] = slab_off[b];
    v_cap[r] = slab_cap[b];
    v_pos[r] = p;
    for (int l = 0; l < L; ++l) v_len[(size_t)l * rows + r] = p;
}

// After a chunk's last layer: the residual of a sequence's last prompt token is what the
// final norm and lm_head read.  One block per row of the chunk.
static __global__ void __launch_bounds__(256) prefill_keep_last(const float* __restrict__ x, const int32_t* __restrict__ cu,
                                                                int B, int g0, int D, float* __restrict__ x_last) {
    const int g = g0 + blockIdx.x, b = seq_of_token(cu, B, g);
    if (g != cu[b + 1] - 1) return;
    const float4* src = reinterpret_cast<const float4*>(x + (size_t)blockIdx.x * D);
    float4* dst = reinterpret_cast<float4*>(x_last + (size_t)b * D);
    for (int k = threadIdx.x; k < D / 4; k += blockDim.x) dst[k] = src[k];
}

// End of the prompt: every layer of sequence b holds its n_b prompt tokens, and the next token
// fed has position n_b.  A slab shorter than the prompt was flagged full when it overflowed.
static __global__ void __launch_bounds__(128) prefill_finish(const int32_t* __restrict__ cu, int B, int L,
                                                             const int32_t* __restrict__ slab_cap,
                                                             int32_t* __restrict__ len, int32_t* __restrict__ pos) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int n = cu[b + 1] - cu[b];
    pos[b] = n;
    const int have = min(n, slab_cap[b]);
    for (int l = 0; l < L; ++l) len[(size_t)l * B + b] = have;
}

}  // namespace first
