// CUDA-core projection path for few active rows: Y[r][f] = W[f] . X[r].
// Weight-streaming GEMV: every weight element is read once from HBM with 16-byte loads
// and used for up to R rows; float32 activations and accumulation.  This is the path
// for layers whose compacted row count is too small to be a dense contraction.
#pragma once
#include "common.cuh"

namespace first {

enum GemvEpilogue { kStore = 0, kScatterAdd = 1 };

// One warp per output feature, grid-stride over features.  X rows [r0, r0+R) of the
// compact activation matrix (row stride K) stay in L1/L2.  rows_valid <= R rows are live.
//   kStore:      Y[(r0+r)*ldy + f]      = dot
//   kScatterAdd: Y[idx[r0+r]*ldy + f]  += dot   (each element owned by one lane: no atomics)
template <typename WT, int R, int EPI>
__global__ void __launch_bounds__(256) gemv_rows(const WT* __restrict__ W, int n_out, int K,
                                                 const float* X, int r0, int rows_valid,
                                                 const int32_t* __restrict__ m_dev,
                                                 float* __restrict__ Y, int64_t ldy, const int32_t* __restrict__ idx,
                                                 uint64_t* stamp) {
    const Stamp stamp_guard(stamp);
    pdl_trigger();
    // m_dev: the active-row count in device memory (the host launches for an upper bound of it)
    if (m_dev) rows_valid = min(rows_valid, __ldg(m_dev) - r0);
    pdl_wait();
    if (rows_valid <= 0) return;
    const int lane = threadIdx.x & 31;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int nwarps = (gridDim.x * blockDim.x) >> 5;
    const float* xr[R];
#pragma unroll
    for (int r = 0; r < R; ++r) xr[r] = X + (size_t)(r0 + (r < rows_valid ? r : 0)) * K;

    for (int f = warp; f < n_out; f += nwarps) {
        const WT* wrow = W + (size_t)f * K;
        float acc[R];
#pragma unroll
        for (int r = 0; r < R; ++r) acc[r] = 0.f;
#pragma unroll 2
        for (int k = lane * 8; k < K; k += 256) {
            float wv[8];
            Load8<WT>::ld_stream(wrow + k, wv);
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const float4 a = __ldg(reinterpret_cast<const float4*>(xr[r] + k));
                const float4 b = __ldg(reinterpret_cast<const float4*>(xr[r] + k) + 1);
                acc[r] = fmaf(wv[0], a.x, acc[r]); acc[r] = fmaf(wv[1], a.y, acc[r]);
                acc[r] = fmaf(wv[2], a.z, acc[r]); acc[r] = fmaf(wv[3], a.w, acc[r]);
                acc[r] = fmaf(wv[4], b.x, acc[r]); acc[r] = fmaf(wv[5], b.y, acc[r]);
                acc[r] = fmaf(wv[6], b.z, acc[r]); acc[r] = fmaf(wv[7], b.w, acc[r]);
            }
        }
#pragma unroll
        for (int r = 0; r < R; ++r) acc[r] = warp_sum(acc[r]);
        if (lane == 0) {
#pragma unroll
            for (int r = 0; r < R; ++r) {
                if (r < rows_valid) {
                    if (EPI == kStore) Y[(size_t)(r0 + r) * ldy + f] = acc[r];
                    else Y[(size_t)idx[r0 + r] * ldy + f] += acc[r];
                }
            }
        }
    }
}

}  // namespace first
