// Shared device helpers for the routed decode step kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace first {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Programmatic dependent launch: let the next kernel of the stream start its prologue while
// this one runs, and wait for the previous kernel's results (both are no-ops when the launch
// carries no programmatic dependency).
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
// Everything an earlier kernel of the step produced must be read after this wait.  The "memory" clobber
// keeps ordinary loads below it, but not loads the compiler may treat as invariant (a const __restrict__
// kernel parameter): pointers to data produced inside a step therefore carry no __restrict__.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// In-step timing aid (off unless asked for): every CTA folds its entry time into the launch's
// first-start word and every warp its exit time into the launch's last-end word, both read from
// the global nanosecond timer.  `slot` points at the start word; the end word sits kStampCap
// words further on.  A null slot costs one predictable branch.
constexpr int kStampCap = 2048;
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
struct Stamp {
    unsigned long long* slot;
    __device__ __forceinline__ explicit Stamp(uint64_t* s) : slot(reinterpret_cast<unsigned long long*>(s)) {
        if (slot && threadIdx.x == 0 && threadIdx.y == 0) atomicMin(slot, global_ns());
    }
    __device__ __forceinline__ ~Stamp() {
        if (slot && (threadIdx.x & 31) == 0) atomicMax(slot + kStampCap, global_ns());
    }
};

// two packed bfloat16 -> two float32 (a bfloat16 is the upper half of a float32)
__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

__device__ __forceinline__ void unpack8(const uint4& u, float (&f)[8]) {
    f[0] = bf_lo(u.x); f[1] = bf_hi(u.x); f[2] = bf_lo(u.y); f[3] = bf_hi(u.y);
    f[4] = bf_lo(u.z); f[5] = bf_hi(u.z); f[6] = bf_lo(u.w); f[7] = bf_hi(u.w);
}

// Load 8 consecutive elements (16-byte aligned for bf16, 32-byte for f32) as float32.
template <typename T>
struct Load8;
template <>
struct Load8<__nv_bfloat16> {
    static __device__ __forceinline__ void ld(const __nv_bfloat16* p, float (&f)[8]) {
        uint4 u = __ldg(reinterpret_cast<const uint4*>(p));
        unpack8(u, f);
    }
    // streaming variant: data read once per step, kept out of L1
    static __device__ __forceinline__ void ld_stream(const __nv_bfloat16* p, float (&f)[8]) {
        uint4 u;
        asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(u.x), "=r"(u.y), "=r"(u.z), "=r"(u.w) : "l"(p));
        unpack8(u, f);
    }
};
template <>
struct Load8<float> {
    static __device__ __forceinline__ void ld(const float* p, float (&f)[8]) {
        float4 a = __ldg(reinterpret_cast<const float4*>(p));
        float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
        f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
    }
    static __device__ __forceinline__ void ld_stream(const float* p, float (&f)[8]) { ld(p, f); }
};

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

}  // namespace first
