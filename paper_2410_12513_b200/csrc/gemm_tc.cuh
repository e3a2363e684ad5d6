// Tensor-core projection path (tcgen05 + TMEM + TMA) for layers with enough active rows
// to make the projection a dense contraction:  Y[j][f] (+)= sum_k W[f][k] * X[j][k].
//
// "Swap-AB": the weight matrix is the 128-row M operand, streamed once from HBM by TMA into
// 128-byte-swizzled shared memory; the compacted activations (m rows, padded to a multiple
// of 16) are the N operand; the float32 accumulator tile [128 features][N rows] lives in
// tensor memory.  Activations arrive as a bfloat16 hi/lo pair (x = hi + lo to 2^-17), and
// each weight tile is multiplied by both halves into the same accumulator, so the result
// keeps float32-grade activations while the weights stay bfloat16.
//
// Work unit = (128-feature tile, K range).  With several K ranges per tile the partial sums
// meet in global memory through float32 reductions (red.global.add).
// The gate/up projection has its own epilogue: its tile is 64 gate rows stacked on the matching
// 64 up rows (two TMA boxes), the whole K range in one CTA, and the epilogue applies
// silu(gate)*up in registers and writes the activation (and its hi/lo split) directly.
// Roles inside a CTA of 10 warps: warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer,
// warps 2..9 = epilogue (two per TMEM lane quadrant, alternate 16-column chunks).  Every wait is bounded.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "first.h"

namespace first {
namespace tc {

constexpr int kBlockM = 128;  // weight rows (output features) per tile
constexpr int kBlockK = 64;   // bf16 elements per 128-byte swizzle row
constexpr int kUmmaK = 16;
constexpr int kABytes = kBlockM * kBlockK * 2;
constexpr uint32_t kSpinLimit = 1u << 22;

enum Epilogue { kEpiStore = 0, kEpiAtomic = 1, kEpiScatterAtomic = 2, kEpiSwiglu = 3 };

struct GemmParams {
    int n_out, K, m, n_pad;
    int kblocks, ksplit;
    int stages, tmem_cols, use_lo;
    int mt;        // 128-row weight tiles per CTA (1 or 2): two tiles share every activation tile, which
                   // halves the activation bytes pulled from L2 per weight byte when there are many rows
    int acc_cols;  // TMEM columns per accumulator (power of two >= n_pad)
    float* Y;
    int64_t ldy;
    const int32_t* idx;
    uint32_t* flags;
    // kEpiSwiglu: the weight matrix is [gate rows (n_out) | up rows (n_out)]; a tile pairs 64 gate
    // features with the same 64 up features and the epilogue writes silu(gate)*up:
    int pair_rows;           // gate rows (= up rows) per tile when mt == 1: at most 64, chosen so that the
                             // tiles fill the GPU's CTA slots in one wave
    float* act;              // [m][n_out] float32 or NULL
    __nv_bfloat16* act_hi;   // [m][n_out] bfloat16 hi/lo split or NULL
    __nv_bfloat16* act_lo;
    uint64_t* stamp;         // in-step timing slot or NULL
    const int32_t* m_dev;    // active-row count in device memory (m is a host-side upper bound of it) or NULL
    int row0;                // first compact row of this launch (launches take 256 rows each)
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after kSpinLimit polls (or when another role already gave up),
// raising the CTA's abort word and the device flag.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_s, uint32_t* flags,
                                          uint32_t limit = kSpinLimit) {
    for (uint32_t it = 0; it < limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 255u) == 255u && *abort_s) return false;
    }
    *abort_s = 1;
    atomicOr(flags, FIRST_FLAG_WAIT_EXPIRED);
    return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                                 uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1, {%3, %4}], [%2], %5;"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "l"(policy) : "memory");
}

// Shared-memory matrix descriptor, K-major operand in 128-byte-swizzled rows:
// start address >> 4, stride between 8-row groups = 1024 bytes, descriptor version 1,
// swizzle mode 2 (128 B).  The leading-dimension field is unused for this layout.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptor for kind::f16: D = f32, A = B = bf16, both K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t instr_desc_bf16(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kBlockM >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Dynamic shared memory: [stages][A mt*16 KB | B_hi n_pad*128 | B_lo n_pad*128] (1024-aligned), then barriers.
template <int EPI>
__global__ void __launch_bounds__(320) gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA,
                                                      const __grid_constant__ CUtensorMap tmA2,
                                                      const __grid_constant__ CUtensorMap tmBh,
                                                      const __grid_constant__ CUtensorMap tmBl, const GemmParams p) {
    const Stamp stamp_guard(p.stamp);
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int b_bytes = p.n_pad * 128;
    const int a_bytes = kABytes * p.mt;
    const int stage_bytes = a_bytes + b_bytes * (p.use_lo ? 2 : 1);
    const uint32_t bars = base + (uint32_t)p.stages * stage_bytes;  // full[S], empty[S], tmem_full : 8 B each
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (p.stages + s); };
    const uint32_t tmem_full_bar = bars + 16u * p.stages;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ int idx_s[256];  // active-row list of the scattering epilogue

    pdl_trigger();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tile = blockIdx.x / p.ksplit, split = blockIdx.x - tile * p.ksplit;
    const int kb0 = (int)((int64_t)p.kblocks * split / p.ksplit), kb1 = (int)((int64_t)p.kblocks * (split + 1) / p.ksplit);
    const int nkb = kb1 - kb0;

    // Thread 0 is the TMA producer.  It sets the barriers up and at once asks for the first weight tiles:
    // they depend neither on the previous kernel nor on the rest of this CTA's set-up (TMEM allocation, the
    // CTA-wide barrier), so HBM is already streaming while those happen.
    uint64_t pol_stream = 0;
    const uint32_t tx = (EPI == kEpiSwiglu && p.mt == 1)
                            ? (uint32_t)(stage_bytes - a_bytes + 2 * p.pair_rows * 128)  // two boxes of R rows
                            : (uint32_t)stage_bytes;
    auto load_a = [&](uint32_t sa, uint32_t bar, int kc) {
        if (EPI == kEpiSwiglu) {
            // gate rows, then the matching up rows: R+R (mt = 1, R = pair_rows <= 64) or 128+128 (mt = 2)
            const int rows = p.mt == 1 ? p.pair_rows : 128;
            const CUtensorMap* tm = p.mt == 1 ? &tmA : &tmA2;
            tma_load_2d_hint(sa, tm, bar, kc, tile * rows, pol_stream);
            tma_load_2d_hint(sa + rows * 128, tm, bar, kc, p.n_out + tile * rows, pol_stream);
        } else {
            for (int a = 0; a < p.mt; ++a)
                tma_load_2d_hint(sa + a * kABytes, &tmA, bar, kc, (tile * p.mt + a) * kBlockM, pol_stream);
        }
    };
    const int npre = min(p.stages, nkb);
    if (threadIdx.x == 0) {
        abort_s = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(tmem_full_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
        for (int i = 0; i < npre; ++i) {
            mbar_expect_tx(full_bar(i), tx);
            load_a(base + (uint32_t)i * stage_bytes, full_bar(i), (kb0 + i) * kBlockK);
        }
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmBh) : "memory");
        if (p.use_lo) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmBl) : "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_s)), "r"((uint32_t)p.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_d = tmem_base_s;

    if (warp == 0) {
        if (lane == 0) {
            // The ring already holds requests for the first weight tiles (set-up above): wait for the
            // previous kernel and add the activation tiles to the same stages.
            pdl_wait();
            for (int i = 0; i < npre; ++i) {
                const uint32_t sa = base + (uint32_t)i * stage_bytes;
                tma_load_2d(sa + a_bytes, &tmBh, full_bar(i), (kb0 + i) * kBlockK, 0);
                if (p.use_lo) tma_load_2d(sa + a_bytes + b_bytes, &tmBl, full_bar(i), (kb0 + i) * kBlockK, 0);
            }
            int issued = npre;
            for (int i = npre; i < nkb; ++i, ++issued) {
                const int s = i % p.stages;
                const uint32_t ph = (uint32_t)(i / p.stages) & 1u;
                if (!mbar_wait(empty_bar(s), ph ^ 1u, &abort_s, p.flags)) break;
                const uint32_t sa = base + (uint32_t)s * stage_bytes;
                mbar_expect_tx(full_bar(s), tx);
                const int kc = (kb0 + i) * kBlockK;
                load_a(sa, full_bar(s), kc);
                tma_load_2d(sa + a_bytes, &tmBh, full_bar(s), kc, 0);
                if (p.use_lo) tma_load_2d(sa + a_bytes + b_bytes, &tmBl, full_bar(s), kc, 0);
            }
            // This lane does not reach the CTA's final barrier before every copy it issued has landed (the last
            // use of each stage; earlier uses were consumed before their stage was refilled).  It does so
            // whether or not any role has given up and whichever role notices first: the CTA's shared memory
            // can therefore never be handed to another CTA with a copy still in flight.  In a normal run the
            // consumers wait for the same barriers anyway, so this costs nothing.
            for (int i = max(0, issued - p.stages); i < issued; ++i) {
                const uint32_t bar = full_bar(i % p.stages), ph = (uint32_t)(i / p.stages) & 1u;
                for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(bar, ph); ++it) {}
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = instr_desc_bf16(p.n_pad);
            bool ok = true;
            for (int i = 0; i < nkb && ok; ++i) {
                const int s = i % p.stages;
                const uint32_t ph = (uint32_t)(i / p.stages) & 1u;
                ok = mbar_wait(full_bar(s), ph, &abort_s, p.flags);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t sa = base + (uint32_t)s * stage_bytes;
                const uint64_t dbh = smem_desc_sw128(sa + a_bytes), dbl = smem_desc_sw128(sa + a_bytes + b_bytes);
                for (int a = 0; a < p.mt; ++a) {
                    const uint64_t da = smem_desc_sw128(sa + a * kABytes);
                    const uint32_t td = tmem_d + (uint32_t)(a * p.acc_cols);
#pragma unroll
                    for (int k = 0; k < kBlockK / kUmmaK; ++k)
                        umma_bf16(td, da + 2u * k, dbh + 2u * k, idesc, (i > 0 || k > 0) ? 1u : 0u);
                    if (p.use_lo) {
#pragma unroll
                        for (int k = 0; k < kBlockK / kUmmaK; ++k) umma_bf16(td, da + 2u * k, dbl + 2u * k, idesc, 1u);
                    }
                }
                umma_commit(empty_bar(s));  // frees the stage once these MMAs have read it
            }
            umma_commit(tmem_full_bar);  // accumulator complete (arrives even after a failed wait)
        }
    } else {
        // Epilogue: 8 warps.  Warp w reads TMEM lanes 32*(w%4) .. +31 (its quadrant); the two warps of a
        // quadrant take alternate 16-column chunks of the accumulator.
        const int quad = warp & 3, half = (warp - 2) >> 2;
        if (EPI == kEpiScatterAtomic) {  // the active-row list is fixed between first_set_mask calls
            for (int e = (int)threadIdx.x - 64; e < p.m; e += 256) idx_s[e] = p.idx[e];
            asm volatile("bar.sync 1, 256;" ::: "memory");
        }
        pdl_wait();  // the epilogue reduces into buffers the previous kernels own
        // rows that exist: the columns beyond them were computed from stale activation rows and are dropped
        const int m_act = p.m_dev ? max(0, min(p.m, __ldg(p.m_dev) - p.row0)) : p.m;
        const bool ok = mbar_wait(tmem_full_bar, 0u, &abort_s, p.flags) && !abort_s;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const bool run = ok && nkb > 0;
        if (EPI == kEpiSwiglu && p.mt == 2) {
            // accumulator 0 = 128 gate features, accumulator 1 = the same 128 up features: no exchange needed
            const int f = tile * 128 + quad * 32 + lane;
            const uint32_t lane_addr = tmem_d + ((uint32_t)(quad * 32) << 16);
            if (run) {
                for (int c0 = half * 16; c0 < p.n_pad; c0 += 32) {
                    uint32_t vg[16], vu[16];
                    tmem_ld16(lane_addr + (uint32_t)c0, vg);
                    tmem_ld16(lane_addr + (uint32_t)(p.acc_cols + c0), vu);
                    if (f < p.n_out) {
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            const int j = c0 + c;
                            if (j < m_act) {
                                const float g = __uint_as_float(vg[c]);
                                const float y = g / (1.f + expf(-g)) * __uint_as_float(vu[c]);
                                const size_t o = (size_t)j * p.n_out + f;
                                if (p.act) p.act[o] = y;
                                if (p.act_hi) {
                                    const __nv_bfloat16 h = __float2bfloat16_rn(y);
                                    p.act_hi[o] = h;
                                    p.act_lo[o] = __float2bfloat16_rn(y - __bfloat162float(h));
                                }
                            }
                        }
                    }
                }
            }
        } else if (EPI == kEpiSwiglu) {
            // Lanes [0, R) of the accumulator hold gate features, lanes [R, 2R) the matching up features
            // (R = pair_rows; lanes from 2R up saw stale shared memory and are ignored).  Per 16-column
            // chunk every lane loads its values once; up lanes park theirs in a small double buffer in
            // shared memory (the ring is idle once the accumulator is complete), the four warps of this
            // half meet at a named barrier, and gate lanes combine.  u[column][feature]: conflict-free.
            const int R = p.pair_rows;
            float* u_s = reinterpret_cast<float*>(smem_raw + (base - smem_u32(smem_raw))) + half * (2 * 16 * 64);
            const uint32_t lane_addr = tmem_d + ((uint32_t)(quad * 32) << 16);
            const int gl = quad * 32 + lane;  // accumulator lane of this thread
            const int f = tile * R + gl;
            int k = 0;
            for (int c0 = half * 16; c0 < p.n_pad; c0 += 32, ++k) {  // every thread of the half takes every trip
                uint32_t v[16];
                tmem_ld16(lane_addr + (uint32_t)c0, v);
                float* ub = u_s + (k & 1) * (16 * 64);
                if (gl >= R && gl < 2 * R) {
#pragma unroll
                    for (int c = 0; c < 16; ++c) ub[c * 64 + (gl - R)] = __uint_as_float(v[c]);
                }
                if (half == 0) asm volatile("bar.sync 2, 128;" ::: "memory");
                else asm volatile("bar.sync 3, 128;" ::: "memory");
                if (run && gl < R && f < p.n_out) {
#pragma unroll
                    for (int c = 0; c < 16; ++c) {
                        const int j = c0 + c;
                        if (j < m_act) {
                            const float g = __uint_as_float(v[c]);
                            const float y = g / (1.f + expf(-g)) * ub[c * 64 + gl];
                            const size_t o = (size_t)j * p.n_out + f;
                            if (p.act) p.act[o] = y;
                            if (p.act_hi) {
                                const __nv_bfloat16 h = __float2bfloat16_rn(y);
                                p.act_hi[o] = h;
                                p.act_lo[o] = __float2bfloat16_rn(y - __bfloat162float(h));
                            }
                        }
                    }
                }
            }
        } else if (run) {
            for (int a = 0; a < p.mt; ++a) {
                const int f = (tile * p.mt + a) * kBlockM + quad * 32 + lane;
                const uint32_t lane_addr = tmem_d + ((uint32_t)(quad * 32) << 16) + (uint32_t)(a * p.acc_cols);
                for (int c0 = half * 16; c0 < p.n_pad; c0 += 32) {
                    uint32_t v[16];
                    tmem_ld16(lane_addr + (uint32_t)c0, v);
                    if (f < p.n_out) {
#pragma unroll
                        for (int c = 0; c < 16; ++c) {
                            const int j = c0 + c;
                            if (j < m_act) {
                                const float val = __uint_as_float(v[c]);
                                if (EPI == kEpiStore) p.Y[(size_t)j * p.ldy + f] = val;
                                else if (EPI == kEpiAtomic) atomicAdd(p.Y + (size_t)j * p.ldy + f, val);
                                else atomicAdd(p.Y + (size_t)idx_s[j] * p.ldy + f, val);
                            }
                        }
                    }
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        // After a failed wait the epilogue may have left without seeing the accumulator complete: the MMAs that
        // were issued (their operands had landed, so they finish) must be done before the tensor memory and the
        // shared memory they use are given back.  The commit above arrives on this barrier once they are.
        if (abort_s && lane == 0)
            for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(tmem_full_bar, 0u); ++it) {}
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"((uint32_t)p.tmem_cols)
                     : "memory");
    }
}

// Exercises the give-up path of mbar_wait without any copy in flight: a barrier that expects one arrival
// which never comes.  The wait runs out after `limit` polls, raises the abort word and the device flag, and
// the kernel returns normally.  out[0] = what the wait returned, out[1] = the abort word.
static __global__ void wait_expiry_selftest(uint32_t limit, uint32_t* flags, int32_t* out) {
    __shared__ uint64_t bar;
    __shared__ int abort_s;
    if (threadIdx.x == 0) {
        abort_s = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const bool ok = mbar_wait(smem_u32(&bar), 0u, &abort_s, flags, limit);
        out[0] = ok ? 1 : 0;
        out[1] = abort_s;
    }
}

}  // namespace tc
}  // namespace first
