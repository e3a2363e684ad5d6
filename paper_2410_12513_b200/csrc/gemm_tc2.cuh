// Tensor-core projections for MANY active rows (from about 96 up to 256): two CTAs on one tile pair.
//
// With many rows the single-CTA kernel (gemm_tc.cuh) stops being bound by the weight stream: every CTA pulls,
// for each 16 KB weight tile, the whole hi/lo activation tile (up to 64 KB) from L2, one pipeline stage grows to
// 64..96 KB, the ring is two deep and the tensor pipe waits for shared-memory fills half of the time.  Here a
// cluster of two CTAs (a CTA pair on neighbouring SMs) works on one unit: `tcgen05.mma.cta_group::2` multiplies
// a 256-row weight tile (128 rows in each CTA's shared memory) by the activation tile whose rows are split between
// the two CTAs, so each SM fetches only HALF of the activation bytes per weight byte and a stage shrinks to
// 56..64 KB (three to four stages in flight).  Each CTA keeps the accumulator rows of its own 128 weight rows in
// its own tensor memory and runs the same epilogues as the single-CTA kernel on them.
//
// Who does what.  Both CTAs: warp 0 lane 0 loads its own weight rows and its own half of the activation rows (plain
// TMA loads, no multicast; the loads of BOTH CTAs report their bytes to the full barrier of the pair's first CTA,
// the "leader").  Leader only: warp 1 lane 0 waits for that barrier and issues the MMAs for the pair; a multicast
// commit then frees the stage in both CTAs, and a last one tells both epilogues that the accumulators are complete.
// Warps 2..9 of each CTA: epilogue.  Tensor memory is allocated and freed by warp 1 of each CTA (cta_group::2
// form); the two CTAs meet at a cluster barrier before freeing it, so neither leaves while its partner may
// still touch its shared memory, tensor memory or barriers.  Every mbarrier wait is bounded.
#pragma once
#include "gemm_tc.cuh"

namespace first {
namespace tc2 {

using tc::GemmParams;
using tc::kABytes;
using tc::kBlockK;
using tc::kBlockM;
using tc::kSpinLimit;
using tc::kUmmaK;
using tc::mbar_init;
using tc::mbar_try_wait;
using tc::mbar_wait;
using tc::smem_desc_sw128;
using tc::smem_u32;
using tc::tmem_ld16;

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory object in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// TMA load whose completion is reported to a barrier that may live in the partner CTA (cta_group::2 form)
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster, int c0,
                                                      int c1, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1, {%3, %4}], [%2], %5;"
        ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(c0), "r"(c1), "l"(policy) : "memory");
}
// Instruction descriptor, kind::f16 across a CTA pair: D = f32, A = B = bf16, K-major, M = 256, N = n.
__device__ __forceinline__ uint32_t instr_desc_bf16_m256(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}
__device__ __forceinline__ void umma2_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
}
// arrives, once the MMAs issued so far are done, on the barrier at this shared-memory offset in BOTH CTAs of the pair
__device__ __forceinline__ void umma2_commit_both(uint32_t bar) {
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(bar), "h"((uint16_t)3) : "memory");
}

// Launched with cluster dimension (2,1,1); grid.x = 2 * units; 320 threads.  Work unit = (tile group, K range):
// a tile group is p.mt weight tiles of 256 rows (128 per CTA); the activation tile has p.n_pad rows (a multiple
// of 32), half of them in each CTA.  Shared memory per stage and CTA: [A: mt x 16 KB | B_hi: n_pad/2 x 128 B | B_lo].
// Epilogues: kEpiStore / kEpiAtomic / kEpiScatterAtomic as in gemm_tc_kernel; kEpiSwiglu with mt == 2 only
// (accumulator 0 = 256 gate features, accumulator 1 = the same 256 up features).  tmB maps have a box of n_pad/2 rows.
template <int EPI>
__global__ void __launch_bounds__(320) gemm_tc2_kernel(const __grid_constant__ CUtensorMap tmA,
                                                       const __grid_constant__ CUtensorMap tmBh,
                                                       const __grid_constant__ CUtensorMap tmBl, const GemmParams p) {
    const Stamp stamp_guard(p.stamp);
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int half_rows = p.n_pad >> 1;
    const int b_bytes = half_rows * 128;
    const int a_bytes = kABytes * p.mt;
    const int stage_bytes = a_bytes + b_bytes * (p.use_lo ? 2 : 1);
    const uint32_t bars = base + (uint32_t)p.stages * stage_bytes;  // full[S], empty[S], tmem_full : 8 B each
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (p.stages + s); };
    const uint32_t tmem_full_bar = bars + 16u * p.stages;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ int idx_s[256];

    pdl_trigger();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();  // 0 = leader of the pair
    const int unit = blockIdx.x >> 1;
    const int tile = unit / p.ksplit, split = unit - tile * p.ksplit;
    const int kb0 = (int)((int64_t)p.kblocks * split / p.ksplit), kb1 = (int)((int64_t)p.kblocks * (split + 1) / p.ksplit);
    const int nkb = kb1 - kb0;

    // weight row of (accumulator a, this CTA's lane 0)
    auto row_of = [&](int a) {
        if (EPI == tc::kEpiSwiglu) return (a == 0 ? 0 : p.n_out) + tile * 256 + (int)rank * 128;
        return (tile * p.mt + a) * 256 + (int)rank * 128;
    };
    uint64_t pol_stream = 0;
    const uint32_t tx_pair = 2u * (uint32_t)stage_bytes;  // bytes both CTAs bring into a stage
    auto load_a = [&](uint32_t sa, uint32_t bar_leader, int kc) {
        for (int a = 0; a < p.mt; ++a) tma_load_2d_pair_hint(sa + a * kABytes, &tmA, bar_leader, kc, row_of(a), pol_stream);
    };
    const int npre = min(p.stages, nkb);
    if (threadIdx.x == 0) {
        abort_s = 0;
        // full: one arrival (the leader's producer, with the byte count of both CTAs); empty: one arrival (the commit)
        for (int s = 0; s < p.stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(tmem_full_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_s)), "r"((uint32_t)p.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    // both CTAs' barriers exist before either CTA's copies or commits can reach them
    cluster_sync_all();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_d = tmem_base_s;

    if (warp == 0) {
        if (lane == 0) {
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
            // The first weight tiles depend on nothing that precedes this kernel: ask for them before the wait.
            for (int i = 0; i < npre; ++i) {
                if (rank == 0) tc::mbar_expect_tx(full_bar(i), tx_pair);
                load_a(base + (uint32_t)i * stage_bytes, mapa(full_bar(i), 0), (kb0 + i) * kBlockK);
            }
            pdl_wait();
            for (int i = 0; i < npre; ++i) {
                const uint32_t sa = base + (uint32_t)i * stage_bytes, fb = mapa(full_bar(i), 0);
                tma_load_2d_pair(sa + a_bytes, &tmBh, fb, (kb0 + i) * kBlockK, (int)rank * half_rows);
                if (p.use_lo) tma_load_2d_pair(sa + a_bytes + b_bytes, &tmBl, fb, (kb0 + i) * kBlockK, (int)rank * half_rows);
            }
            int issued = npre;
            for (int i = npre; i < nkb; ++i, ++issued) {
                const int s = i % p.stages;
                const uint32_t ph = (uint32_t)(i / p.stages) & 1u;
                if (!mbar_wait(empty_bar(s), ph ^ 1u, &abort_s, p.flags)) break;
                const uint32_t sa = base + (uint32_t)s * stage_bytes, fb = mapa(full_bar(s), 0);
                if (rank == 0) tc::mbar_expect_tx(full_bar(s), tx_pair);
                const int kc = (kb0 + i) * kBlockK;
                load_a(sa, fb, kc);
                tma_load_2d_pair(sa + a_bytes, &tmBh, fb, kc, (int)rank * half_rows);
                if (p.use_lo) tma_load_2d_pair(sa + a_bytes + b_bytes, &tmBl, fb, kc, (int)rank * half_rows);
            }
            // The leader's full barriers count the bytes of both CTAs: it does not go on to the pair's final barrier
            // before the last use of every stage has landed, in any run (see gemm_tc_kernel).
            if (rank == 0) {
                for (int i = max(0, issued - p.stages); i < issued; ++i) {
                    const uint32_t bar = full_bar(i % p.stages), ph = (uint32_t)(i / p.stages) & 1u;
                    for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(bar, ph); ++it) {}
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = instr_desc_bf16_m256(p.n_pad);
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
                        umma2_bf16(td, da + 2u * k, dbh + 2u * k, idesc, (i > 0 || k > 0) ? 1u : 0u);
                    if (p.use_lo) {
#pragma unroll
                        for (int k = 0; k < kBlockK / kUmmaK; ++k) umma2_bf16(td, da + 2u * k, dbl + 2u * k, idesc, 1u);
                    }
                }
                umma2_commit_both(empty_bar(s));  // frees the stage in both CTAs once these MMAs have read it
            }
            umma2_commit_both(tmem_full_bar);  // accumulators complete (arrives even after a failed wait)
        }
    } else {
        const int quad = warp & 3, half = (warp - 2) >> 2;
        if (EPI == tc::kEpiScatterAtomic) {
            for (int e = (int)threadIdx.x - 64; e < p.m; e += 256) idx_s[e] = p.idx[e];
            asm volatile("bar.sync 1, 256;" ::: "memory");
        }
        pdl_wait();
        const int m_act = p.m_dev ? max(0, min(p.m, __ldg(p.m_dev) - p.row0)) : p.m;
        const bool ok = mbar_wait(tmem_full_bar, 0u, &abort_s, p.flags) && !abort_s;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const bool run = ok && nkb > 0;
        if (EPI == tc::kEpiSwiglu) {
            const int f = tile * 256 + (int)rank * 128 + quad * 32 + lane;
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
        } else if (run) {
            for (int a = 0; a < p.mt; ++a) {
                const int f = row_of(a) + quad * 32 + lane;
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
                                if (EPI == tc::kEpiStore) p.Y[(size_t)j * p.ldy + f] = val;
                                else if (EPI == tc::kEpiAtomic) atomicAdd(p.Y + (size_t)j * p.ldy + f, val);
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
    if (warp == 1 && lane == 0 && abort_s) {
        // after a failed wait: the MMAs that were issued still finish; see them done before anything is given back
        for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(tmem_full_bar, 0u); ++it) {}
    }
    __syncwarp();
    // Neither CTA of the pair leaves, or frees its tensor memory, while the other may still read its shared memory
    // (the leader's MMAs read the partner's tiles), write its tensor memory or signal its barriers.
    cluster_sync_all();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"((uint32_t)p.tmem_cols)
                     : "memory");
    }
}

}  // namespace tc2
}  // namespace first
