// Grouped-query decode attention over the active rows' bfloat16 caches (head_dim 64/128).
//
// HBM-bound: every cached key and value of an active (sequence, kv head) is read once.
// K/V tiles of 64 tokens are staged by TMA into 128-byte-swizzled shared memory through a
// 3-stage ring (one producer warp, four consumer warps).  With 4..8 query heads per KV
// head the score and PV products are too much arithmetic for the FP32 pipes at HBM speed
// (about 4 FLOP per cache byte), so they run on the tensor cores via mma.sync m16n8k16:
// the group's query heads are the M rows.  Precision: q and the softmax weights are split
// into bfloat16 hi + lo; hi sits in rows 0..7 and lo in rows 8..15 of the same A fragment,
// so one MMA yields both partial products and the thread adds them -- float32-grade q and p
// against the stored bfloat16 keys/values.  Softmax is online, row maxima by quad shuffles.
// The token axis is split in chunks of C tokens per CTA; the CTA that finishes a (row, kv head)
// last (an atomic ticket) merges the chunks and writes the attention output, so no second
// kernel is needed.
#pragma once
#include "common.cuh"
#include "first.h"
#include "gemm_tc.cuh"  // mbarrier / TMA helpers

namespace first {
namespace attn {

constexpr int kTile = 64;    // tokens per stage
constexpr int kStages = 3;
constexpr int kConsumers = 128;

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// (x, y) -> packed bf16 hi parts and packed bf16 remainders
__device__ __forceinline__ void split2(float x, float y, uint32_t& hi, uint32_t& lo) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
    const __nv_bfloat162 l = __floats2bfloat162_rn(x - __low2float(h), y - __high2float(h));
    hi = *reinterpret_cast<const uint32_t*>(&h);
    lo = *reinterpret_cast<const uint32_t*>(&l);
}
__device__ __forceinline__ void bar_consumers() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// When qkv is set the kernel works straight from the QKV projection's output
// ([m][(Hq+2*Hkv)*HD] float32: q heads, k heads, v heads): it rotates and scales q itself, and the
// CTA that holds a row's last chunk rotates the new token's key, rounds key and value to bfloat16,
// writes them at the end of the row's slab and drops them into its shared-memory tile, so that no
// separate rotate-and-append kernel runs.  cs: [B][HD/2] (cos, sin) of each sequence's position.
struct RopeFuse {
    const float* qkv;
    const float2* cs;
    float qscale;
    __nv_bfloat16* k_slab;  // this layer's [Hkv][cap_total][HD]
    __nv_bfloat16* v_slab;
};

// grid (S_max, Hkv, m), 160 threads.  Work item = (active row i, kv head h, chunk c):
// tokens [c*C, min(T, (c+1)*C)), T = len[b]+1 (the new token sits at row len[b]: already written by the
// rotate-and-append kernel, or put there by this kernel, see RopeFuse; T = len[b] if the slab was full
// and nothing is written), taken from rowinfo[i].  Chunks past T exit at once.
// q: [m][Hq][HD] float32, pre-scaled by 1/sqrt(HD) (unused with RopeFuse).  tmK/tmV: [Hkv*cap_total][HD] bf16, box 64x64.
// Scratch: o_part [m][Hq][S_max][HD] (unnormalised), ml_part [m][Hq][S_max] = (max, sum),
// ticket [m][Hkv] (zero between launches: the merging CTA resets it).
// Output: out [m][Hq*HD] float32 and/or its bfloat16 hi/lo split (either may be NULL).
//
// PAIR (prompt processing, where consecutive rows are consecutive tokens of one sequence): a work item may
// serve two rows at once.  rowinfo[i].y bit 61 = row i also serves row i+1 (same slab, one token more, its key
// and value already in the slab); bit 60 = row i is served by row i-1 (its CTAs exit).  The second row's query
// heads take fragment rows G..2G-1 (so 2G <= 8), share every K/V tile with the first row's, and see one token
// more at the end.  Not combined with RopeFuse.
// CL (decode only): the grid is launched as thread-block clusters of gridDim.x CTAs, one cluster per (row, kv head),
// and a split row's chunks meet in the shared memory of the cluster's first CTA instead of in global memory: every
// other chunk writes its partial result there (distributed shared memory, plain remote stores -- no multicast load
// anywhere), arrives at the cluster barrier and leaves; the first CTA waits at that barrier and merges.  No global
// round trip, no fence, no ticket.  Needs (gridDim.x - 1) * GR * (HD + 2) floats of shared memory behind the ring.
template <int HD, int G, bool PAIR = false, bool CL = false>
__global__ void __launch_bounds__(160) attn_split_mma(const __grid_constant__ CUtensorMap tmK,
                                                      const __grid_constant__ CUtensorMap tmV,
                                                      const float* q, int64_t cap_total,
                                                      const longlong2* rowinfo, const int32_t* __restrict__ m_dev,
                                                      int Hq, int C,
                                                      float* __restrict__ o_part, float2* __restrict__ ml_part,
                                                      uint32_t* __restrict__ ticket, float* __restrict__ out,
                                                      __nv_bfloat16* __restrict__ out_hi,
                                                      __nv_bfloat16* __restrict__ out_lo,
                                                      uint32_t* __restrict__ flags, const RopeFuse rf,
                                                      uint64_t* stamp) {
    const Stamp stamp_guard(stamp);
    constexpr int kHalves = HD / 64;              // 128-byte column groups per row
    constexpr int kBox = kTile * 128;             // bytes of one 64-token x 64-element box
    constexpr int kStageBytes = 2 * kHalves * kBox;
    constexpr int kKSteps = HD / 16, kNTiles = HD / 8;
    constexpr int GR = PAIR ? 2 * G : G;  // fragment rows in use
    static_assert(GR <= 8, "query heads of a group (of two rows' groups) are the 8 hi rows of the A fragment");

    pdl_trigger();
    // m_dev: the layer's active-row count (the grid is sized from a host-side upper bound of it)
    if (m_dev && (int)blockIdx.z >= __ldg(m_dev)) {
        pdl_wait();  // a grid must not complete before its predecessor has: later kernels rely on that chain
        return;
    }
    // Set-up that needs nothing from the previous kernel comes first, so that it overlaps that kernel's tail.
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - tc::smem_u32(smem_raw));
    __shared__ uint64_t bar_mem[2 * kStages];
    __shared__ int abort_s;
    __shared__ int last_s;
    auto full_bar = [&](int s) { return tc::smem_u32(&bar_mem[s]); };
    auto empty_bar = [&](int s) { return tc::smem_u32(&bar_mem[kStages + s]); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        abort_s = 0;
        for (int s = 0; s < kStages; ++s) { tc::mbar_init(full_bar(s), 1); tc::mbar_init(empty_bar(s), 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    pdl_wait();
    const int S_max = gridDim.x, c = blockIdx.x, h = blockIdx.y, i = blockIdx.z;
    // (tokens to attend over incl. the new one | batch row << 32, first slab row | append << 62)
    const longlong2 ri = __ldcg(&rowinfo[i]);
    const int T1 = (int)(ri.x & 0xffffffffll);  // tokens row i attends over
    const int brow = (int)(ri.x >> 32);
    const int64_t slab0 = ri.y & ((1ll << 60) - 1);
    const bool append = !PAIR && rf.qkv != nullptr && ((ri.y >> 62) & 1) != 0;
    if (PAIR && ((ri.y >> 60) & 1)) return;              // row i-1's work items serve this row
    const bool two = PAIR && ((ri.y >> 61) & 1);          // this work item also serves row i+1
    const int T = T1 + (two ? 1 : 0);                     // tokens streamed
    // A row of T tokens is cut into ceil(T / C) chunks of equal length (a multiple of the tile), not
    // into full chunks plus a short remainder: its CTAs then finish together.
    const int n_chunks = (T + C - 1) / C;
    if (c >= n_chunks) return;
    const int Cb = ((T + n_chunks - 1) / n_chunks + kTile - 1) / kTile * kTile;
    const int t_begin = c * Cb;
    if (t_begin >= T) return;  // (cannot happen: (n_chunks - 1) * Cb < T)
    const int t_end = min(T, t_begin + Cb);
    const int n_tiles = (t_end - t_begin + kTile - 1) / kTile;


    if (warp == 4) {  // ---------------- producer
        if (lane == 0) {
            const int64_t row0 = (int64_t)h * cap_total + slab0 + t_begin;
            uint64_t pol;  // cached keys/values are read once per step: do not let them displace L2 contents
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
            int issued = 0;
            for (int j = 0; j < n_tiles; ++j, ++issued) {
                const int s = j % kStages;
                const uint32_t ph = (uint32_t)(j / kStages) & 1u;
                if (!tc::mbar_wait(empty_bar(s), ph ^ 1u, &abort_s, flags)) break;
                const uint32_t sa = base + (uint32_t)s * kStageBytes;
                tc::mbar_expect_tx(full_bar(s), kStageBytes);
                const int row = (int)(row0 + (int64_t)j * kTile);
#pragma unroll
                for (int hf = 0; hf < kHalves; ++hf) {
                    tc::tma_load_2d_hint(sa + hf * kBox, &tmK, full_bar(s), hf * 64, row, pol);
                    tc::tma_load_2d_hint(sa + (kHalves + hf) * kBox, &tmV, full_bar(s), hf * 64, row, pol);
                }
            }
            // The producer leaves only when every copy it issued has landed (the last use of each stage), whether
            // or not a role has given up and whoever noticed first.  A CTA's shared memory is released when all
            // of its threads have left, this one included, so it is never reused with a copy in flight.  The
            // consumers wait for the same barriers in a normal run, so this costs nothing.
            for (int j = max(0, issued - kStages); j < issued; ++j) {
                const uint32_t bar = full_bar(j % kStages), ph = (uint32_t)(j / kStages) & 1u;
                for (uint32_t it = 0; it < tc::kSpinLimit && !tc::mbar_try_wait(bar, ph); ++it) {}
            }
        }
        return;
    }

    // ---------------- consumers: warp w owns tokens [16w, 16w+16) of every tile
    const int g = lane >> 2, tq = lane & 3;
    uint32_t qh[kKSteps][2], ql[kKSteps][2];  // A fragments: (k0..k0+1), (k0+8..k0+9) of row g
    const int qkv_stride = (Hq + 2 * (int)gridDim.y) * HD;
    const float2* csr = rf.cs + (size_t)brow * (HD / 2);
    const int rows_live = two ? 2 * G : G;                // fragment rows that carry a query head
    if (!PAIR && rf.qkv) {
        constexpr int kHalf = HD / 2;
        const float* qrow = rf.qkv + (size_t)i * qkv_stride + ((size_t)h * G + (g < G ? g : 0)) * HD;
        auto rot2 = [&](int dd) {  // rotated, scaled q[dd], q[dd+1] (dd even; both on the same side of HD/2)
            const int lo_d = dd < kHalf ? dd : dd - kHalf;
            const float2 a = *reinterpret_cast<const float2*>(qrow + lo_d);
            const float2 bb = *reinterpret_cast<const float2*>(qrow + lo_d + kHalf);
            const float4 cc = *reinterpret_cast<const float4*>(csr + lo_d);  // cos, sin of lo_d and lo_d + 1
            return dd < kHalf ? make_float2((a.x * cc.x - bb.x * cc.y) * rf.qscale, (a.y * cc.z - bb.y * cc.w) * rf.qscale)
                              : make_float2((bb.x * cc.x + a.x * cc.y) * rf.qscale, (bb.y * cc.z + a.y * cc.w) * rf.qscale);
        };
#pragma unroll
        for (int ks = 0; ks < kKSteps; ++ks) {
            float2 v0 = make_float2(0.f, 0.f), v1 = v0;
            if (g < G) {
                v0 = rot2(ks * 16 + 2 * tq);
                v1 = rot2(ks * 16 + 8 + 2 * tq);
            }
            split2(v0.x, v0.y, qh[ks][0], ql[ks][0]);
            split2(v1.x, v1.y, qh[ks][1], ql[ks][1]);
        }
    } else {
        const int gq = g < rows_live ? g : 0;
        const float* qrow = q + ((size_t)(i + gq / G) * Hq + (size_t)h * G + gq % G) * HD;
#pragma unroll
        for (int ks = 0; ks < kKSteps; ++ks) {
            float2 v0 = make_float2(0.f, 0.f), v1 = v0;
            if (g < rows_live) {
                v0 = *reinterpret_cast<const float2*>(qrow + ks * 16 + 2 * tq);
                v1 = *reinterpret_cast<const float2*>(qrow + ks * 16 + 8 + 2 * tq);
            }
            split2(v0.x, v0.y, qh[ks][0], ql[ks][0]);
            split2(v1.x, v1.y, qh[ks][1], ql[ks][1]);
        }
    }
    float o[kNTiles][4];
#pragma unroll
    for (int nt = 0; nt < kNTiles; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
    float m_run = -INFINITY, l_run = 0.f;
    const int mat = lane >> 3, r8 = lane & 7;
    bool ok = true;

    for (int j = 0; j < n_tiles; ++j) {
        const int s = j % kStages;
        const uint32_t ph = (uint32_t)(j / kStages) & 1u;
        if (!tc::mbar_wait(full_bar(s), ph, &abort_s, flags)) { ok = false; break; }
        const uint32_t sK = base + (uint32_t)s * kStageBytes, sV = sK + kHalves * kBox;
        const int tile_t0 = t_begin + j * kTile;
        const int valid = t_end - tile_t0;  // tokens of this tile that exist (may exceed 64)
        // the first row of a pair does not see the last token (its successor's)
        const int lim = valid - ((two && g < G && t_end == T) ? 1 : 0);
        if (valid < kTile) {
            // rows past the end hold someone else's bytes: zero them in V so 0 * garbage stays 0
            uint8_t* vptr = base_ptr + (size_t)s * kStageBytes + kHalves * kBox;
            for (int e = lane; e < 16 * kHalves * 8; e += 32) {
                const int row = warp * 16 + e / (kHalves * 8), cc = e % (kHalves * 8);
                if (row >= valid)
                    *reinterpret_cast<uint4*>(vptr + (cc >> 3) * kBox + row * 128 + (cc & 7) * 16) = make_uint4(0, 0, 0, 0);
            }
            __syncwarp();
        }
        if (append && t_end == T && j == n_tiles - 1) {
            // The new token (row T-1 of the sequence) is the last row of this tile: what TMA fetched for
            // it is whatever the slab held.  The warp that owns the row builds the key and value from
            // the projection output, stores them in the slab for later steps and in the tile for this one.
            const int r = (T - 1) - tile_t0;
            if ((r >> 4) == warp) {
                constexpr int kHalf = HD / 2;
                const float* krow = rf.qkv + (size_t)i * qkv_stride + (size_t)Hq * HD + (size_t)h * HD;
                const float* vrow = krow + (size_t)gridDim.y * HD;
                uint8_t* kst = base_ptr + (size_t)s * kStageBytes;
                uint8_t* vst = kst + kHalves * kBox;
                const size_t grow = ((size_t)h * cap_total + (size_t)slab0 + (size_t)(T - 1)) * HD;
                auto put = [&](uint8_t* st, __nv_bfloat16* slab, int dd, __nv_bfloat162 val) {
                    const int cc = (dd & 63) >> 3;
                    *reinterpret_cast<__nv_bfloat162*>(st + (dd >> 6) * kBox + r * 128 + ((cc ^ (r & 7)) << 4) + (dd & 7) * 2) = val;
                    *reinterpret_cast<__nv_bfloat162*>(slab + grow + dd) = val;
                };
                for (int pp = 2 * lane; pp < kHalf; pp += 64) {
                    const float2 a = *reinterpret_cast<const float2*>(krow + pp);
                    const float2 bb = *reinterpret_cast<const float2*>(krow + pp + kHalf);
                    const float4 cc = *reinterpret_cast<const float4*>(csr + pp);
                    put(kst, rf.k_slab, pp, __floats2bfloat162_rn(a.x * cc.x - bb.x * cc.y, a.y * cc.z - bb.y * cc.w));
                    put(kst, rf.k_slab, pp + kHalf, __floats2bfloat162_rn(bb.x * cc.x + a.x * cc.y, bb.y * cc.z + a.y * cc.w));
                    const float2 va = *reinterpret_cast<const float2*>(vrow + pp);
                    const float2 vb = *reinterpret_cast<const float2*>(vrow + pp + kHalf);
                    put(vst, rf.v_slab, pp, __floats2bfloat162_rn(va.x, va.y));
                    put(vst, rf.v_slab, pp + kHalf, __floats2bfloat162_rn(vb.x, vb.y));
                }
                __syncwarp();
            }
        }
        // ---- scores S[g][token] for this warp's 16 tokens (two n-tiles of 8)
        float sc[2][4];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < kKSteps; ++ks) {
            const int row = warp * 16 + (mat >> 1) * 8 + r8;
            const int cg = 2 * ks + (mat & 1);
            const uint32_t addr = sK + (cg >> 3) * kBox + row * 128 + (((cg & 7) ^ (row & 7)) << 4);
            uint32_t b0, b1, b2, b3;
            ldsm_x4(addr, b0, b1, b2, b3);
            mma16816(sc[0], qh[ks][0], ql[ks][0], qh[ks][1], ql[ks][1], b0, b1);
            mma16816(sc[1], qh[ks][0], ql[ks][0], qh[ks][1], ql[ks][1], b2, b3);
        }
        float sv[4];
        float mx = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int tok = warp * 16 + nt * 8 + 2 * tq + e;
                const float v = (tok < lim) ? sc[nt][e] + sc[nt][e + 2] : -INFINITY;  // hi + lo parts
                sv[nt * 2 + e] = v;
                mx = fmaxf(mx, v);
            }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m_run, mx);
        float p[4];
        float scale = 1.f;
        if (m_new == -INFINITY) {
            p[0] = p[1] = p[2] = p[3] = 0.f;
        } else {
            scale = (m_run == -INFINITY) ? 0.f : __expf(m_run - m_new);
#pragma unroll
            for (int e = 0; e < 4; ++e) p[e] = (sv[e] == -INFINITY) ? 0.f : __expf(sv[e] - m_new);
        }
        m_run = m_new;
        l_run = l_run * scale + (p[0] + p[1] + p[2] + p[3]);
#pragma unroll
        for (int nt = 0; nt < kNTiles; ++nt) { o[nt][0] *= scale; o[nt][1] *= scale; o[nt][2] *= scale; o[nt][3] *= scale; }
        uint32_t ph0, pl0, ph1, pl1;
        split2(p[0], p[1], ph0, pl0);
        split2(p[2], p[3], ph1, pl1);
        // ---- O[g][d] += P[g][token] V[token][d]
#pragma unroll
        for (int n2 = 0; n2 < kNTiles / 2; ++n2) {
            const int row = warp * 16 + (mat & 1) * 8 + r8;
            const int cg = 2 * n2 + (mat >> 1);
            const uint32_t addr = sV + (cg >> 3) * kBox + row * 128 + (((cg & 7) ^ (row & 7)) << 4);
            uint32_t b0, b1, b2, b3;
            ldsm_x4_t(addr, b0, b1, b2, b3);
            mma16816(o[2 * n2], ph0, pl0, ph1, pl1, b0, b1);
            mma16816(o[2 * n2 + 1], ph0, pl0, ph1, pl1, b2, b3);
        }
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(empty_bar(s)) : "memory");
    }

    // ---- merge the four warps' partial softmax states through shared memory (stage memory is free now)
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    bar_consumers();
    float* o_s = reinterpret_cast<float*>(base_ptr);       // [4][GR][HD]
    float* m_s = o_s + 4 * GR * HD;                         // [4][GR]
    float* l_s = m_s + 4 * GR;                              // [4][GR]
    // CL: behind the ring, never touched by a copy: [S_max-1][GR][HD+2] partials of chunks 1.. (written by them,
    // remotely), then this CTA's own partial [GR][HD] and its (max, sum) [2][GR]
    float* part_s = reinterpret_cast<float*>(base_ptr + kStages * kStageBytes);
    float* part0_s = part_s + (gridDim.x - 1) * GR * (HD + 2);
    float* ml0_s = part0_s + GR * HD;
    uint32_t part_remote = 0;
    if (CL) {
        const uint32_t local = base + (uint32_t)(kStages * kStageBytes);
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(part_remote) : "r"(local), "r"(0));
    }
    if (g < GR) {
#pragma unroll
        for (int nt = 0; nt < kNTiles; ++nt) {
            float2 v = make_float2(o[nt][0] + o[nt][2], o[nt][1] + o[nt][3]);
            *reinterpret_cast<float2*>(o_s + ((size_t)warp * GR + g) * HD + nt * 8 + 2 * tq) = v;
        }
        if (tq == 0) { m_s[warp * GR + g] = m_run; l_s[warp * GR + g] = l_run; }
    }
    bar_consumers();
    if (!ok || abort_s) return;
    // query head (row-major over [m][Hq]) of fragment row gg: the second row of a pair follows the first
    auto hq_of = [&](int gg) { return (size_t)(i + gg / G) * Hq + (size_t)h * G + gg % G; };
    auto emit = [&](size_t hq, int d, float y) {
        if (out) out[hq * HD + d] = y;
        if (out_hi) {
            const __nv_bfloat16 hh = __float2bfloat16_rn(y);
            out_hi[hq * HD + d] = hh;
            out_lo[hq * HD + d] = __float2bfloat16_rn(y - __bfloat162float(hh));
        }
    };
    for (int e = threadIdx.x; e < rows_live * HD; e += kConsumers) {
        const int gg = e / HD, d = e - gg * HD;
        const float M = fmaxf(fmaxf(m_s[gg], m_s[GR + gg]), fmaxf(m_s[2 * GR + gg], m_s[3 * GR + gg]));
        float acc = 0.f, l = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const float mw = m_s[w * GR + gg];
            if (mw > -INFINITY) {
                const float f = __expf(mw - M);
                acc += o_s[((size_t)w * GR + gg) * HD + d] * f;
                l += l_s[w * GR + gg] * f;
            }
        }
        if (n_chunks == 1) {
            emit(hq_of(gg), d, acc / l);  // the whole row in one chunk: done
        } else if (CL) {
            if (c == 0) {  // the merging CTA keeps its own partial in registers-to-shared form
                part0_s[gg * HD + d] = acc;
                if (d == 0) { ml0_s[gg] = M; ml0_s[GR + gg] = l; }
            } else {       // chunk c > 0: slot c-1 of the first CTA's buffer
                const uint32_t slot = part_remote + (uint32_t)(((c - 1) * GR + gg) * (HD + 2)) * 4u;
                asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(slot + (uint32_t)d * 4u), "f"(acc) : "memory");
                if (d == 0) {
                    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(slot + (uint32_t)HD * 4u), "f"(M) : "memory");
                    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(slot + (uint32_t)(HD + 1) * 4u), "f"(l) : "memory");
                }
            }
        } else {
            o_part[(hq_of(gg) * S_max + c) * HD + d] = acc;
            if (d == 0) ml_part[hq_of(gg) * S_max + c] = make_float2(M, l);
        }
    }
    if (n_chunks == 1) return;
    if (CL) {
        // Every consumer thread of every live chunk arrives (release: its remote stores are visible to whoever
        // acquires); chunks other than the first leave at once.  Threads that have exited (producer warps, work items
        // past the row's end) are not waited for.
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        if (c != 0) return;
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
        bar_consumers();  // part0_s / ml0_s of all four warps
        float* w_s = o_s;  // [2][GR][64], as below; o_s is free again
        for (int e = threadIdx.x; e < rows_live * n_chunks; e += kConsumers) {
            const int gg = e / n_chunks, sidx = e - gg * n_chunks;
            const float* src = sidx == 0 ? nullptr : part_s + ((sidx - 1) * GR + gg) * (HD + 2) + HD;
            w_s[gg * 64 + sidx] = sidx == 0 ? ml0_s[gg] : src[0];
            w_s[(GR + gg) * 64 + sidx] = sidx == 0 ? ml0_s[GR + gg] : src[1];
        }
        bar_consumers();
        if (threadIdx.x < rows_live) {
            const int gg = threadIdx.x;
            float M = -INFINITY, den = 0.f;
            for (int sidx = 0; sidx < n_chunks; ++sidx) M = fmaxf(M, w_s[gg * 64 + sidx]);
            for (int sidx = 0; sidx < n_chunks; ++sidx) den += w_s[(GR + gg) * 64 + sidx] * __expf(w_s[gg * 64 + sidx] - M);
            const float inv = 1.f / den;
            for (int sidx = 0; sidx < n_chunks; ++sidx) w_s[gg * 64 + sidx] = __expf(w_s[gg * 64 + sidx] - M) * inv;
        }
        bar_consumers();
        for (int e = threadIdx.x; e < rows_live * HD; e += kConsumers) {
            const int gg = e / HD, d = e - gg * HD;
            const float* wv = w_s + gg * 64;
            float acc = part0_s[gg * HD + d] * wv[0];
            for (int sidx = 1; sidx < n_chunks; ++sidx) acc += part_s[((sidx - 1) * GR + gg) * (HD + 2) + d] * wv[sidx];
            emit(hq_of(gg), d, acc);
        }
        return;
    }
    // ---- ticket: the last chunk of this (row, kv head) to get here merges them all
    __threadfence();
    bar_consumers();
    if (threadIdx.x == 0) {
        const uint32_t t = atomicAdd(&ticket[(size_t)i * gridDim.y + h], 1u);
        last_s = (t == (uint32_t)n_chunks - 1u);
        if (last_s) ticket[(size_t)i * gridDim.y + h] = 0u;
    }
    bar_consumers();
    if (!last_s) return;
    __threadfence();
    // Merge: (1) all chunk statistics into shared memory at once, (2) one weight per (head, chunk),
    // (3) weighted sums with independent loads.  o_s is free again (everyone passed the barrier).
    float* w_s = o_s;  // [2][GR][64]
    for (int e = threadIdx.x; e < rows_live * n_chunks; e += kConsumers) {
        const int gg = e / n_chunks, sidx = e - gg * n_chunks;
        const float2 ml = __ldcg(&ml_part[hq_of(gg) * S_max + sidx]);
        w_s[gg * 64 + sidx] = ml.x;
        w_s[(GR + gg) * 64 + sidx] = ml.y;
    }
    bar_consumers();
    if (threadIdx.x < rows_live) {
        const int gg = threadIdx.x;
        float M = -INFINITY, den = 0.f;
        for (int sidx = 0; sidx < n_chunks; ++sidx) M = fmaxf(M, w_s[gg * 64 + sidx]);
        for (int sidx = 0; sidx < n_chunks; ++sidx) den += w_s[(GR + gg) * 64 + sidx] * __expf(w_s[gg * 64 + sidx] - M);
        const float inv = 1.f / den;
        for (int sidx = 0; sidx < n_chunks; ++sidx) w_s[gg * 64 + sidx] = __expf(w_s[gg * 64 + sidx] - M) * inv;
    }
    bar_consumers();
    for (int e = threadIdx.x; e < rows_live * HD; e += kConsumers) {
        const int gg = e / HD, d = e - gg * HD;
        const size_t hq = hq_of(gg);
        const float* src = o_part + (hq * S_max) * HD + d;
        const float* wv = w_s + gg * 64;
        float acc = 0.f;
        int sidx = 0;
        for (; sidx + 4 <= n_chunks; sidx += 4) {
            const float v0 = __ldcg(src + (size_t)(sidx + 0) * HD), v1 = __ldcg(src + (size_t)(sidx + 1) * HD);
            const float v2 = __ldcg(src + (size_t)(sidx + 2) * HD), v3 = __ldcg(src + (size_t)(sidx + 3) * HD);
            acc += v0 * wv[sidx] + v1 * wv[sidx + 1] + v2 * wv[sidx + 2] + v3 * wv[sidx + 3];
        }
        for (; sidx < n_chunks; ++sidx) acc += __ldcg(src + (size_t)sidx * HD) * wv[sidx];
        emit(hq, d, acc);
    }
}

}  // namespace attn
}  // namespace first
