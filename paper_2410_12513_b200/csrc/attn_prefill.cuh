// Causal attention for prompt chunks ("Inference for FiRST", item 1: the prompt runs through every layer), where the
// rows of a launch are consecutive tokens of a few sequences: a work item serves a GROUP of up to eight consecutive
// tokens of one sequence (positions p0 .. p0+n-1 inside one block of eight positions) for one KV head.
//
// Why: with one or two tokens per work item (attn_split_mma and its pair form) every token pair streams its whole
// prefix from L2 again, and the prompt phase's attention is bound by that traffic (sum over tokens of prefix length).
// Here the K/V tiles of a prefix are staged once per eight tokens: each of the four consumer warps owns two tokens of
// the group (their 2 x G query heads are the 8 "hi" rows of its MMA fragment, the bfloat16 remainders the 8 "lo" rows)
// and walks ALL 64 tokens of every tile, so the warps share the tiles and nothing is merged across warps.
// The token axis is still cut into chunks of C tokens per CTA; the CTA that finishes a (group, kv head) last merges
// the chunks (atomic ticket), as in the decode kernel.  Precision, tile staging (TMA into 128-byte-swizzled shared
// memory, 3-stage ring, one producer warp) and the online softmax are those of attn_split_mma.
//
// Row facts come from rope_append (group mode): rowinfo[i].x = tokens row i attends over | batch row << 32;
// rowinfo[i].y = first slab row | (n-1) << 56 for a group leader | 1 << 60 for a row served by its leader.
#pragma once
#include "attn_mma.cuh"

namespace first {
namespace attn {

// grid (S_max, Hkv, ceil(m / 8)), 160 threads: CTA (c, h, z) looks at rows 8z .. 8z+7 and serves, one after the other,
// the groups that START there (almost always exactly one: eight consecutive rows of a sequence hold one multiple of
// eight; more only where sequences or the chunk begin).  A grid over rows would launch eight CTAs per group of which
// seven leave at once -- with 256-row chunks that start-and-leave traffic alone took longer than the attention.
// q: [m][Hq][HD] float32, rotated and pre-scaled.  Scratch and outputs as in attn_split_mma (o_part
// [m][Hq][S_max][HD], ml_part [m][Hq][S_max], ticket [m][Hkv]); m = rows of the launch.
template <int HD, int G>
__global__ void __launch_bounds__(160, 2) attn_group_mma(const __grid_constant__ CUtensorMap tmK,
                                                      const __grid_constant__ CUtensorMap tmV, const float* q,
                                                      int64_t cap_total, const longlong2* rowinfo, int m,
                                                      const int32_t* __restrict__ m_dev, int Hq, int C,
                                                      float* __restrict__ o_part, float2* __restrict__ ml_part,
                                                      uint32_t* __restrict__ ticket, float* __restrict__ out,
                                                      __nv_bfloat16* __restrict__ out_hi,
                                                      __nv_bfloat16* __restrict__ out_lo, uint32_t* __restrict__ flags,
                                                      uint64_t* stamp) {
    const Stamp stamp_guard(stamp);
    constexpr int kHalves = HD / 64;
    constexpr int kBox = kTile * 128;
    constexpr int kStageBytes = 2 * kHalves * kBox;
    constexpr int kKSteps = HD / 16, kNTiles = HD / 8;
    constexpr int GR = 2 * G;  // fragment rows of a warp: two tokens x G query heads
    static_assert(GR <= 8, "two tokens' query heads are the 8 hi rows of the A fragment");
    static_assert((4 * GR * HD + 8 * GR) * 4 <= kStageBytes && 2 * 4 * GR * 64 * 4 <= kStageBytes,
                  "the epilogue's scratch must fit the one stage a group is sure to hold");

    pdl_trigger();
    if (m_dev) m = min(m, __ldg(m_dev));
    if ((int)blockIdx.z * 8 >= m) {
        pdl_wait();
        return;
    }
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
    const int S_max = gridDim.x, c = blockIdx.x, h = blockIdx.y;
    const int g = lane >> 2, tq = lane & 3;
    const int mat = lane >> 3, r8 = lane & 7;
    // Tiles this CTA has been through so far: the ring's stage and phase go on from one group to the next, and every
    // role advances the count by the same amounts (no CTA-wide barrier between groups).
    int tiles_done = 0, issued_total = 0;
  for (int rr = 0; rr < 8; ++rr) {
    const int i = (int)blockIdx.z * 8 + rr;
    if (i >= m) break;
    const longlong2 ri = __ldcg(&rowinfo[i]);
    if ((ri.y >> 60) & 1) continue;                     // served by its group's leader
    const int T1 = (int)(ri.x & 0xffffffffll);          // tokens the leader (first token of the group) attends over
    const int n_mem = (int)((ri.y >> 56) & 15) + 1;     // tokens in the group: rows i .. i+n_mem-1
    const int64_t slab0 = ri.y & ((1ll << 56) - 1);
    const int T = T1 + n_mem - 1;                       // tokens streamed: the last member's view
    const int n_chunks = (T + C - 1) / C;
    if (c >= n_chunks) continue;
    const int Cb = ((T + n_chunks - 1) / n_chunks + kTile - 1) / kTile * kTile;
    const int t_begin = c * Cb;
    if (t_begin >= T) continue;
    const int t_end = min(T, t_begin + Cb);
    const int n_tiles = (t_end - t_begin + kTile - 1) / kTile;
    const int tile0 = tiles_done;
    tiles_done += n_tiles;

    if (warp == 4) {  // ---------------- producer
        if (lane == 0 && !abort_s) {
            const int64_t row0 = (int64_t)h * cap_total + slab0 + t_begin;
            for (int j = 0; j < n_tiles; ++j, ++issued_total) {
                const int jj = tile0 + j, s = jj % kStages;
                const uint32_t ph = (uint32_t)(jj / kStages) & 1u;
                if (!tc::mbar_wait(empty_bar(s), ph ^ 1u, &abort_s, flags)) break;
                const uint32_t sa = base + (uint32_t)s * kStageBytes;
                tc::mbar_expect_tx(full_bar(s), kStageBytes);
                const int row = (int)(row0 + (int64_t)j * kTile);
#pragma unroll
                for (int hf = 0; hf < kHalves; ++hf) {  // (prefixes are re-read by the next group: default L2 policy)
                    tc::tma_load_2d(sa + hf * kBox, &tmK, full_bar(s), hf * 64, row);
                    tc::tma_load_2d(sa + (kHalves + hf) * kBox, &tmV, full_bar(s), hf * 64, row);
                }
            }
        }
        continue;
    }

    // ---------------- consumers: warp w owns members 2w and 2w+1 and walks every token of every tile
    const int mem_a = 2 * warp;                                   // first member of this warp
    const int live = max(0, min(2, n_mem - mem_a));               // members this warp really has (0, 1 or 2)
    const int my_mem = mem_a + (g >= G ? 1 : 0);                  // member of this thread's fragment row
    const bool row_live = g < GR && (g / G) < live;
    const int T1_row = T1 + my_mem;                               // tokens that row attends over
    uint32_t qh[kKSteps][2], ql[kKSteps][2];
    {
        const float* qrow = q + ((size_t)(i + (row_live ? my_mem : 0)) * Hq + (size_t)h * G + (g < GR ? g % G : 0)) * HD;
#pragma unroll
        for (int ks = 0; ks < kKSteps; ++ks) {
            float2 v0 = make_float2(0.f, 0.f), v1 = v0;
            if (row_live) {
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
    bool ok = true;

    for (int j = 0; j < n_tiles; ++j) {
        const int jj = tile0 + j, s = jj % kStages;
        const uint32_t ph = (uint32_t)(jj / kStages) & 1u;
        if (!tc::mbar_wait(full_bar(s), ph, &abort_s, flags)) { ok = false; break; }
        const uint32_t sK = base + (uint32_t)s * kStageBytes, sV = sK + kHalves * kBox;
        const int tile_t0 = t_begin + j * kTile;
        const int valid = t_end - tile_t0;
        if (valid < kTile) {
            // rows past the end hold someone else's bytes: zero them in V (every warp reads the whole tile, so all
            // four zero their 16 rows and meet before anyone multiplies)
            uint8_t* vptr = base_ptr + (size_t)s * kStageBytes + kHalves * kBox;
            for (int e = lane; e < 16 * kHalves * 8; e += 32) {
                const int row = warp * 16 + e / (kHalves * 8), cc = e % (kHalves * 8);
                if (row >= valid)
                    *reinterpret_cast<uint4*>(vptr + (cc >> 3) * kBox + row * 128 + (cc & 7) * 16) = make_uint4(0, 0, 0, 0);
            }
            bar_consumers();
        }
        // tokens of this tile the thread's row may see (causal: its own position is the last one)
        const int lim = row_live ? min(valid, T1_row - tile_t0) : 0;
        // ---- scores S[row][token] for all 64 tokens (eight n-tiles of 8)
        float sc[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < kKSteps; ++ks) {
#pragma unroll
            for (int t16 = 0; t16 < 4; ++t16) {
                const int row = t16 * 16 + (mat >> 1) * 8 + r8;
                const int cg = 2 * ks + (mat & 1);
                const uint32_t addr = sK + (cg >> 3) * kBox + row * 128 + (((cg & 7) ^ (row & 7)) << 4);
                uint32_t b0, b1, b2, b3;
                ldsm_x4(addr, b0, b1, b2, b3);
                mma16816(sc[2 * t16], qh[ks][0], ql[ks][0], qh[ks][1], ql[ks][1], b0, b1);
                mma16816(sc[2 * t16 + 1], qh[ks][0], ql[ks][0], qh[ks][1], ql[ks][1], b2, b3);
            }
        }
        float mx = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int tok = nt * 8 + 2 * tq + e;
                const float v = (tok < lim) ? sc[nt][e] + sc[nt][e + 2] : -INFINITY;  // hi + lo parts
                sc[nt][e] = v;
                mx = fmaxf(mx, v);
            }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m_run, mx);
        float scale = 1.f, psum = 0.f;
        if (m_new == -INFINITY) {
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) sc[nt][0] = sc[nt][1] = 0.f;
        } else {
            scale = (m_run == -INFINITY) ? 0.f : __expf(m_run - m_new);
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const float p = (sc[nt][e] == -INFINITY) ? 0.f : __expf(sc[nt][e] - m_new);
                    sc[nt][e] = p;
                    psum += p;
                }
        }
        m_run = m_new;
        l_run = l_run * scale + psum;
#pragma unroll
        for (int nt = 0; nt < kNTiles; ++nt) { o[nt][0] *= scale; o[nt][1] *= scale; o[nt][2] *= scale; o[nt][3] *= scale; }
        // ---- O[row][d] += P[row][token] V[token][d], 16 tokens at a time
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
            uint32_t ph0, pl0, ph1, pl1;
            split2(sc[2 * kk][0], sc[2 * kk][1], ph0, pl0);
            split2(sc[2 * kk + 1][0], sc[2 * kk + 1][1], ph1, pl1);
#pragma unroll
            for (int n2 = 0; n2 < kNTiles / 2; ++n2) {
                const int row = kk * 16 + (mat & 1) * 8 + r8;
                const int cg = 2 * n2 + (mat >> 1);
                const uint32_t addr = sV + (cg >> 3) * kBox + row * 128 + (((cg & 7) ^ (row & 7)) << 4);
                uint32_t b0, b1, b2, b3;
                ldsm_x4_t(addr, b0, b1, b2, b3);
                mma16816(o[2 * n2], ph0, pl0, ph1, pl1, b0, b1);
                mma16816(o[2 * n2 + 1], ph0, pl0, ph1, pl1, b2, b3);
            }
        }
        __syncwarp();
        // The last stages of a group are handed back only after the group's epilogue, which uses the ring's memory as
        // scratch: the producer, already asking for the next group's tiles, must not refill them meanwhile.
        if (lane == 0 && j < n_tiles - kStages)
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(empty_bar(s)) : "memory");
    }
    auto release_last_stages = [&]() {
        __syncwarp();
        if (lane == 0)
            for (int j = max(0, n_tiles - kStages); j < n_tiles; ++j)
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(empty_bar((tile0 + j) % kStages)) : "memory");
    };

    // ---- each warp's rows are complete for this chunk: hand them over through shared memory
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    bar_consumers();
    // Scratch = the stage of this group's LAST tile: the group holds it until release_last_stages, whereas any other
    // stage may already be receiving the next group's tiles.  A stage (2 x HD x 128 B) holds the 4 x GR x HD floats
    // and, later, the 2 x 32 x 64 merge weights.
    float* o_s = reinterpret_cast<float*>(base_ptr + (size_t)((tile0 + n_tiles - 1) % kStages) * kStageBytes);  // [4][GR][HD]
    float* m_s = o_s + 4 * GR * HD;                         // [4][GR]
    float* l_s = m_s + 4 * GR;                              // [4][GR]
    if (g < GR) {
#pragma unroll
        for (int nt = 0; nt < kNTiles; ++nt) {
            float2 v = make_float2(o[nt][0] + o[nt][2], o[nt][1] + o[nt][3]);
            *reinterpret_cast<float2*>(o_s + ((size_t)warp * GR + g) * HD + nt * 8 + 2 * tq) = v;
        }
        if (tq == 0) { m_s[warp * GR + g] = m_run; l_s[warp * GR + g] = l_run; }
    }
    bar_consumers();
    if (!ok || abort_s) return;  // (a wait gave up: every role of this CTA is on its way out)
    // element r of [4 warps][GR rows]: member 2*(r / GR) + (r % GR) / G, query head h*G + (r % GR) % G
    auto member_of = [&](int r) { return 2 * (r / GR) + (r % GR) / G; };
    auto hq_of = [&](int r) { return (size_t)(i + member_of(r)) * Hq + (size_t)h * G + (r % GR) % G; };
    auto emit = [&](size_t hq, int d, float y) {
        if (out) out[hq * HD + d] = y;
        if (out_hi) {
            const __nv_bfloat16 hh = __float2bfloat16_rn(y);
            out_hi[hq * HD + d] = hh;
            out_lo[hq * HD + d] = __float2bfloat16_rn(y - __bfloat162float(hh));
        }
    };
    constexpr int kRows = 4 * GR;
    for (int e = threadIdx.x; e < kRows * HD; e += kConsumers) {
        const int r = e / HD, d = e - r * HD;
        if (member_of(r) >= n_mem) continue;
        const float acc = o_s[(size_t)r * HD + d], M = m_s[r], l = l_s[r];
        if (n_chunks == 1) {
            emit(hq_of(r), d, acc / l);
        } else {
            o_part[(hq_of(r) * S_max + c) * HD + d] = acc;
            if (d == 0) ml_part[hq_of(r) * S_max + c] = make_float2(M, l);
        }
    }
    if (n_chunks == 1) {
        bar_consumers();  // everyone has read the scratch: the stages may be refilled
        release_last_stages();
        continue;
    }
    // ---- ticket: the last chunk of this (group, kv head) to get here merges them all.  A member that sees fewer
    // tokens than a chunk's first token has an empty partial there (max = -inf, sum = 0): weight zero.
    __threadfence();
    bar_consumers();
    if (threadIdx.x == 0) {
        const uint32_t t = atomicAdd(&ticket[(size_t)i * gridDim.y + h], 1u);
        last_s = (t == (uint32_t)n_chunks - 1u);
        if (last_s) ticket[(size_t)i * gridDim.y + h] = 0u;
    }
    bar_consumers();
    if (!last_s) {
        release_last_stages();
        continue;
    }
    __threadfence();
    float* w_s = o_s;  // [kRows][64] weights, then [kRows][64] sums: 16 KB, inside the same held stage
    for (int e = threadIdx.x; e < kRows * n_chunks; e += kConsumers) {
        const int r = e / n_chunks, sidx = e - r * n_chunks;
        float2 ml = make_float2(-INFINITY, 0.f);
        if (member_of(r) < n_mem) ml = __ldcg(&ml_part[hq_of(r) * S_max + sidx]);
        w_s[r * 64 + sidx] = ml.x;
        w_s[(kRows + r) * 64 + sidx] = ml.y;
    }
    bar_consumers();
    if (threadIdx.x < kRows) {
        const int r = threadIdx.x;
        float M = -INFINITY, den = 0.f;
        for (int sidx = 0; sidx < n_chunks; ++sidx) M = fmaxf(M, w_s[r * 64 + sidx]);
        for (int sidx = 0; sidx < n_chunks; ++sidx)
            den += (w_s[r * 64 + sidx] == -INFINITY) ? 0.f : w_s[(kRows + r) * 64 + sidx] * __expf(w_s[r * 64 + sidx] - M);
        const float inv = den > 0.f ? 1.f / den : 0.f;
        for (int sidx = 0; sidx < n_chunks; ++sidx)
            w_s[r * 64 + sidx] = (w_s[r * 64 + sidx] == -INFINITY) ? 0.f : __expf(w_s[r * 64 + sidx] - M) * inv;
    }
    bar_consumers();
    for (int e = threadIdx.x; e < kRows * HD; e += kConsumers) {
        const int r = e / HD, d = e - r * HD;
        if (member_of(r) >= n_mem) continue;
        const size_t hq = hq_of(r);
        const float* src = o_part + (hq * S_max) * HD + d;
        const float* wv = w_s + r * 64;
        float acc = 0.f;
        for (int sidx = 0; sidx < n_chunks; ++sidx)
            if (wv[sidx] != 0.f) acc += __ldcg(src + (size_t)sidx * HD) * wv[sidx];
        emit(hq, d, acc);
    }
    bar_consumers();
    release_last_stages();
  }  // groups that start in this CTA's eight rows
    if (warp == 4 && lane == 0) {
        // leaves only when every copy it issued has landed (see attn_split_mma)
        for (int jj = max(0, issued_total - kStages); jj < issued_total; ++jj) {
            const uint32_t bar = full_bar(jj % kStages), ph = (uint32_t)(jj / kStages) & 1u;
            for (uint32_t it = 0; it < tc::kSpinLimit && !tc::mbar_try_wait(bar, ph); ++it) {}
        }
    }
}

}  // namespace attn
}  // namespace first
