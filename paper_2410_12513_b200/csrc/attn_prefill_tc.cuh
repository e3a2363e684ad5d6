// Causal attention for prompt chunks on the tcgen05 tensor cores ("Inference for FiRST", item 1: the prompt runs
// through every layer).  The rows of a launch are consecutive tokens of a few sequences, and at 256 rows per chunk
// the score and value products are a dense contraction: 128 x 64 x head_dim per tile and work item.
//
// Work item = (BLOCK of up to TQ = 128/G consecutive tokens of one sequence, KV head, chunk of the token axis).
// The block's tokens x the G query heads of the KV head are the 128 rows of the MMA (row = token * G + head), so
// one staged K/V tile serves all of them.  Per tile of 128 cached tokens:
//   S  = (Q_hi + Q_lo) K^T      tcgen05.mma, Q and K K-major in 128-byte-swizzled shared memory, S in tensor memory
//   P  = exp(S - max)           four warps, one row per thread (tcgen05.ld), causal mask, online softmax; the weights
//                               go back into the columns S came from as packed bfloat16 pairs (tcgen05.st)
//   O += (P_hi + P_lo) V        tcgen05.mma with A = P read from tensor memory, V as the TMA left it ([token][dim]:
//                               an MN-major B operand); O stays in tensor memory over all tiles of the block
// The weights are taken relative to a reference maximum m_ref that follows the running maximum lazily: only when
// a tile's maximum exceeds m_ref by more than 8 (base-2 exponent) is m_ref moved and O (and the running sum)
// scaled down; in between weights may be as large as 2^8, which float32 sums and the bfloat16 hi/lo split carry
// without loss.  O / sum at the end does not depend on which reference was used.
// Operands fetched from shared memory cost the tensor pipe time (measured: about 64 bytes per clock, so a
// 128 x 64 x 16 MMA with both operands there takes 90 clocks instead of 32): hence tiles of 128 tokens for S and P
// kept in tensor memory for PV.  Precision is that of the other attention kernels: q and the softmax weights are
// split into bfloat16 hi + lo against the stored bfloat16 keys and values, float32 accumulation.  S/P is
// double-buffered in tensor memory, so the tensor pipe computes S of tile j+1 while the softmax warps work on tile j.
// The token axis is cut into chunks per CTA; the CTA that finishes a (block, kv head) last merges the chunks
// (atomic ticket), as in the decode kernel.
//
// Roles (320 threads): warp 0 lane 0 = TMA producer, warp 1 lane 0 = MMA issuer (warp 1 owns the tensor memory),
// warps 2..5 and 6..9 = two softmax warpgroups (tensor-memory lane quadrant = warp % 4): a row of the tile belongs
// to one thread of each, the first takes tokens 0..63 of every tile and the first half of the output row, the second
// the rest; they exchange their row maxima through shared memory once per tile (one warp per scheduler alone spends
// its time waiting for its own exp2 and tensor-memory results).  Every wait is bounded.
#pragma once
#include "attn_mma.cuh"

namespace first {
namespace attn {

constexpr int kTcThreads = 320;   // producer warp, MMA warp, two softmax warpgroups
constexpr int kTcMaxRows = 256;  // rows of a launch (a prompt chunk)

// MN-major operand in 128-byte-swizzled rows (row = one K index, 64 MN elements wide): 8-row groups 1024 bytes
// apart along K, 64-element column groups lbo_bytes apart along MN.
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t addr, uint32_t lbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
__device__ __forceinline__ void tmem_ld16_nowait(uint32_t taddr, uint32_t* v) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* v) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
          "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]) : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t* v) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// D[tmem] (+)= A[tmem] * B[smem]: A's row i sits in lane i, two consecutive K elements per 32-bit column
__device__ __forceinline__ void umma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t db, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}"
        ::"r"(tmem_d), "r"(tmem_a), "l"(db), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// (x, y) -> packed bfloat16 pairs hi and lo with hi + lo = x (y) to 16 significant bits: hi is x cut off after
// 8 bits, lo the exact remainder cut off after 8 more (no conversion instructions: masks, subtractions, byte picks)
__device__ __forceinline__ void split2_trunc(float x, float y, uint32_t& hi, uint32_t& lo) {
    const uint32_t xb = __float_as_uint(x), yb = __float_as_uint(y);
    hi = __byte_perm(xb, yb, 0x7632);
    const float xl = x - __uint_as_float(xb & 0xffff0000u), yl = y - __uint_as_float(yb & 0xffff0000u);
    lo = __byte_perm(__float_as_uint(xl), __float_as_uint(yl), 0x7632);
}
__device__ __forceinline__ void bar_softmax() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
// the two warps (one of each warpgroup) that share a tensor-memory lane quadrant: barriers 2..5
__device__ __forceinline__ void bar_quadrant(int quad) { asm volatile("bar.sync %0, 64;" ::"r"(2 + quad) : "memory"); }
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

template <int HD, int G>
struct PrefillTc {
    static constexpr int TQ = 128 / G;                     // tokens of a block
    static constexpr int kTok = 128;                       // cached tokens per tile
    static constexpr int kHalves = HD / 64;                // 64-element column groups of a row
    static constexpr int kBox = kTile * 128;               // one TMA box: 64 tokens x 64 elements
    static constexpr int kHalfBytes = kTok * 128;          // 128 rows x 64 elements (Q rows, or a tile's tokens)
    static constexpr int kTileBytes = kHalves * kHalfBytes;  // a K tile or a V tile
    static constexpr int kQBytes = 2 * kTileBytes;         // hi halves, then lo halves
    static constexpr int kSmem = kQBytes + 4 * kTileBytes + 1024;  // Q, two K tiles, two V tiles
    static constexpr int kTmemCols = 512;  // S/P: 2 x 128 columns, O: HD columns (power of two)
};

// grid (Hkv, Z, S_max), 320 threads, at most 256 rows: CTA (h, z, c) serves the z-th, (z+Z)-th, ... block of the
// launch (so with Z >= the number of blocks, one each; the host takes Z = ceil(m / TQ) + 1, which covers a chunk that
// lies inside one sequence) for KV head h and token chunk c; chunks are the slowest grid dimension, so the CTAs
// of chunks that few rows reach come last.  A block starts at row i when i is the launch's first row, when row i is
// not the token after row i-1 of the same slab, or when its position is a multiple of TQ; it runs to the next start.
// rowinfo[i] = (tokens row i attends over incl. itself | batch row << 32, first slab row) from rope_append (mode 0).
// q: [m][Hq][HD] float32, rotated and pre-scaled.  tmK/tmV: [Hkv*cap_total][HD] bf16, box 64 x 64.  Scratch and
// outputs as in attn_split_mma (o_part [m][Hq][S_max][HD], ml_part [m][Hq][S_max], ticket [m][Hkv]).
// slack_log2: how far (base-2 exponent) a tile's maximum may exceed the reference maximum before the reference moves
// (8 in production; 0 = it follows the running maximum exactly, which exercises the rescaling of O on most tiles).
template <int HD, int G>
__global__ void __launch_bounds__(kTcThreads, 1)  // (ten warps: three share a scheduler's registers, 168 each)
attn_prefill_tc(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const float* q,
                int64_t cap_total, const longlong2* rowinfo, int m, const int32_t* __restrict__ m_dev, int Hq, int C,
                float* __restrict__ o_part, float2* __restrict__ ml_part, uint32_t* __restrict__ ticket,
                float* __restrict__ out, __nv_bfloat16* __restrict__ out_hi, __nv_bfloat16* __restrict__ out_lo,
                uint32_t* __restrict__ flags, float slack_log2, uint64_t* stamp) {
    const Stamp stamp_guard(stamp);
    using P = PrefillTc<HD, G>;
    constexpr int TQ = P::TQ, kTok = P::kTok, kHalves = P::kHalves, kBox = P::kBox, kHalfBytes = P::kHalfBytes;
    constexpr int kTileBytes = P::kTileBytes;
    constexpr int kRows = TQ * G;        // MMA rows that can carry a query head (the rest stay zero)
    constexpr int kOCol0 = 2 * kTok;     // tensor-memory column of the output accumulator

    pdl_trigger();
    if (m_dev) m = min(m, __ldg(m_dev));
    m = min(m, kTcMaxRows);
    __shared__ uint64_t bar_mem[16];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ int last_s;
    __shared__ uint32_t lead_s[kTcMaxRows / 32];  // bit i = row i starts a block
    __shared__ float xch_s[2][2][128];            // [tile parity][warpgroup][row]: row maxima (sums at the end)
    __shared__ int32_t t1_s[kTcMaxRows], slab_s[kTcMaxRows];  // row facts: tokens attended over, first slab row
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h = blockIdx.x, c = blockIdx.z, Hkv = gridDim.x, S_max = gridDim.z;
    const int Ce = (C + kTok - 1) / kTok * kTok;  // chunk length in whole tiles
    pdl_wait();  // (row facts come from the kernel before this one)
    auto t1_of = [&](int i) { return t1_s[i]; };
    auto slab_of = [&](int i) { return slab_s[i]; };  // (< 2^31: the tensor map's row count is)
    // ---- block starts: eight warps' worth of rows, a ballot each
    for (int wbase = warp * 32; wbase < kTcMaxRows; wbase += (kTcThreads / 32) * 32) {
        const int i = wbase + lane;
        bool st = false;
        if (i < m) {
            const longlong2 a = __ldcg(&rowinfo[i]);
            const int t1 = (int)(a.x & 0xffffffffll);
            t1_s[i] = t1;
            slab_s[i] = (int)(a.y & 0x7fffffffll);
            if (i == 0) {
                st = true;
            } else {
                const longlong2 pr = __ldcg(&rowinfo[i - 1]);
                st = (a.y & 0x7fffffffll) != (pr.y & 0x7fffffffll) || t1 != (int)(pr.x & 0xffffffffll) + 1 || (t1 - 1) % TQ == 0;
            }
        }
        const uint32_t bits = __ballot_sync(0xffffffffu, st);
        if (lane == 0) lead_s[wbase >> 5] = bits;
    }
    __syncthreads();
    int n_blocks = 0;
#pragma unroll
    for (int wd = 0; wd < kTcMaxRows / 32; ++wd) n_blocks += __popc(lead_s[wd]);
    // k-th block of the launch -> (first row, rows)
    auto block_at = [&](int k, int& i0, int& n) {
        int wd = 0;
        for (; wd < kTcMaxRows / 32; ++wd) {
            const int cnt = __popc(lead_s[wd]);
            if (k < cnt) break;
            k -= cnt;
        }
        i0 = wd * 32 + (int)__fns(lead_s[wd], 0, k + 1);
        n = 1;  // rows up to the next start, the end of the launch, or TQ
        while (n < TQ && i0 + n < m && !((lead_s[(i0 + n) >> 5] >> ((i0 + n) & 31)) & 1u)) ++n;
    };
    // this CTA's blocks that reach its chunk: none -> leave before anything is set up
    bool any = false;
    for (int k = blockIdx.y; k < n_blocks && !any; k += gridDim.y) {
        int i0, n;
        block_at(k, i0, n);
        any = c < (t1_of(i0) + n - 1 + Ce - 1) / Ce;
    }
    if (!any) return;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - tc::smem_u32(smem_raw));
    const uint32_t q_sm = base, k_sm = base + P::kQBytes, v_sm = k_sm + 2 * kTileBytes;
    auto k_full = [&](int s) { return tc::smem_u32(&bar_mem[s]); };
    auto k_empty = [&](int s) { return tc::smem_u32(&bar_mem[2 + s]); };
    auto v_full = [&](int s) { return tc::smem_u32(&bar_mem[4 + s]); };
    auto v_empty = [&](int s) { return tc::smem_u32(&bar_mem[6 + s]); };
    auto s_full = [&](int b) { return tc::smem_u32(&bar_mem[8 + b]); };
    auto p_full = [&](int b) { return tc::smem_u32(&bar_mem[10 + b]); };
    auto pv_full = [&](int b) { return tc::smem_u32(&bar_mem[12 + b]); };
    const uint32_t q_full = tc::smem_u32(&bar_mem[14]), done_bar = tc::smem_u32(&bar_mem[15]);

    if (threadIdx.x == 0) {
        abort_s = 0;
        for (int b = 0; b < 2; ++b) {
            tc::mbar_init(k_full(b), 1);
            tc::mbar_init(k_empty(b), 1);
            tc::mbar_init(v_full(b), 1);
            tc::mbar_init(v_empty(b), 1);
            tc::mbar_init(s_full(b), 1);
            tc::mbar_init(p_full(b), 8);
            tc::mbar_init(pv_full(b), 1);
        }
        tc::mbar_init(q_full, 8);
        tc::mbar_init(done_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(tc::smem_u32(&tmem_base_s)), "r"((uint32_t)P::kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = tmem_base_s;

    // Tiles and blocks this CTA has been through: ring stages, buffer parities and barrier phases go on from one
    // block to the next, and every role advances the counts by the same amounts.
    int tiles_done = 0, blocks_done = 0, issued_total = 0;
    bool mma_issued = false;

    for (int kb = blockIdx.y; kb < n_blocks; kb += gridDim.y) {
        int i0, n;
        block_at(kb, i0, n);
        const int T1 = t1_of(i0);                   // tokens the block's first row attends over
        const int64_t slab0 = slab_of(i0);
        const int T = T1 + n - 1;                   // tokens streamed: the last row's view
        const int n_chunks = (T + Ce - 1) / Ce;
        if (c >= n_chunks) continue;
        const int Cb = ((T + n_chunks - 1) / n_chunks + kTok - 1) / kTok * kTok;
        const int t_begin = c * Cb;
        if (t_begin >= T) continue;
        const int t_end = min(T, t_begin + Cb);
        const int n_tiles = (t_end - t_begin + kTok - 1) / kTok;
        const int tile0 = tiles_done, blk = blocks_done;
        tiles_done += n_tiles;
        ++blocks_done;

        if (warp == 0) {  // ---------------- producer: K tile j, then V tile j, two of each in flight
            if (lane == 0 && !abort_s) {
                const int64_t row0 = (int64_t)h * cap_total + slab0 + t_begin;
                for (int j = 0; j < n_tiles; ++j, ++issued_total) {
                    const int jj = tile0 + j, s = jj & 1;
                    const uint32_t ph = (uint32_t)(jj >> 1) & 1u;
                    const int row = (int)(row0 + (int64_t)j * kTok);
                    if (!tc::mbar_wait(k_empty(s), ph ^ 1u, &abort_s, flags)) break;
                    tc::mbar_expect_tx(k_full(s), kTileBytes);
#pragma unroll
                    for (int hf = 0; hf < kHalves; ++hf)  // (prefixes are re-read by the next block: default L2 policy)
#pragma unroll
                        for (int bx = 0; bx < kTok / kTile; ++bx)
                            tc::tma_load_2d(k_sm + s * kTileBytes + hf * kHalfBytes + bx * kBox, &tmK, k_full(s), hf * 64,
                                            row + bx * kTile);
                    if (!tc::mbar_wait(v_empty(s), ph ^ 1u, &abort_s, flags)) { ++issued_total; break; }  // (K of this tile is in flight)
                    tc::mbar_expect_tx(v_full(s), kTileBytes);
#pragma unroll
                    for (int hf = 0; hf < kHalves; ++hf)
#pragma unroll
                        for (int bx = 0; bx < kTok / kTile; ++bx)
                            tc::tma_load_2d(v_sm + s * kTileBytes + hf * kHalfBytes + bx * kBox, &tmV, v_full(s), hf * 64,
                                            row + bx * kTile);
                }
            }
            continue;
        }
        if (warp == 1) {  // ---------------- MMA issuer
            if (lane == 0 && !abort_s) {
                const uint32_t idesc_s = tc::instr_desc_bf16(kTok);
                const uint32_t idesc_pv = tc::instr_desc_bf16(HD) | (1u << 16);  // B (= V) is MN-major
                bool ok = tc::mbar_wait(q_full, (uint32_t)blk & 1u, &abort_s, flags);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                // descriptors differ from a base only in the start address (16-byte units in the low bits)
                const uint64_t dq = tc::smem_desc_sw128(q_sm), dk0 = tc::smem_desc_sw128(k_sm);
                const uint64_t dv0 = smem_desc_mn_sw128(v_sm, kHalfBytes);
                auto issue_s = [&](int j) {  // S of tile j: 2 x HD/16 MMAs of 128 x 128 x 16
                    const int jj = tile0 + j, s = jj & 1;
                    if (!tc::mbar_wait(k_full(s), (uint32_t)(jj >> 1) & 1u, &abort_s, flags)) return false;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint64_t dk = dk0 + (uint64_t)((uint32_t)s * (kTileBytes >> 4));
                    const uint32_t td = tmem + (uint32_t)(s * kTok);
#pragma unroll
                    for (int part = 0; part < 2; ++part)  // q_hi, then q_lo
#pragma unroll
                        for (int k = 0; k < HD / 16; ++k) {
                            const uint32_t off = (uint32_t)(((k >> 2) * kHalfBytes + (k & 3) * 32) >> 4);
                            tc::umma_bf16(td, dq + (uint64_t)(off + ((part * kTileBytes) >> 4)), dk + (uint64_t)off, idesc_s,
                                          (part | k) ? 1u : 0u);
                        }
                    tc::umma_commit(k_empty(s));  // the K tile is free once these MMAs have read it
                    tc::umma_commit(s_full(s));
                    mma_issued = true;
                    return true;
                };
                ok = ok && issue_s(0);
                for (int j = 0; j < n_tiles && ok; ++j) {
                    const int jj = tile0 + j, b = jj & 1;
                    const uint32_t ph = (uint32_t)(jj >> 1) & 1u;
                    if (j + 1 < n_tiles && !issue_s(j + 1)) break;
                    if (!tc::mbar_wait(p_full(b), ph, &abort_s, flags)) break;
                    if (!tc::mbar_wait(v_full(b), ph, &abort_s, flags)) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint64_t dv = dv0 + (uint64_t)((uint32_t)b * (kTileBytes >> 4));
                    const uint32_t ta = tmem + (uint32_t)(b * kTok);   // P where S was: per 64 tokens 32 columns hi, 32 lo
                    const uint32_t td = tmem + (uint32_t)kOCol0;
#pragma unroll
                    for (int part = 0; part < 2; ++part)  // p_hi, then p_lo
#pragma unroll
                        for (int k = 0; k < kTok / 16; ++k)
                            umma_bf16_ts(td, ta + (uint32_t)((k >> 2) * 64 + part * 32 + (k & 3) * 8), dv + (uint64_t)((k * 2048) >> 4),
                                         idesc_pv, (j | part | k) ? 1u : 0u);  // the block's first MMA starts O afresh
                    tc::umma_commit(v_empty(b));  // the V tile is free once these MMAs have read it
                    tc::umma_commit(pv_full(b));
                }
            }
            continue;
        }

        // ---------------- softmax warpgroups: a row of the tile = one thread of each
        const int st = (int)threadIdx.x - 64, wg = st >> 7;   // wg: which half of the tile's tokens and of the output row
        const int quad = warp & 3, r = quad * 32 + lane;
        const int tok = r / G, gq = r - tok * G;
        const bool live = r < kRows && tok < n;
        const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
        constexpr int HH = HD / 2;  // output columns of a thread
        {   // Q of this block: float32 -> bfloat16 hi/lo, K-major swizzled rows (the previous block's MMAs are done:
            // its last PV was waited for).  Warp w converts rows 16w .. 16w+15.
            const int sw = warp - 2;
#pragma unroll 16
            for (int e = lane; e < 16 * HD / 4; e += 32) {
                const int rq = sw * 16 + e / (HD / 4), d4 = (e % (HD / 4)) * 4;
                const int tq = rq / G, gg = rq - tq * G;
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if (rq < kRows && tq < n)
                    v = *reinterpret_cast<const float4*>(q + ((size_t)(i0 + tq) * Hq + (size_t)h * G + gg) * HD + d4);
                uint2 hi, lo;
                split2(v.x, v.y, hi.x, lo.x);
                split2(v.z, v.w, hi.y, lo.y);
                const int dd = d4 & 63;
                const uint32_t off = (uint32_t)((d4 >> 6) * kHalfBytes + rq * 128 + (((dd >> 3) ^ (rq & 7)) << 4) + (dd & 7) * 2);
                *reinterpret_cast<uint2*>(base_ptr + off) = hi;
                *reinterpret_cast<uint2*>(base_ptr + kTileBytes + off) = lo;
            }
            fence_async_smem();
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");  // (the previous block's tensor-memory reads)
            __syncwarp();
            if (lane == 0) mbar_arrive(q_full);
        }
        float m_ref = -INFINITY, l_run = 0.f;
        // A failed wait makes `ok` false for good, for the whole warp (the tensor-memory instructions below want the
        // warp together); the warp still goes through every barrier of the loop (its partner and the other warps
        // wait there), only the work is skipped.
        bool ok = true;
        // this row sees tokens t < see of this chunk's range; a row without a query head (all-zero q) is never
        // written out and takes the unmasked path
        const int see = live ? min(T1 + tok, t_end) : 0x7fffffff;
        constexpr float kLog2e = 1.4426950408889634f;
        const float kSlack = slack_log2 / kLog2e;  // m_ref moves only when a tile's maximum is this far above it
        const uint32_t o_addr = lane_addr + (uint32_t)(kOCol0 + wg * HH);  // this thread's half of the output row
        for (int j = 0; j < n_tiles; ++j) {
            const int jj = tile0 + j, b = jj & 1;
            ok = __all_sync(0xffffffffu, ok && tc::mbar_wait(s_full(b), (uint32_t)(jj >> 1) & 1u, &abort_s, flags));
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t s_addr = lane_addr + (uint32_t)(b * kTok + wg * 64);  // this thread's 64 columns
            const int t0 = t_begin + j * kTok;
            const int lim = see - t0 - wg * 64;  // columns of this thread's half the row sees
            const bool whole = lim >= 64;        // every column visible: the usual case away from the diagonal
            uint32_t sv[64];
            float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
            if (ok) {
#pragma unroll
                for (int c0 = 0; c0 < 64; c0 += 16) tmem_ld16_nowait(s_addr + (uint32_t)c0, sv + c0);
                tmem_ld_wait();
                if (whole) {
#pragma unroll
                    for (int k = 0; k < 64; ++k) mx4[k & 3] = fmaxf(mx4[k & 3], __uint_as_float(sv[k]));
                } else {
#pragma unroll
                    for (int k = 0; k < 64; ++k) {
                        if (k >= lim) sv[k] = 0xff800000u;  // -inf: weight 0
                        mx4[k & 3] = fmaxf(mx4[k & 3], __uint_as_float(sv[k]));
                    }
                }
            }
            float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
            xch_s[b][wg][r] = mx;
            bar_quadrant(quad);  // only the partner warp holds the other half of these rows
            mx = fmaxf(mx, xch_s[b][wg ^ 1][r]);  // (written again two tiles on, a barrier later)
            float alpha = 1.f;
            if (m_ref == -INFINITY) {
                m_ref = mx;  // first visible column (or still none): nothing accumulated yet
            } else if (mx > m_ref + kSlack) {
                alpha = ex2_approx((m_ref - mx) * kLog2e);
                m_ref = mx;
                l_run *= alpha;
            }
            const float mb = (m_ref == -INFINITY) ? 0.f : m_ref * kLog2e;  // (then no column is visible: weights 0)
            // weights, their sum, and P back into the columns S came from: 32 columns of bfloat16 pairs (hi), then
            // 32 (lo) -- exactly this thread's 64 columns, whose S values are in its registers
            float sum4[4] = {0.f, 0.f, 0.f, 0.f};
            if (ok) {
#pragma unroll
                for (int qd = 0; qd < 4; ++qd) {  // 16 tokens -> 8 columns hi, 8 columns lo
                    uint32_t phi[8], plo[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const int col = qd * 16 + 2 * k;
                        const float p0 = ex2_approx(fmaf(__uint_as_float(sv[col]), kLog2e, -mb));
                        const float p1 = ex2_approx(fmaf(__uint_as_float(sv[col + 1]), kLog2e, -mb));
                        sum4[k & 3] += p0 + p1;
                        split2_trunc(p0, p1, phi[k], plo[k]);
                    }
                    tmem_st8(s_addr + (uint32_t)(qd * 8), phi);
                    tmem_st8(s_addr + (uint32_t)(32 + qd * 8), plo);
                }
            }
            l_run += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
            if (t0 + kTok > T) {
                // rows past the sequence's end hold someone else's bytes: zero them in V so that 0 * garbage stays 0
                const int valid = T - t0;
                ok = __all_sync(0xffffffffu, ok && tc::mbar_wait(v_full(b), (uint32_t)(jj >> 1) & 1u, &abort_s, flags));
                uint8_t* vptr = base_ptr + P::kQBytes + 2 * kTileBytes + (size_t)b * kTileBytes;
                if (ok)
                    for (int e = st; e < (kTok - valid) * kHalves * 8; e += 256) {
                        const int row = valid + e / (kHalves * 8), cc = e % (kHalves * 8);
                        *reinterpret_cast<uint4*>(vptr + (cc >> 3) * kHalfBytes + row * 128 + (cc & 7) * 16) = make_uint4(0, 0, 0, 0);
                    }
                fence_async_smem();
            }
            // O holds tiles 0 .. j-1 once PV of tile j-1 is done.  Waited for every tile (the barrier's phases are taken
            // in order) but only here, after the weights: by now that PV is over unless the tensor pipe is the slower side.
            if (j > 0) ok = __all_sync(0xffffffffu, ok && tc::mbar_wait(pv_full((jj - 1) & 1), (uint32_t)((jj - 1) >> 1) & 1u, &abort_s, flags));
            if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f) && ok) {
                // some row of this warp moved its reference: scale this warp's rows of O (1 for the others)
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
                for (int c0 = 0; c0 < HH; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld16_nowait(o_addr + (uint32_t)c0, v);
                    tmem_ld16_nowait(o_addr + (uint32_t)(c0 + 16), v + 16);
                    tmem_ld_wait();
#pragma unroll
                    for (int k = 0; k < 32; ++k) v[k] = __float_as_uint(__uint_as_float(v[k]) * alpha);
                    tmem_st16(o_addr + (uint32_t)c0, v);
                    tmem_st16(o_addr + (uint32_t)(c0 + 16), v + 16);
                }
            }
            tmem_st_wait();
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0 && ok) mbar_arrive(p_full(b));
        }
        // the block's output: O is complete once the last PV is
        ok = __all_sync(0xffffffffu, ok && tc::mbar_wait(pv_full((tile0 + n_tiles - 1) & 1), (uint32_t)((tile0 + n_tiles - 1) >> 1) & 1u, &abort_s, flags));
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        float o[HH];
        if (ok) {
#pragma unroll
            for (int c0 = 0; c0 < HH; c0 += 16) tmem_ld16_nowait(o_addr + (uint32_t)c0, reinterpret_cast<uint32_t*>(o) + c0);
            tmem_ld_wait();
        }
        // the row's sum: both halves
        xch_s[0][wg][r] = l_run;
        bar_softmax();
        const float l_tot = l_run + xch_s[0][wg ^ 1][r];
        bar_softmax();  // (xch_s is written again by the next block's first tile)
        ok = ok && !abort_s;
        // ---------------- epilogue: the thread holds its half of the row's unnormalised output, the maximum and the sum
        const size_t hq = ((size_t)(i0 + tok) * Hq + (size_t)h * G + gq);
        if (n_chunks == 1) {
            if (ok && live) {
                const float scale = 1.f / l_tot;
                const size_t o0 = hq * HD + (size_t)wg * HH;
                if (out) {
#pragma unroll
                    for (int d = 0; d < HH; d += 4)
                        *reinterpret_cast<float4*>(out + o0 + d) =
                            make_float4(o[d] * scale, o[d + 1] * scale, o[d + 2] * scale, o[d + 3] * scale);
                }
                if (out_hi) {
#pragma unroll
                    for (int d = 0; d < HH; d += 8) {
                        uint4 hi, lo;
                        split2(o[d] * scale, o[d + 1] * scale, hi.x, lo.x);
                        split2(o[d + 2] * scale, o[d + 3] * scale, hi.y, lo.y);
                        split2(o[d + 4] * scale, o[d + 5] * scale, hi.z, lo.z);
                        split2(o[d + 6] * scale, o[d + 7] * scale, hi.w, lo.w);
                        *reinterpret_cast<uint4*>(out_hi + o0 + d) = hi;
                        *reinterpret_cast<uint4*>(out_lo + o0 + d) = lo;
                    }
                }
            }
            continue;
        }
        if (ok && live) {
#pragma unroll
            for (int d = 0; d < HH; d += 4)
                *reinterpret_cast<float4*>(o_part + (hq * S_max + c) * HD + wg * HH + d) = make_float4(o[d], o[d + 1], o[d + 2], o[d + 3]);
            if (wg == 0) ml_part[hq * S_max + c] = make_float2(m_ref, l_tot);
        }
        // ticket: the last chunk of this (block, kv head) to get here merges them all
        __threadfence();
        bar_softmax();
        if (threadIdx.x == 64) {
            const uint32_t t = ok ? atomicAdd(&ticket[(size_t)i0 * Hkv + h], 1u) : 0u;
            last_s = ok && (t == (uint32_t)n_chunks - 1u);
            if (last_s) ticket[(size_t)i0 * Hkv + h] = 0u;
        }
        bar_softmax();
        const bool last = last_s != 0;
        bar_softmax();  // (last_s is written again by the next block)
        if (!last) continue;
        __threadfence();
        // Merge, all 256 threads side by side (a thread per row would wait for one load after the other):
        // (1) every chunk's (max, sum) into shared memory -- Q's memory is free, the block's MMAs are done --
        // (2) one weight per (row, chunk), (3) weighted sums, eight (sixteen) rows per pass with coalesced loads.
        {
            const int rows_live = n * G, tid = st;
            float2* w_s = reinterpret_cast<float2*>(base_ptr);  // [rows_live][n_chunks]
            auto hq_of = [&](int rw) { return (size_t)(i0 + rw / G) * Hq + (size_t)h * G + rw % G; };
            for (int e = tid; e < rows_live * n_chunks; e += 256) {
                const int rw = e / n_chunks, sidx = e - rw * n_chunks;
                w_s[e] = __ldcg(&ml_part[hq_of(rw) * S_max + sidx]);
            }
            bar_softmax();
            if (tid < rows_live) {
                float2* wr = w_s + tid * n_chunks;
                float M = -INFINITY, den = 0.f;
                for (int sidx = 0; sidx < n_chunks; ++sidx) M = fmaxf(M, wr[sidx].x);
                for (int sidx = 0; sidx < n_chunks; ++sidx) den += wr[sidx].y * __expf(wr[sidx].x - M);
                const float inv = 1.f / den;
                for (int sidx = 0; sidx < n_chunks; ++sidx) wr[sidx].x = __expf(wr[sidx].x - M) * inv;
            }
            bar_softmax();
            constexpr int LPR = HD / 4, RPP = 256 / LPR;  // lanes per row (a float4 each), rows per pass
            const int d4 = (tid % LPR) * 4;
#pragma unroll 2
            for (int rb = 0; rb < rows_live; rb += RPP) {
                const int rw = rb + tid / LPR;
                if (rw < rows_live) {
                    const size_t hqr = hq_of(rw);
                    const float4* src = reinterpret_cast<const float4*>(o_part + hqr * S_max * HD + d4);
                    const float2* wr = w_s + rw * n_chunks;
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
                    for (int sidx = 0; sidx < n_chunks; ++sidx) {
                        const float4 v = __ldcg(src + (size_t)sidx * (HD / 4));
                        const float w = wr[sidx].x;
                        acc.x += v.x * w;
                        acc.y += v.y * w;
                        acc.z += v.z * w;
                        acc.w += v.w * w;
                    }
                    if (out) *reinterpret_cast<float4*>(out + hqr * HD + d4) = acc;
                    if (out_hi) {
                        uint2 hi, lo;
                        split2(acc.x, acc.y, hi.x, lo.x);
                        split2(acc.z, acc.w, hi.y, lo.y);
                        *reinterpret_cast<uint2*>(out_hi + hqr * HD + d4) = hi;
                        *reinterpret_cast<uint2*>(out_lo + hqr * HD + d4) = lo;
                    }
                }
            }
            bar_softmax();  // (the next block's Q goes where the weights are)
        }
    }

    // ---------------- leave: no copy in flight, no MMA in flight, tensor memory given back
    if (warp == 0 && lane == 0) {
        // every copy issued has landed (the last use of each stage; earlier uses were consumed before the refill)
        for (int j = max(0, issued_total - 2); j < issued_total; ++j) {
            const uint32_t ph = (uint32_t)(j >> 1) & 1u;
            for (uint32_t it = 0; it < tc::kSpinLimit && !tc::mbar_try_wait(k_full(j & 1), ph); ++it) {}
            for (uint32_t it = 0; it < tc::kSpinLimit && !tc::mbar_try_wait(v_full(j & 1), ph); ++it) {}
        }
    }
    if (warp == 1 && lane == 0 && mma_issued) {
        // every MMA issued is done (operands that landed are consumed; in a normal run the softmax warps have
        // already waited for the last PV, so this returns at once)
        tc::umma_commit(done_bar);
        for (uint32_t it = 0; it < tc::kSpinLimit && !tc::mbar_try_wait(done_bar, 0u); ++it) {}
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)P::kTmemCols)
                     : "memory");
    }
}

}  // namespace attn
}  // namespace first
