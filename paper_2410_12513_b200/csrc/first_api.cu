// C ABI of the routed decode step: context, argument checks, launch sequence.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include <type_traits>
#include <unordered_map>

#include "attn_mma.cuh"
#include "attn_prefill.cuh"
#include "attn_prefill_tc.cuh"
#include "attn_simple.cuh"
#include "common.cuh"
#include "first.h"
#include "gemm_tc.cuh"
#include "gemm_tc2.cuh"
#include "gemv.cuh"
#include "prefill.cuh"
#include "router.cuh"
#include "step.cuh"

using namespace first;

#define CU_TRY(expr)                                                                                   \
    do {                                                                                               \
        cudaError_t e_ = (expr);                                                                       \
        if (e_ != cudaSuccess) {                                                                       \
            std::snprintf(g_last_cuda_error, sizeof g_last_cuda_error, "%s: %s", #expr, cudaGetErrorString(e_)); \
            return FIRST_E_CUDA;                                                                       \
        }                                                                                              \
    } while (0)

static thread_local char g_last_cuda_error[256] = "";

enum KernelClass { kClsStepBegin = 0, kClsRmsnorm, kClsGemv, kClsGemmTc, kClsRopeAppend, kClsAttn, kClsAttnCombine,
                   kClsSiluMul, kClsStepEnd, kClsRouterScores, kClsRouterFinalize, kClsPlan, kClsPrefillAux, kNumClasses };
static const char* const kClassNames[kNumClasses] = {"step_begin", "rmsnorm_rows", "gemv_rows", "gemm_tc",
                                                     "rope_append", "attn_split", "attn_combine", "silu_mul",
                                                     "step_end", "router_token_scores", "router_finalize",
                                                     "plan_compact", "prefill_aux"};

struct first_ctx {
    first_model_desc d{};
    const void *embed = nullptr, *lm_head = nullptr;
    const float* final_norm = nullptr;
    std::vector<const float*> attn_norm, ffn_norm;
    std::vector<const void*> wqkv, wo, w_gate_up, w_down;
    int qd = 0, kvd = 0, qkvd = 0, group = 0;
    int n_sm = 148;
    // scratch (device)
    float *x = nullptr, *xn = nullptr, *qkv = nullptr, *q = nullptr, *att = nullptr, *gu = nullptr, *act = nullptr;
    float *o_part = nullptr, *logits_int = nullptr, *tokscore = nullptr;
    __nv_bfloat16 *xh = nullptr, *xl = nullptr, *acth = nullptr, *actl = nullptr;  // hi/lo activation splits
    // TMA descriptors of the weight matrices (bf16 models)
    std::vector<CUtensorMap> tm_wqkv, tm_wo, tm_wgu, tm_wgu64, tm_wd;  // tm_wgu64: 64-row boxes (gate|up pairing)
    CUtensorMap tm_lm{};
    bool tc_ready = false;
    int pair_rows = 64;  // gate (= up) rows per tile of the fused gate/up projection; tm_wgu64 has boxes of this many rows
    struct KvMap { int64_t cap_total; CUtensorMap map; };
    std::unordered_map<const void*, KvMap> kv_maps;  // TMA descriptors of cache tensors, by base pointer
    float2 *ml_part = nullptr, *cs = nullptr;
    double* inv_freq = nullptr;
    int32_t *idx = nullptr, *cnt = nullptr, *slot = nullptr;
    uint32_t *flags = nullptr, *ticket = nullptr;
    longlong2* rowinfo = nullptr;  // per active row: (tokens to attend over, first slab row)
    int64_t tok_cap = 0;
    int max_splits = 16;
    int attn_chunk = -1;
    // plan (host side)
    std::vector<int32_t> cnt_h;
    int B = 0;
    bool has_mask = false;
    int64_t launches = 0;
    // per-kernel-class timing (off unless first_profile enables it)
    bool profiling = false;
    std::vector<cudaEvent_t> ev_pool;
    std::vector<int> ev_cls;  // class of event pair i (events 2i, 2i+1)
    double prof_ms[kNumClasses] = {};
    int64_t prof_launches[kNumClasses] = {};
    // CUDA graphs of whole steps, keyed by every pointer the step touches and the plan version
    struct StepGraph {
        std::vector<const void*> key;
        cudaGraphExec_t exec = nullptr;
        int64_t n_launches = 0;
        uint64_t last_use = 0;
    };
    std::vector<StepGraph> graphs;
    uint64_t plan_version = 0, use_clock = 0;  // plan_version: bumped by option and sampling changes
    uint8_t* mask_dev = nullptr;               // [max_batch][L]: device copy of a mask given on the host
    cudaStream_t cap_stream = nullptr;  // steps are recorded here (the caller's stream may be the default one)
    int use_graph = 1;
    int use_pdl = 1;
    bool pdl_next = false;  // the next kernel launch may overlap its predecessor (programmatic dependent launch)
    // in-step timing (option "stamp"): first-CTA start / last-warp end of every launch of a step
    int stamp_on = 0;
    uint64_t* stamps = nullptr;  // [2][kStampCap]: starts, ends
    int stamp_n = 0;
    std::vector<int> stamp_cls;
    // options
    int norm_threads_max = 512;   // threads per norm CTA (one row each): 512 measured 8 % faster in-step than 1024 at D = 4096
    int attn_cluster = 0;   // split attention rows merge through a thread-block cluster's shared memory
    int tc2_min_rows = 96;  // from this many rows on a projection launch uses the CTA-pair kernel (0 = never)
    int tc2_mt2_all = 0;    // CTA-pair kernel: two weight tiles per unit for the reducing epilogues too
    int max_gemv_rows = -1;
    int attn_simple = -1;
    int tc_use_lo = 1;
    int fuse_swiglu = 1;
    int fuse_rope = 1;  // the tuned attention kernel rotates q and appends the new key/value itself
    int prefill_pair = 1;  // prompt chunks: two consecutive tokens of a sequence share one attention work item
    int prefill_group = 1; // prompt chunks: up to eight consecutive tokens share one (takes precedence over pairs)
    int prefill_lo = 1;    // 0 = prompt chunks' projections multiply by the bfloat16 hi half of the activations alone
    int prefill_slack = 8; // (its reference maximum moves when a tile's maximum exceeds it by more than 2^this)
    int prefill_tc = 1;    // prompt chunks: attention on the tcgen05 tensor cores, blocks of 128/G tokens (takes precedence over groups)
    int prefill_rows = 0;  // rows per prompt chunk (0: 256)
    int tune_pair_rows = 1;
    int tc_smem_kb = 110;  // shared-memory budget per projection CTA when two CTAs per SM are wanted
    int tc_lo_max_rows = 1 << 30;  // the hi/lo activation split is used up to this many active rows, hi alone above
    int tc_mt2_min_rows = -1;  // from this many active rows on, a projection CTA takes two weight tiles (-1: by shape)
    int tc_ksplit_cap = 1;          // bound the number of K ranges by the reduction traffic they add
    // sampling of the next token (greedy while sample_k <= 1)
    int sample_k = 0;
    float sample_inv_T = 1.f;
    const float* sample_u = nullptr;
    // batched prefill: per-row tables of a chunk (each prompt token is a row), an all-keep mask, the residual of
    // every sequence's last prompt token, and (allocated on first use) the per-layer token scores of the routers
    int32_t *pf_cu = nullptr, *pf_tok = nullptr, *pf_cap = nullptr, *pf_pos = nullptr, *pf_len = nullptr;
    int64_t* pf_off = nullptr;
    uint8_t* pf_ones = nullptr;
    float *x_last = nullptr, *pf_score = nullptr;
    int64_t pf_score_cap = 0;
};

// What a chunk of a batched prefill does beyond a decode step: router l scores the chunk's rows as they
// enter layer l (token scores of layer l at tokscore + l*stride + g0), and the step ends after the last layer.
struct PrefillHook {
    const float *router_w, *router_b;  // dev [L][D], dev [L] or nullptr
    int mode;
    float* tokscore;
    int64_t stride, g0;
};

constexpr int kSimpleSplitsMax = 16;

namespace {

template <typename T>
int dev_alloc(T** p, size_t n) {
    CU_TRY(cudaMalloc(reinterpret_cast<void**>(p), n * sizeof(T)));
    return FIRST_OK;
}

// Brackets one kernel launch: counts it and, when profiling, records an event pair around it.
struct Launch {
    first_ctx* c;
    cudaStream_t st;
    bool on;
    Launch(first_ctx* c_, cudaStream_t st_, int cls) : c(c_), st(st_), on(c_->profiling) {
        c->launches += 1;
        if (on) {
            const size_t i = c->ev_cls.size();
            while (c->ev_pool.size() < 2 * (i + 1)) {
                cudaEvent_t e;
                if (cudaEventCreate(&e) != cudaSuccess) { on = false; return; }
                c->ev_pool.push_back(e);
            }
            c->ev_cls.push_back(cls);
            cudaEventRecord(c->ev_pool[2 * i], st);
        }
    }
    ~Launch() {
        if (on) cudaEventRecord(c->ev_pool[2 * (c->ev_cls.size() - 1) + 1], st);
    }
};

// Timing slot of the next launch of a step (NULL while in-step timing is off or the table is full).
uint64_t* stamp_slot(first_ctx* c, int cls) {
    if (!c->stamp_on || !c->stamps || c->stamp_n >= kStampCap) return nullptr;
    c->stamp_cls.push_back(cls);
    return c->stamps + c->stamp_n++;
}

#define FIRST_LAUNCH(cls, ...)      \
    do {                            \
        Launch guard_(c, st, cls);  \
        __VA_ARGS__;                \
    } while (0)

// Launch through cudaLaunchKernelEx so that, inside a step, each kernel may start while its
// predecessor drains (programmatic stream serialization); kernels call griddepcontrol.wait
// before touching anything the predecessor produces.
template <typename... P, typename... A>
int launch_k(first_ctx* c, cudaStream_t st, int cls, void (*kern)(P...), dim3 grid, dim3 block, size_t smem,
             A&&... args) {
    Launch guard(c, st, cls);
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = (c->use_pdl && !c->profiling && c->pdl_next) ? 1 : 0;
    c->pdl_next = true;
    if constexpr (sizeof...(A) + 1 == sizeof...(P)) {
        // the kernel's last parameter is its in-step timing slot
        uint64_t* stamp = stamp_slot(c, cls);
        CU_TRY(cudaLaunchKernelEx(&cfg, kern, std::forward<A>(args)..., stamp));
    } else {
        CU_TRY(cudaLaunchKernelEx(&cfg, kern, static_cast<P>(args)...));
    }
    return FIRST_OK;
}

int check_launch(first_ctx*) {
    CU_TRY(cudaGetLastError());
    return FIRST_OK;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess) p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// 2-D bfloat16 row-major matrix [rows][cols] -> TMA descriptor with a [box_rows][64] box in
// 128-byte-swizzled rows; out-of-range elements read as zero.
int make_map(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows, bool weights) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return FIRST_E_CUDA;
    if ((reinterpret_cast<uintptr_t>(ptr) & 15u) || (cols * 2) % 16) return FIRST_E_UNSUPPORTED;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)tc::kBlockK, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    weights ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        std::snprintf(g_last_cuda_error, sizeof g_last_cuda_error, "cuTensorMapEncodeTiled failed with %d", (int)r);
        return FIRST_E_CUDA;
    }
    return FIRST_OK;
}

constexpr int kTcSmemMax = 210 * 1024;

// K ranges per weight tile for the reducing epilogues.  The CTAs of a projection should fill the
// GPU's CTA slots (SMs x CTAs that fit per SM) in whole waves: among the counts allowed, take the
// smallest whose last wave is nearly full.  Every range adds m*n_out float32 reductions: the count
// is kept below K / (4 m), so that this traffic stays under about half of the weight bytes.
int tc_ksplit(const first_ctx* c, int tiles, int K, int epi, int m, int slots) {
    if (epi == tc::kEpiStore || epi == tc::kEpiSwiglu) return 1;
    const int kblocks = (K + tc::kBlockK - 1) / tc::kBlockK;
    int cap = std::max(1, kblocks / 4);
    // ... except that idle SMs cost more than the reduction traffic: the bound never goes below the count that
    // fills one wave of the slots (256 rows: O projection 64 -> 144 work units on 148 SMs)
    if (c->tc_ksplit_cap)
        cap = std::min(cap, std::max(std::max(1, K / (4 * std::max(std::min(m, 256), 1))), slots / std::max(tiles, 1)));
    cap = std::min(cap, std::max(1, (2 * slots + tiles - 1) / tiles));  // never more than two waves' worth
    double best_eff = 0.0;
    for (int ks = 1; ks <= cap; ++ks) {
        const int units = tiles * ks, waves = (units + slots - 1) / slots;
        best_eff = std::max(best_eff, (double)units / ((double)waves * slots));
    }
    for (int ks = 1; ks <= cap; ++ks) {
        const int units = tiles * ks, waves = (units + slots - 1) / slots;
        if ((double)units / ((double)waves * slots) >= 0.97 * best_eff) return ks;
    }
    return 1;
}

// Launch shape of one tensor-core projection of mm (<= 256) compact rows: a pure function of the sizes and the
// options, so that the kernel BEFORE a projection can know which weight tiles that projection will ask for first.
struct TcShape {
    int n_pad, use_lo, mt, tile_rows, tiles, stage_bytes, stages, ksplit, acc_cols, tmem_cols, kblocks;
};
TcShape tc_shape(const first_ctx* c, int n_out, int K, int mm, int epi) {
    TcShape t{};
    t.n_pad = (mm + 15) / 16 * 16;
    t.kblocks = (K + tc::kBlockK - 1) / tc::kBlockK;
    t.use_lo = (c->tc_use_lo && mm <= c->tc_lo_max_rows) ? 1 : 0;
    // Two weight tiles per CTA share every activation tile.  Worth it exactly when the activation tiles are
    // so wide that only one single-tile CTA would fit per SM anyway (from 96 rows): the tile pair halves the
    // activation bytes an SM pulls from L2 per weight byte (config 3: -4 %; 115 rows: -16 % per step);
    // below that, two single-tile CTAs per SM overlap each other's set-up and epilogue and win.
    const int stage1 = tc::kABytes + t.n_pad * 128 * (t.use_lo ? 2 : 1);
    if (c->tc_mt2_min_rows >= 0) t.mt = (mm >= c->tc_mt2_min_rows) ? 2 : 1;
    else t.mt = (3 * stage1 > c->tc_smem_kb * 1024) ? 2 : 1;
    if (epi == tc::kEpiSwiglu && n_out % 128) t.mt = 1;
    t.tile_rows = epi == tc::kEpiSwiglu ? (t.mt == 1 ? c->pair_rows : 128) : tc::kBlockM * t.mt;
    t.tiles = (n_out + t.tile_rows - 1) / t.tile_rows;
    t.stage_bytes = tc::kABytes * t.mt + t.n_pad * 128 * (t.use_lo ? 2 : 1);
    const int budget = (3 * t.stage_bytes <= c->tc_smem_kb * 1024) ? c->tc_smem_kb * 1024 : 200 * 1024;
    const bool one_per_sm = budget != c->tc_smem_kb * 1024;
    t.stages = std::max(1, std::min(8, budget / t.stage_bytes));
    t.ksplit = tc_ksplit(c, t.tiles, K, epi, mm, c->n_sm * (one_per_sm ? 1 : 2));
    int cols = 32;
    while (cols < t.n_pad) cols *= 2;
    t.acc_cols = cols;
    t.tmem_cols = std::max(32, cols * t.mt);
    return t;
}

// The CTA-pair kernel (gemm_tc2.cuh) for launches of many rows.  Units = (group of two 256-row weight tiles, K
// range); the K ranges fill the SM pairs in whole waves.
constexpr int kTc2SmemMax = 231000;  // dynamic bytes; the kernels' static shared memory (about 1 KB) comes on top

bool tc2_wanted(const first_ctx* c, int mm, int n_out, int epi) {
    if (c->tc2_min_rows <= 0 || mm < c->tc2_min_rows || mm > 256) return false;
    if (epi == tc::kEpiSwiglu && n_out % 256) return false;
    return true;
}

int launch_gemm_tc2(first_ctx* c, cudaStream_t st, const CUtensorMap& tmA, int n_out, int K, const __nv_bfloat16* Xh,
                    const __nv_bfloat16* Xl, int mm, int r0, int epi, float* Y, int64_t ldy, const int32_t* idx,
                    bool pre_zeroed, float* act, __nv_bfloat16* act_hi, __nv_bfloat16* act_lo, const int32_t* m_dev) {
    int rc;
    tc::GemmParams p{};
    p.n_out = n_out; p.K = K; p.m = mm;
    p.n_pad = (mm + 31) / 32 * 32;  // half of the activation rows in each CTA, in whole 16-row groups
    p.kblocks = (K + tc::kBlockK - 1) / tc::kBlockK;
    p.use_lo = (c->tc_use_lo && mm <= c->tc_lo_max_rows) ? 1 : 0;
    // Two 256-row weight tiles per unit share every activation tile where the epilogue is cheap (plain stores,
    // SwiGLU).  The reducing epilogues take one tile per unit: the same SM pairs are then filled with half as many
    // K ranges, and every K range costs m x n_out float32 reductions (7 M per launch at 192 rows with the larger
    // units, which alone took 8 us).
    p.mt = (epi == tc::kEpiStore || epi == tc::kEpiSwiglu || c->tc2_mt2_all) ? 2 : 1;
    p.pair_rows = 0;
    const int tiles = epi == tc::kEpiSwiglu ? (n_out + 255) / 256 : (n_out + 256 * p.mt - 1) / (256 * p.mt);
    const int stage_bytes = tc::kABytes * p.mt + (p.n_pad / 2) * 128 * (p.use_lo ? 2 : 1);
    p.stages = std::max(2, std::min(8, (kTc2SmemMax - 1280) / stage_bytes));
    // K ranges: as many as keep all units in ONE wave of the SM pairs (one CTA fits per SM here, so a second wave
    // would pay set-up and epilogue again, back to back), at least four k-blocks each.
    const int slots = std::max(1, c->n_sm / 2);
    p.ksplit = 1;
    if (epi == tc::kEpiAtomic || epi == tc::kEpiScatterAtomic)
        p.ksplit = std::max(1, std::min(p.kblocks / 4, slots / std::max(tiles, 1)));
    int cols = 32;
    while (cols < p.n_pad) cols *= 2;
    p.acc_cols = cols;
    p.tmem_cols = std::max(32, cols * p.mt);
    p.act = act; p.act_hi = act_hi; p.act_lo = act_lo;
    p.Y = Y; p.ldy = ldy; p.idx = idx;
    p.flags = c->flags;
    p.stamp = stamp_slot(c, kClsGemmTc);
    p.m_dev = m_dev;
    p.row0 = r0;
    CUtensorMap tmBh, tmBl;
    if ((rc = make_map(&tmBh, Xh, mm, K, p.n_pad / 2, false))) return rc;
    if ((rc = make_map(&tmBl, Xl, mm, K, p.n_pad / 2, false))) return rc;
    const size_t smem = (size_t)p.stages * stage_bytes + 1024 + 8 * (2 * p.stages + 1) + 64;
    int e = epi;
    if (e == tc::kEpiAtomic) {
        if (p.ksplit == 1) e = tc::kEpiStore;
        else if (!pre_zeroed) {
            CU_TRY(cudaMemsetAsync(p.Y, 0, (size_t)mm * ldy * sizeof(float), st));
            c->pdl_next = false;
        }
    }
    auto kern = e == tc::kEpiStore ? tc2::gemm_tc2_kernel<tc::kEpiStore>
                : e == tc::kEpiAtomic ? tc2::gemm_tc2_kernel<tc::kEpiAtomic>
                : e == tc::kEpiSwiglu ? tc2::gemm_tc2_kernel<tc::kEpiSwiglu>
                                      : tc2::gemm_tc2_kernel<tc::kEpiScatterAtomic>;
    Launch guard(c, st, kClsGemmTc);
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(2 * tiles * p.ksplit);
    cfg.blockDim = dim3(320);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = (c->use_pdl && !c->profiling && c->pdl_next) ? 2 : 1;
    c->pdl_next = true;
    CU_TRY(cudaLaunchKernelEx(&cfg, kern, tmA, tmBh, tmBl, p));
    return FIRST_OK;
}

// Y (+)= X . W^T on the tensor cores.  Xh/Xl: [m][K] bf16 hi/lo activations (compact rows).
//   epi kEpiStore: Y[j*ldy+f] = ..;  kEpiAtomic: Y zeroed here, then reduced into;
//   kEpiScatterAtomic: Y[idx[j]*ldy+f] += ..
int launch_gemm_tc(first_ctx* c, cudaStream_t st, const CUtensorMap& tmA, const CUtensorMap& tmA2, int n_out, int K,
                   const __nv_bfloat16* Xh, const __nv_bfloat16* Xl, int m, int epi, float* Y, int64_t ldy,
                   const int32_t* idx, bool pre_zeroed, float* act = nullptr, __nv_bfloat16* act_hi = nullptr,
                   __nv_bfloat16* act_lo = nullptr, const int32_t* m_dev = nullptr) {
    int rc;
    for (int r0 = 0; r0 < m; r0 += 256) {
        const int mm = std::min(256, m - r0);
        if (tc2_wanted(c, mm, n_out, epi)) {  // many rows: a CTA pair per unit shares the activation tiles
            if ((rc = launch_gemm_tc2(c, st, epi == tc::kEpiSwiglu ? tmA2 : tmA, n_out, K, Xh + (size_t)r0 * K,
                                      Xl + (size_t)r0 * K, mm, r0, epi,
                                      Y ? Y + (epi == tc::kEpiScatterAtomic ? 0 : (size_t)r0 * ldy) : nullptr, ldy,
                                      idx ? idx + r0 : nullptr, pre_zeroed, act ? act + (size_t)r0 * n_out : nullptr,
                                      act_hi ? act_hi + (size_t)r0 * n_out : nullptr,
                                      act_lo ? act_lo + (size_t)r0 * n_out : nullptr, m_dev)))
                return rc;
            continue;
        }
        const TcShape t = tc_shape(c, n_out, K, mm, epi);
        tc::GemmParams p{};
        p.n_out = n_out; p.K = K; p.m = mm;
        p.n_pad = t.n_pad;
        p.kblocks = t.kblocks;
        p.use_lo = t.use_lo;
        p.mt = t.mt;
        p.pair_rows = c->pair_rows;
        const int tiles = t.tiles;
        p.act = act ? act + (size_t)r0 * n_out : nullptr;
        p.act_hi = act_hi ? act_hi + (size_t)r0 * n_out : nullptr;
        p.act_lo = act_lo ? act_lo + (size_t)r0 * n_out : nullptr;
        const int stage_bytes = t.stage_bytes;
        p.stages = t.stages;
        p.ksplit = t.ksplit;
        p.acc_cols = t.acc_cols;
        p.tmem_cols = t.tmem_cols;
        p.Y = Y ? Y + (epi == tc::kEpiScatterAtomic ? 0 : (size_t)r0 * ldy) : nullptr;
        p.ldy = ldy;
        p.idx = idx ? idx + r0 : nullptr;
        p.flags = c->flags;
        p.stamp = stamp_slot(c, kClsGemmTc);
        p.m_dev = m_dev;
        p.row0 = r0;
        CUtensorMap tmBh, tmBl;
        if ((rc = make_map(&tmBh, Xh + (size_t)r0 * K, mm, K, p.n_pad, false))) return rc;
        if ((rc = make_map(&tmBl, Xl + (size_t)r0 * K, mm, K, p.n_pad, false))) return rc;
        const size_t smem = (size_t)p.stages * stage_bytes + 1024 + 8 * (2 * p.stages + 1) + 64;
        int e = epi;
        if (e == tc::kEpiAtomic) {
            if (p.ksplit == 1) e = tc::kEpiStore;
            else if (!pre_zeroed) {
                CU_TRY(cudaMemsetAsync(p.Y, 0, (size_t)mm * ldy * sizeof(float), st));
                c->pdl_next = false;
            }
        }
        const int grid = tiles * p.ksplit;
        auto kern = e == tc::kEpiStore ? tc::gemm_tc_kernel<tc::kEpiStore>
                    : e == tc::kEpiAtomic ? tc::gemm_tc_kernel<tc::kEpiAtomic>
                    : e == tc::kEpiSwiglu ? tc::gemm_tc_kernel<tc::kEpiSwiglu>
                                          : tc::gemm_tc_kernel<tc::kEpiScatterAtomic>;
        if ((rc = launch_k(c, st, kClsGemmTc, kern, dim3(grid), dim3(320), smem, tmA, tmA2, tmBh, tmBl, p))) return rc;
    }
    return FIRST_OK;
}

int tc_setup(first_ctx* c) {
    const first_model_desc& d = c->d;
    int rc;
    const int L = d.n_layers;
    // Rows per half-tile of the fused gate/up projection: as large as 64, but small enough that the
    // tiles fill two CTA slots per SM in a single wave (8B shape on 148 SMs: 49 rows -> 293 tiles).
    c->pair_rows = 64;
    if (c->tune_pair_rows && d.ffn_dim > 64 * c->n_sm) {
        const int want = (d.ffn_dim + 2 * c->n_sm - 1) / (2 * c->n_sm);
        if (want <= 64) c->pair_rows = std::max(8, want);
    }
    c->tm_wqkv.resize(L); c->tm_wo.resize(L); c->tm_wgu.resize(L); c->tm_wgu64.resize(L); c->tm_wd.resize(L);
    for (int l = 0; l < L; ++l) {
        if ((rc = make_map(&c->tm_wqkv[l], c->wqkv[l], c->qkvd, d.d_model, tc::kBlockM, true)) ||
            (rc = make_map(&c->tm_wo[l], c->wo[l], d.d_model, c->qd, tc::kBlockM, true)) ||
            (rc = make_map(&c->tm_wgu[l], c->w_gate_up[l], 2 * (uint64_t)d.ffn_dim, d.d_model, tc::kBlockM, true)) ||
            (rc = make_map(&c->tm_wgu64[l], c->w_gate_up[l], 2 * (uint64_t)d.ffn_dim, d.d_model, c->pair_rows, true)) ||
            (rc = make_map(&c->tm_wd[l], c->w_down[l], d.d_model, d.ffn_dim, tc::kBlockM, true)))
            return rc;
    }
    if ((rc = make_map(&c->tm_lm, c->lm_head, d.vocab, d.d_model, tc::kBlockM, true))) return rc;
    CU_TRY(cudaFuncSetAttribute(tc::gemm_tc_kernel<tc::kEpiStore>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmemMax));
    CU_TRY(cudaFuncSetAttribute(tc::gemm_tc_kernel<tc::kEpiAtomic>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmemMax));
    CU_TRY(cudaFuncSetAttribute(tc::gemm_tc_kernel<tc::kEpiScatterAtomic>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmemMax));
    CU_TRY(cudaFuncSetAttribute(tc::gemm_tc_kernel<tc::kEpiSwiglu>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmemMax));
    CU_TRY(cudaFuncSetAttribute(tc2::gemm_tc2_kernel<tc::kEpiStore>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTc2SmemMax));
    CU_TRY(cudaFuncSetAttribute(tc2::gemm_tc2_kernel<tc::kEpiAtomic>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTc2SmemMax));
    CU_TRY(cudaFuncSetAttribute(tc2::gemm_tc2_kernel<tc::kEpiScatterAtomic>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTc2SmemMax));
    CU_TRY(cudaFuncSetAttribute(tc2::gemm_tc2_kernel<tc::kEpiSwiglu>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTc2SmemMax));
    c->tc_ready = true;
    return FIRST_OK;
}

template <typename WT, int EPI>
int launch_gemv(first_ctx* c, cudaStream_t st, const void* W, int n_out, int K, const float* X, int m, float* Y,
                int64_t ldy, const int32_t* idx, const int32_t* m_dev) {
    const int blocks = std::min((n_out + 7) / 8, c->n_sm * 8);
    for (int r0 = 0; r0 < m; r0 += 8) {
        const int rv = std::min(8, m - r0);
        const WT* w = static_cast<const WT*>(W);
        auto kern = rv == 1 ? gemv_rows<WT, 1, EPI> : rv == 2 ? gemv_rows<WT, 2, EPI>
                    : rv <= 4 ? gemv_rows<WT, 4, EPI> : gemv_rows<WT, 8, EPI>;
        int rc = launch_k(c, st, kClsGemv, kern, dim3(blocks), dim3(256), 0, w, n_out, K, X, r0, rv, m_dev, Y, ldy, idx);
        if (rc) return rc;
    }
    return FIRST_OK;
}

// One layer's view of the cache tables: shared by all layers, or (first_kv_cache::per_layer) this layer's
// rows of the [L][B] tables and its own tensor height.
struct LayerKv {
    const int64_t* slab_off;
    const int32_t* slab_cap;
    int64_t cap_total;
};
LayerKv layer_kv(const first_kv_cache* kv, int l, int B) {
    if (!kv->per_layer) return {kv->slab_off, kv->slab_cap, kv->cap_total};
    return {kv->slab_off + (size_t)l * B, kv->slab_cap + (size_t)l * B, kv->cap_total_l[l]};
}

template <typename KT, int HD>
int launch_attn_simple_g(first_ctx* c, cudaStream_t st, int S, int m, const KT* kc, const KT* vc,
                         const LayerKv* kv, const int32_t* len_l, const int32_t* idx, const int32_t* m_dev) {
    dim3 grid(S, c->d.n_kv_heads, m);
#define FIRST_ATTN_CASE(G)                                                                                  \
    case G:                                                                                                 \
        return launch_k(c, st, kClsAttn, attn_split_simple<KT, HD, G>, grid, dim3(128), 0, c->q, kc, vc,    \
                        kv->cap_total, kv->slab_off, len_l, kv->slab_cap, idx, m_dev, c->d.n_q_heads, c->o_part,   \
                        c->ml_part, c->d.max_tokens_per_seq);
    switch (c->group) {
        FIRST_ATTN_CASE(1)
        FIRST_ATTN_CASE(2)
        FIRST_ATTN_CASE(3)
        FIRST_ATTN_CASE(4)
        FIRST_ATTN_CASE(8)
        default: return FIRST_E_UNSUPPORTED;
    }
#undef FIRST_ATTN_CASE
    return check_launch(c);
}

template <typename KT>
int launch_attn_simple(first_ctx* c, cudaStream_t st, int S, int m, const void* kc, const void* vc,
                       const LayerKv* kv, const int32_t* len_l, const int32_t* idx, const int32_t* m_dev) {
    const KT *k = static_cast<const KT*>(kc), *v = static_cast<const KT*>(vc);
    switch (c->d.head_dim) {
        case 32: return launch_attn_simple_g<KT, 32>(c, st, S, m, k, v, kv, len_l, idx, m_dev);
        case 64: return launch_attn_simple_g<KT, 64>(c, st, S, m, k, v, kv, len_l, idx, m_dev);
        case 128: return launch_attn_simple_g<KT, 128>(c, st, S, m, k, v, kv, len_l, idx, m_dev);
        default: return FIRST_E_UNSUPPORTED;
    }
}

int kv_map_for(first_ctx* c, const void* ptr, int64_t cap_total, const CUtensorMap** out) {
    auto it = c->kv_maps.find(ptr);
    if (it == c->kv_maps.end() || it->second.cap_total != cap_total) {
        first_ctx::KvMap e{};
        e.cap_total = cap_total;
        int rc = make_map(&e.map, ptr, (uint64_t)c->d.n_kv_heads * (uint64_t)cap_total, c->d.head_dim, attn::kTile, false);
        if (rc) return rc;
        it = c->kv_maps.insert_or_assign(ptr, e).first;
    }
    *out = &it->second.map;
    return FIRST_OK;
}

template <int HD, int G, bool PAIR = false>
int launch_attn_mma_hg(first_ctx* c, cudaStream_t st, dim3 grid, const CUtensorMap& tk, const CUtensorMap& tv,
                       const LayerKv* kv, const void* kc, const void* vc, int C, float* out,
                       __nv_bfloat16* out_hi, __nv_bfloat16* out_lo, bool fuse_rope, float qscale,
                       const int32_t* m_dev) {
    constexpr int smem = attn::kStages * 2 * (HD / 64) * attn::kTile * 128 + 1024;
    attn::RopeFuse rf{};
    if (fuse_rope) {
        rf.qkv = c->qkv;
        rf.cs = c->cs;
        rf.qscale = qscale;
        rf.k_slab = static_cast<__nv_bfloat16*>(const_cast<void*>(kc));
        rf.v_slab = static_cast<__nv_bfloat16*>(const_cast<void*>(vc));
    }
    // Split rows: the chunks of a (row, kv head) form a thread-block cluster and merge through the first CTA's shared
    // memory when the cluster is small enough (at most 8 CTAs) and its partial results fit beside the ring without
    // costing the second CTA per SM.
    constexpr int GR = G;
    const int S = (int)grid.x;
    const int part_bytes = ((S - 1) * GR * (HD + 2) + GR * HD + 2 * GR) * 4;
    if (!PAIR && c->attn_cluster && S > 1 && S <= 8 && smem + part_bytes <= 113 * 1024) {
        if constexpr (!PAIR) {
            Launch guard(c, st, kClsAttn);
            cudaLaunchConfig_t cfg{};
            cfg.gridDim = grid;
            cfg.blockDim = dim3(160);
            cfg.dynamicSmemBytes = smem + part_bytes;
            cfg.stream = st;
            cudaLaunchAttribute at[2];
            at[0].id = cudaLaunchAttributeClusterDimension;
            at[0].val.clusterDim.x = S;
            at[0].val.clusterDim.y = 1;
            at[0].val.clusterDim.z = 1;
            at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            at[1].val.programmaticStreamSerializationAllowed = 1;
            cfg.attrs = at;
            cfg.numAttrs = (c->use_pdl && !c->profiling && c->pdl_next) ? 2 : 1;
            c->pdl_next = true;
            uint64_t* stamp = stamp_slot(c, kClsAttn);
            CU_TRY(cudaLaunchKernelEx(&cfg, attn::attn_split_mma<HD, G, false, true>, tk, tv, (const float*)c->q, kv->cap_total,
                                      (const longlong2*)c->rowinfo, m_dev, c->d.n_q_heads, C, c->o_part, c->ml_part, c->ticket,
                                      out, out_hi, out_lo, c->flags, rf, stamp));
            return FIRST_OK;
        }
    }
    return launch_k(c, st, kClsAttn, attn::attn_split_mma<HD, G, PAIR>, grid, dim3(160), smem, tk, tv, c->q, kv->cap_total,
                    c->rowinfo, m_dev, c->d.n_q_heads, C, c->o_part, c->ml_part, c->ticket, out,
                    out_hi, out_lo, c->flags, rf);
}

template <int HD, int G>
int attn_mma_set_attr() {
    constexpr int smem = attn::kStages * 2 * (HD / 64) * attn::kTile * 128 + 1024;
    CU_TRY(cudaFuncSetAttribute(attn::attn_split_mma<HD, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    CU_TRY(cudaFuncSetAttribute(attn::attn_split_mma<HD, G, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 113 * 1024));
    CU_TRY(cudaFuncSetAttribute(attn::attn_prefill_tc<HD, G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                attn::PrefillTc<HD, G>::kSmem));
    if constexpr (2 * G <= 8)  // the group form used on prompt chunks
        CU_TRY(cudaFuncSetAttribute(attn::attn_group_mma<HD, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    if constexpr (2 * G <= 8)  // the two-rows-per-work-item form used on prompt chunks
        CU_TRY(cudaFuncSetAttribute(attn::attn_split_mma<HD, G, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    return FIRST_OK;
}

// Opt the attention kernel of this model's (head_dim, group) into its shared-memory size (done once, at create).
int attn_mma_setup(first_ctx* c) {
#define FIRST_ATTN_MMA(HD, G) \
    if (c->d.head_dim == HD && c->group == G) return attn_mma_set_attr<HD, G>();
    FIRST_ATTN_MMA(128, 1) FIRST_ATTN_MMA(128, 2) FIRST_ATTN_MMA(128, 3) FIRST_ATTN_MMA(128, 4) FIRST_ATTN_MMA(128, 8)
    FIRST_ATTN_MMA(64, 1) FIRST_ATTN_MMA(64, 2) FIRST_ATTN_MMA(64, 3) FIRST_ATTN_MMA(64, 4) FIRST_ATTN_MMA(64, 8)
#undef FIRST_ATTN_MMA
    return FIRST_OK;
}

// Tuned attention for bfloat16 caches with head_dim 64/128; returns FIRST_E_UNSUPPORTED otherwise.
int launch_attn_mma(first_ctx* c, cudaStream_t st, int m, const void* kc, const void* vc, const LayerKv* kv,
                    const int32_t* len_l, const int32_t* idx, float* out, __nv_bfloat16* out_hi,
                    __nv_bfloat16* out_lo, bool fuse_rope, float qscale, int pair, const int32_t* m_dev) {
    const first_model_desc& d = c->d;
    if ((uint64_t)d.n_kv_heads * (uint64_t)kv->cap_total >= (1ull << 31)) return FIRST_E_UNSUPPORTED;
    int C = c->attn_chunk;
    if (C <= 0) {
        const double est = 0.6 * (double)m * d.n_kv_heads * d.max_tokens_per_seq;
        C = (int)(est / (4.0 * c->n_sm));
        C = std::max(1024, std::min(2048, C));
        // few rows: smaller chunks until there is at least one work item per SM
        while (C > 128 && est / C < c->n_sm) C /= 2;
        // many rows: whole rows already fill the CTA slots several times over, and an unsplit row needs no merge
        if (m * d.n_kv_heads >= 3 * c->n_sm && d.max_tokens_per_seq <= 2048) C = d.max_tokens_per_seq;
    }
    if (pair == 3 && c->attn_chunk <= 0) {
        // blocks of 128/G tokens: (m * G / 128) * Hkv work items per token chunk, one CTA per SM -- cut the token
        // axis so that the longest rows' items just about fill the SMs
        const double items = std::max(1.0, (double)m * c->group / 128.0) * d.n_kv_heads;
        C = std::max(256, (int)(d.max_tokens_per_seq * std::min(1.0, items / c->n_sm)));
    }
    if (pair == 3) C = std::max(C, (d.max_tokens_per_seq + 31) / 32);  // (its merge keeps 32 chunks' weights per row)
    C = std::max(C, (d.max_tokens_per_seq + c->max_splits - 1) / c->max_splits);
    C = (C + attn::kTile - 1) / attn::kTile * attn::kTile;
    const int S = (d.max_tokens_per_seq + C - 1) / C;
    const CUtensorMap *tk, *tv;
    int rc;
    if ((rc = kv_map_for(c, kc, kv->cap_total, &tk)) || (rc = kv_map_for(c, vc, kv->cap_total, &tv))) return rc;
    dim3 grid(S, d.n_kv_heads, m);
#define FIRST_ATTN_TC(HD, G)                                                                                     \
    if (pair == 3 && d.head_dim == HD && c->group == G) {                                                        \
        constexpr int TQ = attn::PrefillTc<HD, G>::TQ;                                                           \
        return launch_k(c, st, kClsAttn, attn::attn_prefill_tc<HD, G>, dim3(grid.y, (m + TQ - 1) / TQ + 1, grid.x), \
                        dim3(attn::kTcThreads), attn::PrefillTc<HD, G>::kSmem, *tk, *tv, c->q, kv->cap_total,    \
                        c->rowinfo, m, m_dev, d.n_q_heads, C, c->o_part, c->ml_part, c->ticket, out, out_hi,     \
                        out_lo, c->flags, (float)c->prefill_slack);                                              \
    }
    FIRST_ATTN_TC(128, 1) FIRST_ATTN_TC(128, 2) FIRST_ATTN_TC(128, 3) FIRST_ATTN_TC(128, 4) FIRST_ATTN_TC(128, 8)
    FIRST_ATTN_TC(64, 1) FIRST_ATTN_TC(64, 2) FIRST_ATTN_TC(64, 3) FIRST_ATTN_TC(64, 4) FIRST_ATTN_TC(64, 8)
#undef FIRST_ATTN_TC
#define FIRST_ATTN_GROUP(HD, G)                                                                                  \
    if (pair == 2 && d.head_dim == HD && c->group == G) {                                                        \
        constexpr int smem = attn::kStages * 2 * (HD / 64) * attn::kTile * 128 + 1024;                           \
        return launch_k(c, st, kClsAttn, attn::attn_group_mma<HD, G>, dim3(grid.x, grid.y, (m + 7) / 8),         \
                        dim3(160), smem, *tk, *tv, c->q, kv->cap_total, c->rowinfo, m, m_dev, d.n_q_heads, C,    \
                        c->o_part, c->ml_part, c->ticket, out, out_hi, out_lo, c->flags);                        \
    }
    FIRST_ATTN_GROUP(128, 1) FIRST_ATTN_GROUP(128, 2) FIRST_ATTN_GROUP(128, 3) FIRST_ATTN_GROUP(128, 4)
    FIRST_ATTN_GROUP(64, 1) FIRST_ATTN_GROUP(64, 2) FIRST_ATTN_GROUP(64, 3) FIRST_ATTN_GROUP(64, 4)
#undef FIRST_ATTN_GROUP
#define FIRST_ATTN_PAIR(HD, G)                            \
    if (pair && d.head_dim == HD && c->group == G)        \
        return launch_attn_mma_hg<HD, G, true>(c, st, grid, *tk, *tv, kv, kc, vc, C, out, out_hi, out_lo, false, qscale, m_dev);
    FIRST_ATTN_PAIR(128, 1) FIRST_ATTN_PAIR(128, 2) FIRST_ATTN_PAIR(128, 3) FIRST_ATTN_PAIR(128, 4)
    FIRST_ATTN_PAIR(64, 1) FIRST_ATTN_PAIR(64, 2) FIRST_ATTN_PAIR(64, 3) FIRST_ATTN_PAIR(64, 4)
#undef FIRST_ATTN_PAIR
#define FIRST_ATTN_MMA(HD, G)                 \
    if (d.head_dim == HD && c->group == G)    \
        return launch_attn_mma_hg<HD, G>(c, st, grid, *tk, *tv, kv, kc, vc, C, out, out_hi, out_lo, fuse_rope, qscale, m_dev);
    FIRST_ATTN_MMA(128, 1) FIRST_ATTN_MMA(128, 2) FIRST_ATTN_MMA(128, 3) FIRST_ATTN_MMA(128, 4) FIRST_ATTN_MMA(128, 8)
    FIRST_ATTN_MMA(64, 1) FIRST_ATTN_MMA(64, 2) FIRST_ATTN_MMA(64, 3) FIRST_ATTN_MMA(64, 4) FIRST_ATTN_MMA(64, 8)
#undef FIRST_ATTN_MMA
    return FIRST_E_UNSUPPORTED;
}

// One projection of m compact rows: tensor cores when the row count makes it a dense
// contraction (bf16 weights), the CUDA-core GEMV otherwise.
//   out_mode 0: Y[j][f] = ..   (compact rows, row stride ldy)
//   out_mode 1: Y[idx[j]][f] += ..   (scatter-add into the residual stream)
template <typename WT>
int project(first_ctx* c, cudaStream_t st, bool use_tc, const void* W, const CUtensorMap* tm, int n_out, int K,
            const float* X, const __nv_bfloat16* Xh, const __nv_bfloat16* Xl, int m, int out_mode, float* Y,
            int64_t ldy, const int32_t* idx, const int32_t* m_dev, bool allow_split = true, bool pre_zeroed = false) {
    if (use_tc) {
        const int epi = out_mode == 1 ? tc::kEpiScatterAtomic : (allow_split ? tc::kEpiAtomic : tc::kEpiStore);
        return launch_gemm_tc(c, st, *tm, *tm, n_out, K, Xh, Xl, m, epi, Y, ldy, idx, pre_zeroed, nullptr, nullptr,
                              nullptr, m_dev);
    }
    if (out_mode == 1) return launch_gemv<WT, kScatterAdd>(c, st, W, n_out, K, X, m, Y, ldy, idx, m_dev);
    return launch_gemv<WT, kStore>(c, st, W, n_out, K, X, m, Y, ldy, nullptr, m_dev);
}

template <typename WT>
int logits_tail(first_ctx* c, cudaStream_t st, int B, float* logits, int32_t* next_tokens, int32_t* pos);

// The whole step, for one weight/cache element type.
template <typename WT>
int decode_step_impl(first_ctx* c, const int32_t* tokens, const first_kv_cache* kv, float* logits,
                     int32_t* next_tokens, float* layer_inputs, cudaStream_t st, const PrefillHook* ph = nullptr) {
    const first_model_desc& d = c->d;
    const int B = c->B, D = d.d_model, F = d.ffn_dim, V = d.vocab, L = d.n_layers, hd = d.head_dim;
    constexpr bool kBf16 = std::is_same<WT, __nv_bfloat16>::value;
    const int gemv_max = c->max_gemv_rows >= 0 ? c->max_gemv_rows : 0;
    auto tc_for = [&](int m) { return kBf16 && c->tc_ready && m > gemv_max; };
    int rc;
    if (c->stamp_on && c->stamps) {  // fresh timing slots for this step: starts at the largest value, ends at zero
        c->stamp_n = 0;
        c->stamp_cls.clear();
        CU_TRY(cudaMemsetAsync(c->stamps, 0xff, sizeof(uint64_t) * kStampCap, st));
        CU_TRY(cudaMemsetAsync(c->stamps + kStampCap, 0, sizeof(uint64_t) * kStampCap, st));
    }
    c->pdl_next = false;  // the first kernel of a step has no predecessor to overlap
    if ((rc = launch_k(c, st, kClsStepBegin, step_begin<WT>, dim3(B), dim3(256), 0, tokens,
                       static_cast<const WT*>(c->embed), D, V, kv->pos, c->inv_freq, hd / 2, c->x, c->cs, c->flags)))
        return rc;

    int S = (d.max_tokens_per_seq + 255) / 256;
    S = std::max(1, std::min(S, kSimpleSplitsMax));
    const float qscale = 1.0f / std::sqrt((float)hd);
    const int norm_threads = std::max(32, std::min(c->norm_threads_max, (D / 4 + 31) / 32 * 32));  // at most norm_threads_max threads, a float4 or two each
    const bool mma_attn = kBf16 && c->tc_ready && (hd == 64 || hd == 128) && c->attn_simple <= 0;
    const bool fuse_rope = mma_attn && c->fuse_rope;
    // prompt chunks: consecutive rows are consecutive tokens of a sequence and may share attention work items
    const bool route_here = ph && ph->router_w;
    // (0 = each row its own work items, 1 = pairs of consecutive tokens, 2 = groups of up to eight)
    // (3 = blocks of 128/G tokens on the tcgen05 tensor cores)
    const bool tc_blocks = ph && mma_attn && !fuse_rope && c->prefill_tc && B <= attn::kTcMaxRows &&
                           (c->group == 1 || c->group == 2 || c->group == 3 || c->group == 4 || c->group == 8);
    const int pair_rows = tc_blocks ? 3
                          : (ph && mma_attn && !fuse_rope && 2 * c->group <= 8) ? (c->prefill_group ? 2 : c->prefill_pair ? 1 : 0) : 0;

    for (int l = 0; l < L; ++l) {
        if (layer_inputs) {
            CU_TRY(cudaMemcpyAsync(layer_inputs + (size_t)l * B * D, c->x, (size_t)B * D * sizeof(float),
                                   cudaMemcpyDeviceToDevice, st));
            c->pdl_next = false;
        }
        const int m = c->cnt_h[l];  // launch rows: the layer's active-row count, or an upper bound of it
        if (m == 0) continue;  // every sequence skips this layer: no launch at all
        const bool t = tc_for(m);
        const int32_t* idx = c->idx + (size_t)l * B;
        const int32_t* m_dev = c->cnt + l;  // the count itself, read by the kernels
        int32_t* len_l = kv->len + (size_t)l * B;
        const LayerKv lkv = layer_kv(kv, l, B);
        float* f32 = t ? nullptr : c->xn;
        __nv_bfloat16 *xh = t ? c->xh : nullptr, *xl = t ? c->xl : nullptr;
        // split-K projections reduce into float32 accumulators that the preceding norm kernel clears
        const bool zero_qkv = t;  // (cleared even when a projection ends up with one K range and plain stores)
        const bool fused_ffn = t && c->fuse_swiglu && (F % 64 == 0) && m <= 256;
        const bool zero_gu = t && !fused_ffn;
        // ---- attention half
        if ((rc = launch_k(c, st, kClsRmsnorm, rmsnorm_rows, dim3(m), dim3(norm_threads), 0, c->x, idx, m_dev, D, c->attn_norm[l],
                           d.rms_eps, f32, xh, xl, zero_qkv ? c->qkv : nullptr, c->qkvd, static_cast<int32_t*>(nullptr),
                           fuse_rope ? lkv.slab_cap : nullptr, fuse_rope ? c->rowinfo : nullptr,
                           fuse_rope ? static_cast<const int32_t*>(len_l) : nullptr, fuse_rope ? lkv.slab_off : nullptr,
                           c->flags,
                           // prompt chunks (all rows active, idx[i] = i): router l scores the rows it normalises
                           route_here ? ph->router_w + (size_t)l * D : nullptr,
                           route_here && ph->router_b ? ph->router_b + l : nullptr, route_here ? ph->mode : 0,
                           route_here ? ph->tokscore + (size_t)l * ph->stride + ph->g0 : nullptr, d.max_tokens_per_seq)))
            return rc;
        if ((rc = project<WT>(c, st, t, c->wqkv[l], t ? &c->tm_wqkv[l] : nullptr, c->qkvd, D, c->xn, c->xh, c->xl, m, 0,
                              c->qkv, c->qkvd, nullptr, m_dev, true, zero_qkv)))
            return rc;
        // The tuned attention kernel rotates q itself and appends the new token's key and value (its
        // row facts come from the norm kernel above); the general path has a kernel for that.
        if (!fuse_rope &&
            (rc = launch_k(c, st, kClsRopeAppend, rope_append<WT>, dim3((d.n_q_heads + 2 * d.n_kv_heads + 7) / 8, m), dim3(hd / 2, 8),
                           0, c->qkv, idx, m_dev, d.n_q_heads, d.n_kv_heads, hd, c->cs, qscale, c->q,
                           static_cast<WT*>(kv->k[l]), static_cast<WT*>(kv->v[l]), lkv.cap_total, lkv.slab_off,
                           lkv.slab_cap, len_l, c->flags, mma_attn ? c->rowinfo : nullptr, pair_rows,
                           d.max_tokens_per_seq)))
            return rc;
        if (mma_attn) {
            if ((rc = launch_attn_mma(c, st, m, kv->k[l], kv->v[l], &lkv, len_l, idx, t ? nullptr : c->att, xh, xl,
                                      fuse_rope, qscale, pair_rows, m_dev)))
                return rc;
        } else {
            if ((rc = launch_attn_simple<WT>(c, st, S, m, kv->k[l], kv->v[l], &lkv, len_l, idx, m_dev))) return rc;
            if ((rc = launch_k(c, st, kClsAttnCombine, attn_combine, dim3(m * d.n_q_heads), dim3(128), 0, c->o_part,
                               c->ml_part, m_dev, d.n_q_heads, S, hd, t ? nullptr : c->att, xh, xl)))
                return rc;
        }
        if ((rc = project<WT>(c, st, t, c->wo[l], t ? &c->tm_wo[l] : nullptr, D, c->qd, c->att, c->xh, c->xl, m, 1, c->x,
                              D, idx, m_dev)))
            return rc;
        // ---- feed-forward half (its norm kernel also advances the cache length of the rows it handles)
        if ((rc = launch_k(c, st, kClsRmsnorm, rmsnorm_rows, dim3(m), dim3(norm_threads), 0, c->x, idx, m_dev, D, c->ffn_norm[l],
                           d.rms_eps, f32, xh, xl, zero_gu ? c->gu : nullptr, 2 * F, len_l, lkv.slab_cap, static_cast<longlong2*>(nullptr), static_cast<const int32_t*>(nullptr), static_cast<const int64_t*>(nullptr), static_cast<uint32_t*>(nullptr),
                           static_cast<const float*>(nullptr), static_cast<const float*>(nullptr), 0, static_cast<float*>(nullptr), d.max_tokens_per_seq)))
            return rc;
        if (fused_ffn) {
            // gate/up projection with silu(gate)*up applied in its epilogue: the activation is written once
            if ((rc = launch_gemm_tc(c, st, c->tm_wgu64[l], c->tm_wgu[l], F, D, c->xh, c->xl, m, tc::kEpiSwiglu, nullptr, 0, nullptr,
                                     false, nullptr, c->acth, c->actl, m_dev)))
                return rc;
        } else {
            if ((rc = project<WT>(c, st, t, c->w_gate_up[l], t ? &c->tm_wgu[l] : nullptr, 2 * F, D, c->xn, c->xh, c->xl,
                                  m, 0, c->gu, 2 * F, nullptr, m_dev, true, zero_gu)))
                return rc;
            if ((rc = launch_k(c, st, kClsSiluMul, silu_mul, dim3(std::min((m * F + 255) / 256, c->n_sm * 8)),
                               dim3(256), 0, c->gu, m, m_dev, F, t ? nullptr : c->act, t ? c->acth : nullptr,
                               t ? c->actl : nullptr)))
                return rc;
        }
        if ((rc = project<WT>(c, st, t, c->w_down[l], t ? &c->tm_wd[l] : nullptr, D, F, c->act, c->acth, c->actl, m, 1,
                              c->x, D, idx, m_dev)))
            return rc;
    }
    if (ph) return FIRST_OK;  // a prefill chunk ends here: logits are taken once, from the last prompt tokens
    return logits_tail<WT>(c, st, B, logits, next_tokens, kv->pos);
}

// Final norm, lm_head and next token of rows 0..B-1 of the residual stream; pos += 1.
template <typename WT>
int logits_tail(first_ctx* c, cudaStream_t st, int B, float* logits, int32_t* next_tokens, int32_t* pos) {
    const first_model_desc& d = c->d;
    const int D = d.d_model, V = d.vocab;
    constexpr bool kBf16 = std::is_same<WT, __nv_bfloat16>::value;
    const int gemv_max = c->max_gemv_rows >= 0 ? c->max_gemv_rows : 0;
    auto tc_for = [&](int m) { return kBf16 && c->tc_ready && m > gemv_max; };
    const int norm_threads = std::max(32, std::min(c->norm_threads_max, (D / 4 + 31) / 32 * 32));
    int rc;
    float* lg = logits ? logits : (next_tokens ? c->logits_int : nullptr);
    if (lg) {
        const bool t = tc_for(B);
        if ((rc = launch_k(c, st, kClsRmsnorm, rmsnorm_rows, dim3(B), dim3(norm_threads), 0, c->x, nullptr, nullptr, D, c->final_norm,
                           d.rms_eps, t ? nullptr : c->xn, t ? c->xh : nullptr, t ? c->xl : nullptr, nullptr, 0, nullptr,
                           nullptr, static_cast<longlong2*>(nullptr), static_cast<const int32_t*>(nullptr), static_cast<const int64_t*>(nullptr), static_cast<uint32_t*>(nullptr),
                           static_cast<const float*>(nullptr), static_cast<const float*>(nullptr), 0, static_cast<float*>(nullptr), d.max_tokens_per_seq)))
            return rc;
        if ((rc = project<WT>(c, st, t, c->lm_head, t ? &c->tm_lm : nullptr, V, D, c->xn, c->xh, c->xl, B, 0, lg, V,
                              nullptr, nullptr, false)))
            return rc;
    }
    if (next_tokens && lg && c->sample_k > 1)
        return launch_k(c, st, kClsStepEnd, step_end_sample, dim3(B), dim3(1024), 0, lg, V, c->sample_k, c->sample_inv_T,
                        c->sample_u, next_tokens, pos);
    return launch_k(c, st, kClsStepEnd, step_end, dim3(B), dim3(1024), 0, lg, V, next_tokens, pos);
}

}  // namespace

extern "C" {

const char* first_status_string(int status) {
    switch (status) {
        case FIRST_OK: return "ok";
        case FIRST_E_ARG: return "bad argument";
        case FIRST_E_SHAPE: return "inconsistent shape";
        case FIRST_E_UNSUPPORTED: return "unsupported shape or dtype";
        case FIRST_E_CAPACITY: return "capacity exceeded";
        case FIRST_E_CUDA: return g_last_cuda_error[0] ? g_last_cuda_error : "CUDA error";
        case FIRST_E_DEVICE_FLAG: return "device flag set";
        case FIRST_E_STATE: return "call out of order";
        default: return "unknown status";
    }
}

int first_create(const first_model_desc* desc, const first_weights* w, first_ctx** out) {
    if (!desc || !w || !out) return FIRST_E_ARG;
    *out = nullptr;
    const first_model_desc& d = *desc;
    if (d.n_layers <= 0 || d.d_model <= 0 || d.n_q_heads <= 0 || d.n_kv_heads <= 0 || d.head_dim <= 0 ||
        d.ffn_dim <= 0 || d.vocab <= 0 || d.max_batch <= 0 || d.max_tokens_per_seq <= 0 || !(d.rope_base > 0.f) ||
        !(d.rms_eps >= 0.f))
        return FIRST_E_ARG;
    if (d.dtype != FIRST_DTYPE_F32 && d.dtype != FIRST_DTYPE_BF16) return FIRST_E_ARG;
    if (d.n_q_heads % d.n_kv_heads) return FIRST_E_SHAPE;
    const int group = d.n_q_heads / d.n_kv_heads;
    if (d.head_dim != 32 && d.head_dim != 64 && d.head_dim != 128) return FIRST_E_UNSUPPORTED;
    if (group != 1 && group != 2 && group != 3 && group != 4 && group != 8) return FIRST_E_UNSUPPORTED;
    if (d.d_model % 8 || d.ffn_dim % 8) return FIRST_E_UNSUPPORTED;
    if (!w->embed || !w->lm_head || !w->final_norm || !w->attn_norm || !w->wqkv || !w->wo || !w->ffn_norm ||
        !w->w_gate_up || !w->w_down)
        return FIRST_E_ARG;
    for (int l = 0; l < d.n_layers; ++l)
        if (!w->attn_norm[l] || !w->wqkv[l] || !w->wo[l] || !w->ffn_norm[l] || !w->w_gate_up[l] || !w->w_down[l])
            return FIRST_E_ARG;

    first_ctx* c = new (std::nothrow) first_ctx();
    if (!c) return FIRST_E_ARG;
    c->d = d;
    c->embed = w->embed;
    c->lm_head = w->lm_head;
    c->final_norm = w->final_norm;
    c->attn_norm.assign(w->attn_norm, w->attn_norm + d.n_layers);
    c->ffn_norm.assign(w->ffn_norm, w->ffn_norm + d.n_layers);
    c->wqkv.assign(w->wqkv, w->wqkv + d.n_layers);
    c->wo.assign(w->wo, w->wo + d.n_layers);
    c->w_gate_up.assign(w->w_gate_up, w->w_gate_up + d.n_layers);
    c->w_down.assign(w->w_down, w->w_down + d.n_layers);
    c->group = group;
    c->qd = d.n_q_heads * d.head_dim;
    c->kvd = d.n_kv_heads * d.head_dim;
    c->qkvd = c->qd + 2 * c->kvd;
    c->cnt_h.assign(d.n_layers, 0);

    int dev = 0, rc = FIRST_OK;
    auto fail = [&](int code) { first_destroy(c); return code; };
    if (cudaGetDevice(&dev) != cudaSuccess) return fail(FIRST_E_CUDA);
    cudaDeviceGetAttribute(&c->n_sm, cudaDevAttrMultiProcessorCount, dev);
    const size_t MB = d.max_batch;
    c->max_splits = std::max(kSimpleSplitsMax, std::min(64, (d.max_tokens_per_seq + 127) / 128));
    const int xw = std::max(d.d_model, c->qd);
    if ((rc = dev_alloc(&c->x, MB * d.d_model)) || (rc = dev_alloc(&c->xn, MB * xw)) ||
        (rc = dev_alloc(&c->qkv, MB * c->qkvd)) || (rc = dev_alloc(&c->q, MB * c->qd)) ||
        (rc = dev_alloc(&c->att, MB * c->qd)) || (rc = dev_alloc(&c->gu, MB * 2 * d.ffn_dim)) ||
        (rc = dev_alloc(&c->act, MB * d.ffn_dim)) ||
        (rc = dev_alloc(&c->o_part, MB * d.n_q_heads * c->max_splits * d.head_dim)) ||
        (rc = dev_alloc(&c->ml_part, MB * d.n_q_heads * c->max_splits)) ||
        (rc = dev_alloc(&c->cs, MB * (d.head_dim / 2))) || (rc = dev_alloc(&c->inv_freq, (size_t)d.head_dim / 2)) ||
        (rc = dev_alloc(&c->idx, MB * d.n_layers)) || (rc = dev_alloc(&c->cnt, (size_t)d.n_layers)) ||
        (rc = dev_alloc(&c->slot, MB * d.n_layers)) || (rc = dev_alloc(&c->flags, (size_t)1)) ||
        (rc = dev_alloc(&c->ticket, MB * d.n_kv_heads)) || (rc = dev_alloc(&c->rowinfo, MB)) ||
        (rc = dev_alloc(&c->mask_dev, MB * d.n_layers)))
        return fail(rc);
    if (cudaMemset(c->ticket, 0, MB * d.n_kv_heads * sizeof(uint32_t)) != cudaSuccess) return fail(FIRST_E_CUDA);
    if ((rc = dev_alloc(&c->pf_cu, MB + 1)) || (rc = dev_alloc(&c->pf_tok, MB)) || (rc = dev_alloc(&c->pf_cap, MB)) ||
        (rc = dev_alloc(&c->pf_pos, MB)) || (rc = dev_alloc(&c->pf_len, MB * d.n_layers)) ||
        (rc = dev_alloc(&c->pf_off, MB)) || (rc = dev_alloc(&c->pf_ones, MB * d.n_layers)) ||
        (rc = dev_alloc(&c->x_last, MB * d.d_model)))
        return fail(rc);
    if (cudaMemset(c->pf_ones, 1, MB * d.n_layers) != cudaSuccess) return fail(FIRST_E_CUDA);
    if (d.dtype == FIRST_DTYPE_BF16) {
        if ((rc = dev_alloc(&c->xh, MB * xw)) || (rc = dev_alloc(&c->xl, MB * xw)) ||
            (rc = dev_alloc(&c->acth, MB * d.ffn_dim)) || (rc = dev_alloc(&c->actl, MB * d.ffn_dim)))
            return fail(rc);
        if ((rc = tc_setup(c)) || (rc = attn_mma_setup(c))) return fail(rc);
    }
    if (cudaStreamCreateWithFlags(&c->cap_stream, cudaStreamNonBlocking) != cudaSuccess) return fail(FIRST_E_CUDA);
    c->tok_cap = (int64_t)d.max_batch * d.max_tokens_per_seq;
    if ((rc = dev_alloc(&c->tokscore, (size_t)c->tok_cap))) return fail(rc);
    std::vector<double> inv(d.head_dim / 2);
    for (int i = 0; i < d.head_dim / 2; ++i) inv[i] = std::pow((double)d.rope_base, -2.0 * i / (double)d.head_dim);
    if (cudaMemcpy(c->inv_freq, inv.data(), inv.size() * sizeof(double), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemset(c->flags, 0, sizeof(uint32_t)) != cudaSuccess)
        return fail(FIRST_E_CUDA);
    *out = c;
    return FIRST_OK;
}

int first_destroy(first_ctx* c) {
    if (!c) return FIRST_OK;
    void* ptrs[] = {c->x, c->xn, c->qkv, c->q, c->att, c->gu, c->act, c->o_part, c->logits_int, c->tokscore,
                    c->ml_part, c->cs, c->inv_freq, c->idx, c->cnt, c->slot, c->flags, c->xh, c->xl, c->acth, c->actl, c->ticket, c->rowinfo,
                    c->pf_cu, c->pf_tok, c->pf_cap, c->pf_pos, c->pf_len, c->pf_off, c->pf_ones, c->x_last, c->pf_score,
                    c->stamps, c->mask_dev};
    for (void* p : ptrs)
        if (p) cudaFree(p);
    for (cudaEvent_t e : c->ev_pool) cudaEventDestroy(e);
    for (auto& e : c->graphs) cudaGraphExecDestroy(e.exec);
    if (c->cap_stream) cudaStreamDestroy(c->cap_stream);
    delete c;
    return FIRST_OK;
}

int first_prefill_route(first_ctx* c, int32_t layer, const void* hidden, int32_t hidden_dtype,
                        const int32_t* cu_seqlens, int32_t B, int64_t total_tokens, const float* router_w,
                        const float* router_b, float tau, int32_t mode, uint8_t* mask, float* scores, void* stream) {
    if (!c || !hidden || !cu_seqlens || !router_w || !mask) return FIRST_E_ARG;
    if (layer < 0 || layer >= c->d.n_layers || B <= 0 || total_tokens <= 0) return FIRST_E_ARG;
    if (hidden_dtype != FIRST_DTYPE_F32 && hidden_dtype != FIRST_DTYPE_BF16) return FIRST_E_ARG;
    if (mode != FIRST_ROUTER_MEAN_OF_SIGMOID && mode != FIRST_ROUTER_SIGMOID_OF_MEAN) return FIRST_E_ARG;
    if (!(tau > 0.f && tau < 1.f)) return FIRST_E_ARG;
    if (total_tokens > c->tok_cap || total_tokens > 0x7fffffffLL) return FIRST_E_CAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int D = c->d.d_model;
    if (D > 12288) return FIRST_E_UNSUPPORTED;  // the router vector is staged in 48 KB of shared memory
    const int64_t want = (total_tokens + 7) / 8;
    const int blocks = (int)std::min<int64_t>(want, (int64_t)c->n_sm * 8);
    const size_t smem = (size_t)D * sizeof(float);
    if (hidden_dtype == FIRST_DTYPE_BF16)
        FIRST_LAUNCH(kClsRouterScores, (router_token_scores<__nv_bfloat16><<<blocks, 256, smem, st>>>(static_cast<const __nv_bfloat16*>(hidden),
                                                                      total_tokens, D, router_w, router_b, mode,
                                                                      c->tokscore)));
    else
        FIRST_LAUNCH(kClsRouterScores, (router_token_scores<float><<<blocks, 256, smem, st>>>(static_cast<const float*>(hidden), total_tokens, D,
                                                              router_w, router_b, mode, c->tokscore)));
    int rc = check_launch(c);
    if (rc) return rc;
    FIRST_LAUNCH(kClsRouterFinalize, (router_finalize<<<B, 256, 0, st>>>(c->tokscore, cu_seqlens, total_tokens, c->d.n_layers, layer, mode, tau, mask, scores,
                                       c->flags)));
    return check_launch(c);
}

int first_set_mask(first_ctx* c, const uint8_t* mask, int32_t B, void* stream) {
    if (!c || !mask || B <= 0) return FIRST_E_ARG;
    if (B > c->d.max_batch) return FIRST_E_CAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    c->has_mask = false;
    FIRST_LAUNCH(kClsPlan, (plan_compact<<<c->d.n_layers, 32, 0, st>>>(mask, B, c->d.n_layers, c->idx, c->cnt, c->slot, c->flags)));
    int rc = check_launch(c);
    if (rc) return rc;
    uint32_t fl = 0;
    CU_TRY(cudaMemcpyAsync(c->cnt_h.data(), c->cnt, sizeof(int32_t) * c->d.n_layers, cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaMemcpyAsync(&fl, c->flags, sizeof fl, cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaStreamSynchronize(st));
    if (fl & FIRST_FLAG_BAD_MASK) return FIRST_E_DEVICE_FLAG;
    c->B = B;
    c->has_mask = true;  // launch rows = the exact counts; recorded step graphs are looked up by them
    return FIRST_OK;
}

int first_set_mask_host(first_ctx* c, const uint8_t* mask, int32_t B, void* stream) {
    if (!c || !mask || B <= 0) return FIRST_E_ARG;
    if (B > c->d.max_batch) return FIRST_E_CAPACITY;
    const int L = c->d.n_layers;
    std::vector<int32_t> cnt(L, 0);
    for (int b = 0; b < B; ++b)
        for (int l = 0; l < L; ++l) {
            const uint8_t mk = mask[(size_t)b * L + l];
            if (mk > 1) return FIRST_E_ARG;
            cnt[l] += mk;
        }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    CU_TRY(cudaStreamIsCapturing(st, &cap));
    if (cap != cudaStreamCaptureStatusNone) return FIRST_E_STATE;
    c->has_mask = false;
    // pageable source: the runtime takes its own copy before returning, and does not wait for the stream
    CU_TRY(cudaMemcpyAsync(c->mask_dev, mask, (size_t)B * L, cudaMemcpyHostToDevice, st));
    FIRST_LAUNCH(kClsPlan, (plan_compact<<<L, 32, 0, st>>>(c->mask_dev, B, L, c->idx, c->cnt, c->slot, c->flags)));
    int rc = check_launch(c);
    if (rc) return rc;
    // Launch rows: the count rounded up to the next multiple of 16 (the projections pad to that anyway).  The
    // kernels read the exact count from device memory, so a batch change that keeps every layer inside its
    // bucket finds its recorded step graph again.
    for (int l = 0; l < L; ++l) c->cnt_h[l] = cnt[l] == 0 ? 0 : std::min<int>(B, (cnt[l] + 15) / 16 * 16);
    c->B = B;
    c->has_mask = true;
    return FIRST_OK;
}

int first_get_plan(first_ctx* c, int32_t* idx, int32_t* cnt, int32_t* slot) {
    if (!c || !idx || !cnt) return FIRST_E_ARG;
    if (!c->has_mask) return FIRST_E_STATE;
    const size_t n = (size_t)c->d.n_layers * c->B;
    CU_TRY(cudaMemcpy(idx, c->idx, n * sizeof(int32_t), cudaMemcpyDeviceToHost));
    CU_TRY(cudaMemcpy(cnt, c->cnt, (size_t)c->d.n_layers * sizeof(int32_t), cudaMemcpyDeviceToHost));
    if (slot) CU_TRY(cudaMemcpy(slot, c->slot, n * sizeof(int32_t), cudaMemcpyDeviceToHost));
    return FIRST_OK;
}

int first_decode_step(first_ctx* c, const int32_t* tokens, const first_kv_cache* kv, float* logits,
                      int32_t* next_tokens, float* layer_inputs, void* stream) {
    if (!c || !tokens || !kv) return FIRST_E_ARG;
    if (!c->has_mask) return FIRST_E_STATE;
    if (!kv->k || !kv->v || !kv->slab_off || !kv->slab_cap || !kv->len || !kv->pos) return FIRST_E_ARG;
    if (kv->per_layer ? !kv->cap_total_l : kv->cap_total <= 0) return FIRST_E_ARG;
    for (int l = 0; l < c->d.n_layers; ++l) {
        if (c->cnt_h[l] == 0) continue;
        if (!kv->k[l] || !kv->v[l]) return FIRST_E_ARG;
        if (kv->per_layer && kv->cap_total_l[l] <= 0) return FIRST_E_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    auto run = [&](cudaStream_t s) {
        if (c->d.dtype == FIRST_DTYPE_BF16)
            return decode_step_impl<__nv_bfloat16>(c, tokens, kv, logits, next_tokens, layer_inputs, s);
        return decode_step_impl<float>(c, tokens, kv, logits, next_tokens, layer_inputs, s);
    };
    if (!logits && next_tokens && !c->logits_int) {  // allocate outside any capture
        int rc = dev_alloc(&c->logits_int, (size_t)c->d.max_batch * c->d.vocab);
        if (rc) return rc;
    }
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    CU_TRY(cudaStreamIsCapturing(st, &cap));
    if (!c->use_graph || c->profiling || cap != cudaStreamCaptureStatusNone) return run(st);

    // The launch sequence of a step depends only on the plan and on the pointers: replay it as one graph.
    std::vector<const void*> key;
    key.reserve(12 + 2 * c->d.n_layers);
    key.push_back(tokens); key.push_back(logits); key.push_back(next_tokens); key.push_back(layer_inputs);
    key.push_back(kv->slab_off); key.push_back(kv->slab_cap); key.push_back(kv->len); key.push_back(kv->pos);
    key.push_back(reinterpret_cast<const void*>(static_cast<uintptr_t>(kv->cap_total)));
    key.push_back(reinterpret_cast<const void*>(static_cast<uintptr_t>(kv->per_layer)));
    if (kv->per_layer)
        for (int l = 0; l < c->d.n_layers; ++l)
            key.push_back(reinterpret_cast<const void*>(static_cast<uintptr_t>(kv->cap_total_l[l])));
    key.push_back(reinterpret_cast<const void*>(static_cast<uintptr_t>(c->plan_version)));  // options, sampling
    key.push_back(reinterpret_cast<const void*>(static_cast<uintptr_t>(c->B)));
    for (int l = 0; l < c->d.n_layers; ++l)  // the launch sequence is a function of the rows launched per layer
        key.push_back(reinterpret_cast<const void*>(static_cast<uintptr_t>(c->cnt_h[l])));
    for (int l = 0; l < c->d.n_layers; ++l) { key.push_back(kv->k[l]); key.push_back(kv->v[l]); }
    first_ctx::StepGraph* g = nullptr;
    for (auto& e : c->graphs)
        if (e.key == key) { g = &e; break; }
    if (!g) {
        if (c->graphs.size() >= 16) {  // drop the least recently used
            size_t lru = 0;
            for (size_t i = 1; i < c->graphs.size(); ++i)
                if (c->graphs[i].last_use < c->graphs[lru].last_use) lru = i;
            cudaGraphExecDestroy(c->graphs[lru].exec);
            c->graphs.erase(c->graphs.begin() + lru);
        }
        const int64_t l0 = c->launches;
        CU_TRY(cudaStreamBeginCapture(c->cap_stream, cudaStreamCaptureModeThreadLocal));
        const int rc = run(c->cap_stream);
        cudaGraph_t graph = nullptr;
        const cudaError_t e = cudaStreamEndCapture(c->cap_stream, &graph);
        if (rc) {
            if (graph) cudaGraphDestroy(graph);
            return rc;
        }
        CU_TRY(e);
        first_ctx::StepGraph sg;
        sg.key = key;
        sg.n_launches = c->launches - l0;
        c->launches = l0;
        const cudaError_t e2 = cudaGraphInstantiate(&sg.exec, graph, 0);
        cudaGraphDestroy(graph);
        CU_TRY(e2);
        c->graphs.push_back(std::move(sg));
        g = &c->graphs.back();
    }
    g->last_use = ++c->use_clock;
    CU_TRY(cudaGraphLaunch(g->exec, st));
    c->launches += g->n_launches;
    return FIRST_OK;
}

int first_prefill(first_ctx* c, const int32_t* tokens, const int32_t* cu_seqlens, int32_t B, const first_kv_cache* kv,
                  const float* router_w, const float* router_b, float tau, int32_t mode, uint8_t* mask, float* scores,
                  float* logits, int32_t* next_tokens, void* stream) {
    if (!c || !tokens || !cu_seqlens || !kv || B <= 0) return FIRST_E_ARG;
    if (!kv->k || !kv->v || !kv->slab_off || !kv->slab_cap || !kv->len || !kv->pos) return FIRST_E_ARG;
    if (kv->per_layer) return FIRST_E_UNSUPPORTED;  // the prompt fills every layer: one table serves them all
    if (kv->cap_total <= 0) return FIRST_E_ARG;
    const first_model_desc& d = c->d;
    const int L = d.n_layers, D = d.d_model;
    for (int l = 0; l < L; ++l)
        if (!kv->k[l] || !kv->v[l]) return FIRST_E_ARG;
    if (router_w) {
        if (!mask) return FIRST_E_ARG;
        if (mode != FIRST_ROUTER_MEAN_OF_SIGMOID && mode != FIRST_ROUTER_SIGMOID_OF_MEAN) return FIRST_E_ARG;
        if (!(tau > 0.f && tau < 1.f)) return FIRST_E_ARG;
        if (D > 12288) return FIRST_E_UNSUPPORTED;
    }
    if (B > d.max_batch) return FIRST_E_CAPACITY;
    if (cu_seqlens[0] != 0) return FIRST_E_ARG;
    for (int b = 0; b < B; ++b) {
        const int64_t n = (int64_t)cu_seqlens[b + 1] - cu_seqlens[b];
        if (n <= 0) return FIRST_E_ARG;  // every sequence brings at least one prompt token
        if (n > d.max_tokens_per_seq) return FIRST_E_CAPACITY;
    }
    const int64_t total = cu_seqlens[B];
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    CU_TRY(cudaStreamIsCapturing(st, &cap));
    if (cap != cudaStreamCaptureStatusNone) return FIRST_E_STATE;  // this call waits for the stream
    if (router_w && (int64_t)L * total > c->pf_score_cap) {
        if (c->pf_score) cudaFree(c->pf_score);
        c->pf_score = nullptr;
        c->pf_score_cap = 0;
        int rc = dev_alloc(&c->pf_score, (size_t)L * total);
        if (rc) return rc;
        c->pf_score_cap = (int64_t)L * total;
    }
    if (!logits && next_tokens && !c->logits_int) {
        int rc = dev_alloc(&c->logits_int, (size_t)d.max_batch * d.vocab);
        if (rc) return rc;
    }
    CU_TRY(cudaMemcpyAsync(c->pf_cu, cu_seqlens, sizeof(int32_t) * (B + 1), cudaMemcpyHostToDevice, st));

    // Each prompt token is a row of its own for the step kernels, so the rotate-and-append kernel must finish
    // a chunk's keys and values before attention starts (a row attends over earlier rows of its own chunk).
    struct Restore {
        first_ctx* c; int fuse_rope;
        ~Restore() { c->fuse_rope = fuse_rope; c->has_mask = false; }
    } restore{c, c->fuse_rope};
    c->fuse_rope = 0;

    first_kv_cache vkv = *kv;
    vkv.slab_off = c->pf_off;
    vkv.slab_cap = c->pf_cap;
    vkv.len = c->pf_len;
    vkv.pos = c->pf_pos;
    // Rows per chunk: as many as one projection launch takes (measured on 34.8 k prompt tokens at the 8B shape:
    // 128 rows 1.66 s, 144 1.59 s, 160 1.52 s, 256 1.34 s: fewer passes over the weights win).
    const int chunk = std::max(1, std::min(c->prefill_rows > 0 ? c->prefill_rows : 256, 256));
    const int R = (int)std::min<int64_t>(std::min(d.max_batch, chunk), total);
    int plan_rows = 0, rc;
    for (int64_t g0 = 0; g0 < total; g0 += R) {
        const int rows = (int)std::min<int64_t>(R, total - g0);
        if (rows != plan_rows) {  // all-keep plan over this many rows (at most twice per call)
            if ((rc = first_set_mask(c, c->pf_ones, rows, stream))) return rc;
            plan_rows = rows;
        }
        FIRST_LAUNCH(kClsPrefillAux, (prefill_rows<<<(rows + 127) / 128, 128, 0, st>>>(
                                         tokens, c->pf_cu, B, (int)g0, rows, L, kv->slab_off, kv->slab_cap, c->pf_tok,
                                         c->pf_off, c->pf_cap, c->pf_pos, c->pf_len)));
        if ((rc = check_launch(c))) return rc;
        const PrefillHook ph{router_w, router_b, mode, c->pf_score, total, g0};
        const int lo_rows_saved = c->tc_lo_max_rows;
        if (!c->prefill_lo) c->tc_lo_max_rows = 0;
        rc = d.dtype == FIRST_DTYPE_BF16
                 ? decode_step_impl<__nv_bfloat16>(c, c->pf_tok, &vkv, nullptr, nullptr, nullptr, st, &ph)
                 : decode_step_impl<float>(c, c->pf_tok, &vkv, nullptr, nullptr, nullptr, st, &ph);
        c->tc_lo_max_rows = lo_rows_saved;
        if (rc) return rc;
        FIRST_LAUNCH(kClsPrefillAux, (prefill_keep_last<<<rows, 256, 0, st>>>(c->x, c->pf_cu, B, (int)g0, D, c->x_last)));
        if ((rc = check_launch(c))) return rc;
    }
    if (router_w)
        for (int l = 0; l < L; ++l) {
            FIRST_LAUNCH(kClsRouterFinalize, (router_finalize<<<B, 256, 0, st>>>(c->pf_score + (size_t)l * total, c->pf_cu, total, L, l,
                                                                                 mode, tau, mask, scores, c->flags)));
            if ((rc = check_launch(c))) return rc;
        }
    FIRST_LAUNCH(kClsPrefillAux, (prefill_finish<<<(B + 127) / 128, 128, 0, st>>>(c->pf_cu, B, L, kv->slab_cap, kv->len, kv->pos)));
    if ((rc = check_launch(c))) return rc;
    if (logits || next_tokens) {
        CU_TRY(cudaMemcpyAsync(c->x, c->x_last, (size_t)B * D * sizeof(float), cudaMemcpyDeviceToDevice, st));
        c->pdl_next = false;
        // the tail advances a position counter: hand it the chunk table, pos[] already holds the prompt lengths
        rc = d.dtype == FIRST_DTYPE_BF16 ? logits_tail<__nv_bfloat16>(c, st, B, logits, next_tokens, c->pf_pos)
                                         : logits_tail<float>(c, st, B, logits, next_tokens, c->pf_pos);
        if (rc) return rc;
    }
    CU_TRY(cudaStreamSynchronize(st));  // cu_seqlens was read from host memory; the plan of the last chunk is dropped
    return FIRST_OK;
}

int first_last_device_flags(first_ctx* c, uint32_t* flags, void* stream) {
    if (!c || !flags) return FIRST_E_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CU_TRY(cudaMemcpyAsync(flags, c->flags, sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaMemsetAsync(c->flags, 0, sizeof(uint32_t), st));
    CU_TRY(cudaStreamSynchronize(st));
    if (*flags & FIRST_FLAG_WAIT_EXPIRED) {
        // A kernel gave up on a wait: the step's outputs are undefined, and an attention work item that left
        // early took no merge ticket.  Put the ticket counters back to zero so that later steps merge correctly.
        CU_TRY(cudaMemsetAsync(c->ticket, 0, (size_t)c->d.max_batch * c->d.n_kv_heads * sizeof(uint32_t), st));
        CU_TRY(cudaStreamSynchronize(st));
    }
    return *flags ? FIRST_E_DEVICE_FLAG : FIRST_OK;
}

int first_selftest_wait_expiry(first_ctx* c, int32_t polls, int32_t* returned, int32_t* abort_word, void* stream) {
    if (!c || polls <= 0 || polls > (1 << 20) || !returned || !abort_word) return FIRST_E_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t* out = reinterpret_cast<int32_t*>(c->rowinfo);  // 16 bytes of scratch nothing else uses between steps
    tc::wait_expiry_selftest<<<1, 32, 0, st>>>((uint32_t)polls, c->flags, out);
    CU_TRY(cudaGetLastError());
    int32_t h[2] = {-1, -1};
    CU_TRY(cudaMemcpyAsync(h, out, sizeof h, cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaStreamSynchronize(st));
    *returned = h[0];
    *abort_word = h[1];
    return FIRST_OK;
}

int64_t first_launch_count(const first_ctx* c) { return c ? c->launches : 0; }

int first_get_desc(const first_ctx* c, first_model_desc* out) {
    if (!c || !out) return FIRST_E_ARG;
    *out = c->d;
    return FIRST_OK;
}

int64_t first_graph_count(const first_ctx* c) { return c ? (int64_t)c->graphs.size() : 0; }

int first_profile(first_ctx* c, int32_t enable) {
    if (!c) return FIRST_E_ARG;
    c->profiling = enable != 0;
    c->ev_cls.clear();
    for (int k = 0; k < kNumClasses; ++k) { c->prof_ms[k] = 0.0; c->prof_launches[k] = 0; }
    return FIRST_OK;
}

int first_profile_read(first_ctx* c, int32_t n, double* ms, int64_t* launches, void* stream) {
    if (!c || !ms || !launches || n < kNumClasses) return FIRST_E_ARG;
    CU_TRY(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    for (size_t i = 0; i < c->ev_cls.size(); ++i) {
        float t = 0.f;
        CU_TRY(cudaEventElapsedTime(&t, c->ev_pool[2 * i], c->ev_pool[2 * i + 1]));
        c->prof_ms[c->ev_cls[i]] += t;
        c->prof_launches[c->ev_cls[i]] += 1;
    }
    c->ev_cls.clear();
    for (int k = 0; k < n; ++k) {
        ms[k] = k < kNumClasses ? c->prof_ms[k] : 0.0;
        launches[k] = k < kNumClasses ? c->prof_launches[k] : 0;
    }
    return FIRST_OK;
}

int first_set_sampling(first_ctx* c, int32_t top_k, float temperature, const float* uniforms) {
    if (!c || top_k < 0 || !(temperature >= 0.f)) return FIRST_E_ARG;
    if (top_k > FIRST_SAMPLE_TOPK_MAX) return FIRST_E_UNSUPPORTED;
    if (top_k > c->d.vocab) return FIRST_E_ARG;
    const bool greedy = top_k <= 1 || temperature == 0.f;
    if (!greedy && !uniforms) return FIRST_E_ARG;
    c->sample_k = greedy ? 0 : top_k;
    c->sample_inv_T = greedy ? 1.f : 1.f / temperature;
    c->sample_u = greedy ? nullptr : uniforms;
    c->plan_version += 1;  // cached step graphs end in the previous choice of kernel and pointer
    return FIRST_OK;
}

int first_sample_topk(const float* logits, int32_t B, int32_t vocab, int32_t top_k, float temperature,
                      const float* uniforms, int32_t* tokens, void* stream) {
    if (!logits || !uniforms || !tokens || B <= 0 || vocab <= 0 || top_k <= 0 || top_k > vocab || !(temperature >= 0.f))
        return FIRST_E_ARG;
    if (top_k > FIRST_SAMPLE_TOPK_MAX) return FIRST_E_UNSUPPORTED;
    const bool greedy = top_k == 1 || temperature == 0.f;
    step_end_sample<<<B, 1024, 0, static_cast<cudaStream_t>(stream)>>>(logits, vocab, greedy ? 1 : top_k,
                                                                        greedy ? 1.f : 1.f / temperature, uniforms, tokens,
                                                                        nullptr, nullptr);
    return cudaGetLastError() == cudaSuccess ? FIRST_OK : FIRST_E_CUDA;
}

int first_step_trace(first_ctx* c, int32_t max_n, int32_t* cls, uint64_t* t_start, uint64_t* t_end, int32_t* n_out,
                     void* stream) {
    if (!c || !cls || !t_start || !t_end || !n_out || max_n < 0) return FIRST_E_ARG;
    *n_out = 0;
    if (!c->stamp_on || !c->stamps) return FIRST_E_STATE;
    const int n = std::min<int>(c->stamp_n, max_n);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CU_TRY(cudaMemcpyAsync(t_start, c->stamps, sizeof(uint64_t) * n, cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaMemcpyAsync(t_end, c->stamps + kStampCap, sizeof(uint64_t) * n, cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaStreamSynchronize(st));
    for (int i = 0; i < n; ++i) cls[i] = c->stamp_cls[i];
    *n_out = n;
    return FIRST_OK;
}

int32_t first_kernel_class_count(void) { return kNumClasses; }
const char* first_kernel_class_name(int32_t k) { return (k >= 0 && k < kNumClasses) ? kClassNames[k] : ""; }

int first_set_option(first_ctx* c, const char* name, int64_t value) {
    if (!c || !name) return FIRST_E_ARG;
    if (!std::strcmp(name, "max_gemv_rows")) c->max_gemv_rows = (int)value;
    else if (!std::strcmp(name, "attn_simple")) c->attn_simple = (int)value;
    else if (!std::strcmp(name, "tc_use_lo")) c->tc_use_lo = value != 0;
    else if (!std::strcmp(name, "attn_chunk")) c->attn_chunk = (int)value;
    else if (!std::strcmp(name, "use_graph")) c->use_graph = value != 0;
    else if (!std::strcmp(name, "use_pdl")) c->use_pdl = value != 0;
    else if (!std::strcmp(name, "fuse_swiglu")) c->fuse_swiglu = value != 0;
    else if (!std::strcmp(name, "fuse_rope")) c->fuse_rope = value != 0;
    else if (!std::strcmp(name, "prefill_pair")) c->prefill_pair = value != 0;
    else if (!std::strcmp(name, "prefill_group")) c->prefill_group = value != 0;
    else if (!std::strcmp(name, "prefill_tc")) c->prefill_tc = value != 0;
    else if (!std::strcmp(name, "prefill_lo")) c->prefill_lo = value != 0;
    else if (!std::strcmp(name, "prefill_slack")) c->prefill_slack = (int)std::max<int64_t>(0, std::min<int64_t>(value, 16));
    else if (!std::strcmp(name, "prefill_rows")) c->prefill_rows = value > 0 ? (int)value : 0;
    else if (!std::strcmp(name, "tc_lo_max_rows")) c->tc_lo_max_rows = value >= 0 ? (int)value : (1 << 30);
    else if (!std::strcmp(name, "tc_mt2_min_rows")) c->tc_mt2_min_rows = value > 0 ? (int)value : -1;
    else if (!std::strcmp(name, "tc_ksplit_cap")) c->tc_ksplit_cap = value != 0;
    else if (!std::strcmp(name, "tc_smem_kb")) c->tc_smem_kb = value > 0 ? (int)value : 110;
    else if (!std::strcmp(name, "tc2_min_rows")) c->tc2_min_rows = value < 0 ? 96 : (int)value;
    else if (!std::strcmp(name, "tc2_mt2_all")) c->tc2_mt2_all = value > 0;
    else if (!std::strcmp(name, "attn_cluster")) c->attn_cluster = value > 0;
    else if (!std::strcmp(name, "norm_threads")) c->norm_threads_max = value >= 32 ? std::min<int>(1024, (int)value / 32 * 32) : 512;
    else if (!std::strcmp(name, "stamp")) {
        c->stamp_on = value > 0;
        if (c->stamp_on && !c->stamps) {
            int rc = dev_alloc(&c->stamps, (size_t)2 * kStampCap);
            if (rc) { c->stamp_on = 0; return rc; }
        }
    }
    else return FIRST_E_ARG;
    c->plan_version += 1;  // cached step graphs were built under the old options
    return FIRST_OK;
}

}  // extern "C"
