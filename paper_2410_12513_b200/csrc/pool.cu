// Slab pool for batches whose membership changes between decode steps.
//
// "Inference for FiRST", item 2: a sequence's layer decisions are taken once, on its prompt, and hold for its
// whole decode; a skipped (sequence, layer) needs no cache.  Sequences therefore come and go independently,
// and a sequence that joins needs cache rows only in the layers it keeps.  The pool hands out row ranges of
// caller-owned per-layer cache tensors on that basis, keeps the per-layer slab tables the decode step reads
// (first_kv_cache with per_layer = 1) in device memory, and rebuilds the per-layer active-row plan from the
// masks it holds on the host -- no call here waits for the stream.
#include <algorithm>
#include <cstring>
#include <new>
#include <utility>
#include <vector>

#include <cuda_runtime.h>

#include "first.h"

namespace {

constexpr int kMaxLayers = 96;  // the per-call tables below travel as kernel parameters

struct JoinArgs {            // one sequence entering (or leaving) slot `slot`
    int64_t off[kMaxLayers];      // first row of its slab in layer l (kept layers)
    const void* src_k[kMaxLayers];  // source cache tensors to import the prompt's keys/values from, or NULL
    const void* src_v[kMaxLayers];
    uint8_t keep[kMaxLayers];
};

// grid (L, Hkv), 128 threads.  Block (l, h): thread 0 of head 0 writes the tables of (l, slot); if the layer is
// kept and a source is given, the block copies the n tokens of head h from the source slab to the new one.
__global__ void __launch_bounds__(128) pool_join(const __grid_constant__ JoinArgs a, int slot, int B, int cap, int n,
                                                 int hd_bytes, int64_t src_cap_total, const int64_t* src_off, int src_seq,
                                                 void* const* dst_k, void* const* dst_v, const int64_t* rows,
                                                 int64_t* off, int32_t* capt, int32_t* len, int32_t* pos) {
    const int l = blockIdx.x, h = blockIdx.y;
    const bool keep = a.keep[l] != 0;
    if (h == 0 && threadIdx.x == 0) {
        off[(size_t)l * B + slot] = keep ? a.off[l] : 0;
        capt[(size_t)l * B + slot] = keep ? cap : 0;
        len[(size_t)l * B + slot] = keep ? n : 0;
        if (l == 0) pos[slot] = n;
    }
    if (!keep || !a.src_k[l] || n <= 0) return;
    const size_t bytes = (size_t)n * hd_bytes;  // head_dim * element size is a multiple of 16
    const size_t s0 = ((size_t)h * src_cap_total + (size_t)src_off[src_seq]) * hd_bytes;
    const size_t d0 = ((size_t)h * rows[l] + (size_t)a.off[l]) * hd_bytes;
    for (int which = 0; which < 2; ++which) {
        const uint4* src = reinterpret_cast<const uint4*>(static_cast<const uint8_t*>(which ? a.src_v[l] : a.src_k[l]) + s0);
        uint4* dst = reinterpret_cast<uint4*>(static_cast<uint8_t*>(which ? dst_v[l] : dst_k[l]) + d0);
        for (size_t e = threadIdx.x; e < bytes / 16; e += blockDim.x) dst[e] = src[e];
    }
}

}  // namespace

struct first_pool {
    first_ctx* ctx = nullptr;
    first_model_desc d{};
    int B = 0, L = 0;
    std::vector<int64_t> rows;                                    // token rows of layer l's tensors
    std::vector<std::vector<std::pair<int64_t, int64_t>>> free_;  // per layer: (start, length), sorted by start
    struct Seq { bool live = false; int cap = 0; std::vector<uint8_t> keep; std::vector<int64_t> off; };
    std::vector<Seq> seq;
    std::vector<void*> k_h, v_h;
    // device tables
    void **k_d = nullptr, **v_d = nullptr;
    int64_t *rows_d = nullptr, *off_d = nullptr;
    int32_t *cap_d = nullptr, *len_d = nullptr, *pos_d = nullptr;
};

namespace {

bool take(std::vector<std::pair<int64_t, int64_t>>& fl, int64_t want, int64_t* start) {
    for (size_t i = 0; i < fl.size(); ++i)
        if (fl[i].second >= want) {  // first fit
            *start = fl[i].first;
            fl[i].first += want;
            fl[i].second -= want;
            if (fl[i].second == 0) fl.erase(fl.begin() + i);
            return true;
        }
    return false;
}

void give(std::vector<std::pair<int64_t, int64_t>>& fl, int64_t start, int64_t len) {
    auto it = std::lower_bound(fl.begin(), fl.end(), std::make_pair(start, (int64_t)0));
    it = fl.insert(it, {start, len});
    if (it + 1 != fl.end() && it->first + it->second == (it + 1)->first) {  // merge with the next range
        it->second += (it + 1)->second;
        fl.erase(it + 1);
    }
    if (it != fl.begin() && (it - 1)->first + (it - 1)->second == it->first) {  // and with the previous one
        (it - 1)->second += it->second;
        fl.erase(it);
    }
}

}  // namespace

extern "C" {

int first_pool_create(first_ctx* ctx, int32_t max_seqs, const int64_t* rows_per_layer, void* const* k, void* const* v,
                      first_pool** out) {
    if (!ctx || !rows_per_layer || !k || !v || !out || max_seqs <= 0) return FIRST_E_ARG;
    *out = nullptr;
    first_model_desc d{};
    int rc = first_get_desc(ctx, &d);
    if (rc) return rc;
    if (max_seqs > d.max_batch) return FIRST_E_CAPACITY;
    if (d.n_layers > kMaxLayers) return FIRST_E_UNSUPPORTED;
    first_pool* p = new (std::nothrow) first_pool();
    if (!p) return FIRST_E_ARG;
    p->ctx = ctx; p->d = d; p->B = max_seqs; p->L = d.n_layers;
    p->rows.assign(rows_per_layer, rows_per_layer + p->L);
    p->free_.resize(p->L);
    p->seq.resize(max_seqs);
    p->k_h.assign(k, k + p->L);
    p->v_h.assign(v, v + p->L);
    for (int l = 0; l < p->L; ++l) {
        if (p->rows[l] < 0 || (p->rows[l] > 0 && (!k[l] || !v[l]))) { delete p; return FIRST_E_ARG; }
        if (p->rows[l] > 0) p->free_[l].push_back({0, p->rows[l]});
    }
    const size_t LB = (size_t)p->L * p->B;
    bool ok = cudaMalloc(&p->k_d, sizeof(void*) * p->L) == cudaSuccess && cudaMalloc(&p->v_d, sizeof(void*) * p->L) == cudaSuccess &&
              cudaMalloc(&p->rows_d, sizeof(int64_t) * p->L) == cudaSuccess && cudaMalloc(&p->off_d, sizeof(int64_t) * LB) == cudaSuccess &&
              cudaMalloc(&p->cap_d, sizeof(int32_t) * LB) == cudaSuccess && cudaMalloc(&p->len_d, sizeof(int32_t) * LB) == cudaSuccess &&
              cudaMalloc(&p->pos_d, sizeof(int32_t) * p->B) == cudaSuccess;
    ok = ok && cudaMemcpy(p->k_d, p->k_h.data(), sizeof(void*) * p->L, cudaMemcpyHostToDevice) == cudaSuccess &&
         cudaMemcpy(p->v_d, p->v_h.data(), sizeof(void*) * p->L, cudaMemcpyHostToDevice) == cudaSuccess &&
         cudaMemcpy(p->rows_d, p->rows.data(), sizeof(int64_t) * p->L, cudaMemcpyHostToDevice) == cudaSuccess &&
         cudaMemset(p->off_d, 0, sizeof(int64_t) * LB) == cudaSuccess && cudaMemset(p->cap_d, 0, sizeof(int32_t) * LB) == cudaSuccess &&
         cudaMemset(p->len_d, 0, sizeof(int32_t) * LB) == cudaSuccess && cudaMemset(p->pos_d, 0, sizeof(int32_t) * p->B) == cudaSuccess;
    if (!ok) { first_pool_destroy(p); return FIRST_E_CUDA; }
    *out = p;
    return FIRST_OK;
}

int first_pool_destroy(first_pool* p) {
    if (!p) return FIRST_OK;
    void* ptrs[] = {p->k_d, p->v_d, p->rows_d, p->off_d, p->cap_d, p->len_d, p->pos_d};
    for (void* q : ptrs)
        if (q) cudaFree(q);
    delete p;
    return FIRST_OK;
}

int first_seq_join(first_pool* p, const uint8_t* mask_row, int32_t capacity, const first_kv_cache* src, int32_t src_seq,
                   int32_t n_tokens, int32_t* slot_out, void* stream) {
    if (!p || !mask_row || !slot_out || capacity <= 0 || n_tokens < 0 || n_tokens > capacity) return FIRST_E_ARG;
    if (capacity > p->d.max_tokens_per_seq) return FIRST_E_CAPACITY;
    if (src && (src->per_layer || !src->k || !src->v || !src->slab_off || src->cap_total <= 0 || src_seq < 0)) return FIRST_E_ARG;
    for (int l = 0; l < p->L; ++l) {
        if (mask_row[l] > 1) return FIRST_E_ARG;
        if (src && mask_row[l] && (!src->k[l] || !src->v[l])) return FIRST_E_ARG;
    }
    int slot = -1;
    for (int b = 0; b < p->B; ++b)
        if (!p->seq[b].live) { slot = b; break; }
    if (slot < 0) return FIRST_E_CAPACITY;  // every batch row is taken
    JoinArgs a{};
    first_pool::Seq sq;
    sq.live = true; sq.cap = capacity;
    sq.keep.assign(mask_row, mask_row + p->L);
    sq.off.assign(p->L, 0);
    for (int l = 0; l < p->L; ++l) {
        if (!mask_row[l]) continue;
        if (!take(p->free_[l], capacity, &sq.off[l])) {  // this layer has no room: hand back what was taken
            for (int j = 0; j < l; ++j)
                if (mask_row[j]) give(p->free_[j], sq.off[j], capacity);
            return FIRST_E_CAPACITY;
        }
    }
    for (int l = 0; l < p->L; ++l) {
        a.off[l] = sq.off[l];
        a.keep[l] = mask_row[l];
        a.src_k[l] = src ? src->k[l] : nullptr;
        a.src_v[l] = src ? src->v[l] : nullptr;
    }
    const int esz = p->d.dtype == FIRST_DTYPE_BF16 ? 2 : 4;
    pool_join<<<dim3(p->L, p->d.n_kv_heads), 128, 0, static_cast<cudaStream_t>(stream)>>>(
        a, slot, p->B, capacity, n_tokens, p->d.head_dim * esz, src ? src->cap_total : 0, src ? src->slab_off : nullptr,
        src_seq, p->k_d, p->v_d, p->rows_d, p->off_d, p->cap_d, p->len_d, p->pos_d);
    if (cudaGetLastError() != cudaSuccess) {
        for (int l = 0; l < p->L; ++l)
            if (mask_row[l]) give(p->free_[l], sq.off[l], capacity);
        return FIRST_E_CUDA;
    }
    p->seq[slot] = std::move(sq);
    *slot_out = slot;
    return FIRST_OK;
}

int first_seq_leave(first_pool* p, int32_t slot, void* stream) {
    if (!p || slot < 0 || slot >= p->B) return FIRST_E_ARG;
    first_pool::Seq& sq = p->seq[slot];
    if (!sq.live) return FIRST_E_STATE;
    JoinArgs a{};  // keep = 0 everywhere: the slot's tables go back to "no slab, nothing present"
    pool_join<<<dim3(p->L, 1), 128, 0, static_cast<cudaStream_t>(stream)>>>(
        a, slot, p->B, 0, 0, 0, 0, nullptr, 0, p->k_d, p->v_d, p->rows_d, p->off_d, p->cap_d, p->len_d, p->pos_d);
    if (cudaGetLastError() != cudaSuccess) return FIRST_E_CUDA;
    for (int l = 0; l < p->L; ++l)
        if (sq.keep[l]) give(p->free_[l], sq.off[l], sq.cap);
    sq = first_pool::Seq();
    return FIRST_OK;
}

int first_pool_commit(first_pool* p, void* stream) {
    if (!p) return FIRST_E_ARG;
    std::vector<uint8_t> mask((size_t)p->B * p->L, 0);
    for (int b = 0; b < p->B; ++b)
        if (p->seq[b].live) std::memcpy(&mask[(size_t)b * p->L], p->seq[b].keep.data(), p->L);
    return first_set_mask_host(p->ctx, mask.data(), p->B, stream);
}

int first_pool_kv(first_pool* p, first_kv_cache* out) {
    if (!p || !out) return FIRST_E_ARG;
    std::memset(out, 0, sizeof *out);
    out->k = p->k_h.data();
    out->v = p->v_h.data();
    out->slab_off = p->off_d;
    out->slab_cap = p->cap_d;
    out->len = p->len_d;
    out->pos = p->pos_d;
    out->per_layer = 1;
    out->cap_total_l = p->rows.data();
    return FIRST_OK;
}

int first_pool_stats(first_pool* p, int64_t* rows_held, int64_t* largest_free, int32_t* live) {
    if (!p) return FIRST_E_ARG;
    for (int l = 0; l < p->L; ++l) {
        int64_t fr = 0, big = 0;
        for (auto& r : p->free_[l]) { fr += r.second; big = std::max(big, r.second); }
        if (rows_held) rows_held[l] = p->rows[l] - fr;
        if (largest_free) largest_free[l] = big;
    }
    if (live) {
        *live = 0;
        for (auto& sq : p->seq) *live += sq.live ? 1 : 0;
    }
    return FIRST_OK;
}

}  // extern "C"
