/*
 * first.h -- C ABI of the router-selective decode step of FiRST (arXiv 2410.12513)
 * for one NVIDIA B200 (sm_100a).
 *
 * The method (paper sections in quotes):
 *   "Adaptive Router Module": before every transformer layer i sits a router R_i, a
 *     bias-free linear map D -> 1.  It is applied to every prompt token's hidden state
 *     entering layer i, a sigmoid is taken per token, and the mean over the sequence's
 *     tokens is rho_i, the probability of running layer i for that sequence.
 *   "Proposed Solution": at inference rho_i is rounded, keep = (rho_i >= 0.5), and
 *     H_i = H_{i-1} + keep * phi_i(H_{i-1}) (Eq. 3 and the unnumbered inference rule):
 *     a skipped layer is the identity on that sequence's residual stream.
 *   "Inference for FiRST": (1) nothing is skipped during prefill; (2) the decisions
 *     taken on the prompt are cached and every decode step obeys them, so a kept layer
 *     always holds the K/V of all earlier tokens and a skipped layer needs none.
 *
 * This library is the decode-time hot path of that: score the routers on prefill hidden
 * states (first_prefill_route), turn the per-sequence masks into per-layer lists of
 * active rows (first_set_mask), and run decode steps in which each layer's kernels see
 * only the rows that keep it (first_decode_step).  first_prefill is the step before it:
 * the whole prompt phase of a ragged batch (caches of all layers, router decisions, first
 * token) in one call, for callers that have no prefill of their own.
 *
 * General conventions
 *   - Every function returns a status: 0 = FIRST_OK, negative = error; nothing throws.
 *   - Pointers marked "dev" are device memory of the current CUDA device, "host" are
 *     ordinary host memory.  All tensors are owned by the caller and only borrowed:
 *     weights for the lifetime of the context, everything else for the call (the
 *     kernels of a call may still be running on `stream` when it returns).
 *   - The library allocates device memory in first_create (its own scratch) and frees it in
 *     first_destroy; the two later allocations are stated where they happen (first_prefill's
 *     token scores, the internal logits row buffer of first_decode_step without `logits`).
 *   - Work is enqueued on the CUDA stream passed as `void *stream` (a cudaStream_t;
 *     NULL = the default stream).  Only first_set_mask, first_prefill, first_last_device_flags
 *     and the measurement aids wait for the stream.
 *   - Layers are numbered from 0.  mask[b][l] is a byte, 1 = sequence b runs layer l,
 *     0 = it skips it.  All matrices are row-major; linear weights are [out][in].
 *   - dtype FIRST_DTYPE_F32: weight matrices and KV cache are float32.
 *     dtype FIRST_DTYPE_BF16: weight matrices and KV cache are bfloat16.
 *     Norm gains, router weights, the residual stream and logits are always float32.
 *   - Errors the host cannot see without a device read (cache slab full, token id out
 *     of range, mask byte not 0/1, a bounded wait that ran out) set bits in a device
 *     flag word; the offending row is left untouched.  first_last_device_flags reads it.
 */
#ifndef FIRST_H
#define FIRST_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define FIRST_OK 0
#define FIRST_E_ARG (-1)         /* NULL pointer, negative size, value out of range */
#define FIRST_E_SHAPE (-2)       /* sizes inconsistent with the model description */
#define FIRST_E_UNSUPPORTED (-3) /* a shape or dtype the kernels do not cover */
#define FIRST_E_CAPACITY (-4)    /* batch or token count beyond what the context was sized for */
#define FIRST_E_CUDA (-5)        /* a CUDA runtime or driver call failed */
#define FIRST_E_DEVICE_FLAG (-6) /* the device flag word is non-zero */
#define FIRST_E_STATE (-7)       /* call order: e.g. decode before first_set_mask */

#define FIRST_DTYPE_F32 0
#define FIRST_DTYPE_BF16 1

#define FIRST_FLAG_KV_FULL 1u      /* a kept (sequence, layer) had len == slab_cap */
#define FIRST_FLAG_BAD_TOKEN 2u    /* token id outside [0, vocab) */
#define FIRST_FLAG_BAD_MASK 4u     /* mask byte other than 0 or 1 */
#define FIRST_FLAG_WAIT_EXPIRED 8u /* a bounded wait inside a kernel gave up */
#define FIRST_FLAG_EMPTY_SEQ 16u   /* a router call saw a sequence with no tokens */
#define FIRST_FLAG_BAD_SEQ_TABLE 32u /* a router call saw cu_seqlens entries that are negative, decreasing or
                                        beyond total_tokens; that sequence's mask byte and score are unwritten */

#define FIRST_ROUTER_MEAN_OF_SIGMOID 0 /* the paper's order: rho = mean_j sigmoid(z_j) */
#define FIRST_ROUTER_SIGMOID_OF_MEAN 1 /* pooled variant:    rho = sigmoid(mean_j z_j) */

typedef struct first_ctx first_ctx;

/* Decoder shape (the paper uses LLaMA-3 models; the block is the public LLaMA block:
 * RMSNorm, rotary q/k with half-split pairing, grouped-query causal attention, SwiGLU). */
typedef struct {
    int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, ffn_dim, vocab;
    float rope_base, rms_eps;
    int32_t dtype;              /* FIRST_DTYPE_* */
    int32_t max_batch;          /* largest B any later call will use */
    int32_t max_tokens_per_seq; /* largest slab capacity of any sequence */
} first_model_desc;

/* Weights.  The pointer-array members are HOST arrays of n_layers DEVICE pointers. */
typedef struct {
    const void *embed;              /* dev [vocab][d_model]                         */
    const void *lm_head;            /* dev [vocab][d_model]                         */
    const float *final_norm;        /* dev [d_model]                                */
    const float *const *attn_norm;  /* host[L] -> dev [d_model]                     */
    const void *const *wqkv;        /* host[L] -> dev [(Hq+2*Hkv)*hd][d_model]: q rows, k rows, v rows */
    const void *const *wo;          /* host[L] -> dev [d_model][Hq*hd]              */
    const float *const *ffn_norm;   /* host[L] -> dev [d_model]                     */
    const void *const *w_gate_up;   /* host[L] -> dev [2*ffn_dim][d_model]: gate rows, then up rows */
    const void *const *w_down;      /* host[L] -> dev [d_model][ffn_dim]            */
} first_weights;

/* KV cache, caller-owned.  Layer l's keys are one tensor [Hkv][cap_total][hd]; sequence
 * b owns token rows slab_off[b] .. slab_off[b]+slab_cap[b]-1 of every head ("ragged
 * slabs").  len[l][b] tokens are present.  Item (2) of "Inference for FiRST": a kept
 * (b,l) gains one token per step, a skipped (b,l) is neither read nor written and its
 * len stays where prefill left it.  pos[b] is the absolute index of the token being
 * fed (the rotary position), advanced by one per step for every sequence. */
typedef struct {
    void *const *k;          /* host[L] -> dev [Hkv][cap_total][hd] */
    void *const *v;          /* host[L] -> dev [Hkv][cap_total][hd] */
    const int64_t *slab_off; /* dev [B] */
    const int32_t *slab_cap; /* dev [B] */
    int32_t *len;            /* dev [L][B], updated by first_decode_step */
    int32_t *pos;            /* dev [B],    updated by first_decode_step */
    int64_t cap_total;       /* token rows per head in each layer tensor (per_layer = 0) */
    /* Per-layer slab tables.  A sequence that skips layer l needs no cache there during decode
     * ("Inference for FiRST", item 2), so once the masks are known a caller can keep, per layer,
     * slabs only for the sequences that keep it and hand the memory of the others back.  With
     * per_layer = 1: slab_off is dev [L][B], slab_cap dev [L][B] (0 for a skipped (l,b); its
     * slab_off is ignored), layer l's tensors are [Hkv][cap_total_l[l]][hd], cap_total is unused.
     * The heights are baked into recorded step graphs: call first_set_mask after changing them. */
    int32_t per_layer;             /* 0 (tables shared by all layers) or 1 */
    const int64_t *cap_total_l;    /* host [L], per_layer = 1 only */
} first_kv_cache;

/* Create a context for one model on the current device: validates the description,
 * borrows the weights, allocates scratch sized by max_batch / max_tokens_per_seq.
 * Errors: FIRST_E_ARG, FIRST_E_SHAPE (head_dim*heads, divisibility), FIRST_E_UNSUPPORTED
 * (head_dim not in {32,64,128}; Hq/Hkv not in {1,2,3,4,8}; d_model, ffn_dim not multiples
 * of 8), FIRST_E_CUDA. */
int first_create(const first_model_desc *desc, const first_weights *weights, first_ctx **out);
int first_destroy(first_ctx *ctx);

/* Router of ONE layer on that layer's prefill input ("Adaptive Router Module"; rounding
 * rule of "Proposed Solution").  hidden holds the hidden states entering `layer` for all
 * prompt tokens of a ragged batch, sequence b at rows cu_seqlens[b] .. cu_seqlens[b+1]-1.
 *   z_j = router_w . hidden[j] (+ *router_b if router_b != NULL; the paper has no bias)
 *   mode FIRST_ROUTER_MEAN_OF_SIGMOID: rho_b = mean_j sigmoid(z_j)
 *   mode FIRST_ROUTER_SIGMOID_OF_MEAN: rho_b = sigmoid(mean_j z_j)
 *   mask[b][layer] = (rho_b >= tau) ? 1 : 0   (equality keeps the layer), scores[b][layer] = rho_b.
 * Token scores are float32, the per-sequence mean is taken in float64 in a fixed order,
 * so the result does not depend on the launch shape.
 *   ctx           required: it owns the per-token scratch the two passes share
 *   hidden        dev [total_tokens][d_model], float32 or bfloat16 (hidden_dtype)
 *   cu_seqlens    dev int32 [B+1], cu_seqlens[0] = 0, non-decreasing; every sequence needs
 *                 at least one token (an empty one sets FIRST_FLAG_EMPTY_SEQ and its mask
 *                 byte and score are left unwritten)
 *   total_tokens  host value of cu_seqlens[B] (sizes the launch); at most
 *                 max_batch*max_tokens_per_seq (the scratch capacity).  The device table is checked
 *                 against it: a sequence whose rows are negative, run backwards or end beyond
 *                 total_tokens sets FIRST_FLAG_BAD_SEQ_TABLE, reads nothing and leaves its mask
 *                 byte and score unwritten
 *   router_w      dev float32 [d_model];  router_b  dev float32 [1] or NULL
 *   mask          dev uint8 [B][n_layers] (only column `layer` is written)
 *   scores        dev float32 [B][n_layers] or NULL
 * Errors: FIRST_E_ARG, FIRST_E_CAPACITY, FIRST_E_UNSUPPORTED (d_model > 12288), FIRST_E_CUDA. */
int first_prefill_route(first_ctx *ctx, int32_t layer, const void *hidden, int32_t hidden_dtype,
                        const int32_t *cu_seqlens, int32_t B, int64_t total_tokens, const float *router_w,
                        const float *router_b, float tau, int32_t mode, uint8_t *mask, float *scores,
                        void *stream);

/* The router call for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a deployment variant of first_prefill_route, same arithmetic, same
 * kernels, same results.)
 *
 * Who needs it: first_prefill_route takes its per-token scratch from a context, and
 * creating a context calls cudaMalloc.  Some hosts cannot do that at the point where they
 * want to route a batch: a serving process whose framework allocator has already reserved
 * the whole GPU, so that a raw cudaMalloc fails; a plugin that runs under a fixed memory
 * budget it may not exceed; code on a latency-critical path where cudaMalloc's implicit
 * device-wide synchronisation is not acceptable.  This entry point needs no context and
 * calls no cudaMalloc, cudaFree or other allocating routine.  Its scratch is a fixed array
 * compiled into the library image: FIRST_STATIC_ROUTE_MAX_TOKENS float32 token scores plus
 * a 256-byte header (4 MiB + 256 B).  Every GPU on which a process loads this library
 * holds that array until the process exits, whether or not this call is ever used.
 *
 * Arguments are those of first_prefill_route, with n_layers and d_model passed directly
 * (d_model a multiple of 8, at most 12288) and
 *   flags   dev uint32 [1] or NULL: receives FIRST_FLAG_EMPTY_SEQ / FIRST_FLAG_BAD_SEQ_TABLE (OR-ed in, never cleared
 *           here).  With NULL a word inside the built-in scratch is used; it is reset to
 *           zero at the start of every call and cannot be read back by the caller.
 * Limits and rules:
 *   - total_tokens > FIRST_STATIC_ROUTE_MAX_TOKENS returns FIRST_E_CAPACITY, nothing runs.
 *   - The first call on each device looks up the array's device address (once per device,
 *     with that device current).  Make that first call outside any stream capture.
 *   - All calls on a device share the one array and it keeps the previous call's contents.
 *     Token scores are fully rewritten before they are read, so stale contents are harmless,
 *     but two calls whose kernels overlap on the GPU (different streams, or different host
 *     threads on different streams) race on it: keep calls on one stream, or order them.
 * Errors: FIRST_E_ARG, FIRST_E_UNSUPPORTED (d_model), FIRST_E_CAPACITY, FIRST_E_CUDA. */
#define FIRST_STATIC_ROUTE_MAX_TOKENS 1048576
int first_prefill_route_static(int32_t layer, int32_t n_layers, int32_t d_model, const void *hidden,
                               int32_t hidden_dtype, const int32_t *cu_seqlens, int32_t B, int64_t total_tokens,
                               const float *router_w, const float *router_b, float tau, int32_t mode,
                               uint8_t *mask, float *scores, uint32_t *flags, void *stream);

/* Prompt phase of a ragged batch, in one call ("Inference for FiRST", item 1: no layer is skipped
 * while the prompt is processed; "Adaptive Router Module": router l reads the hidden states that
 * enter layer l, for every prompt token, and its mean over the sequence decides the layer for that
 * sequence).  For every sequence b with prompt tokens[cu_seqlens[b] .. cu_seqlens[b+1]-1]:
 * all layers run on all prompt tokens (causal attention inside the prompt), the rotated keys and
 * the values of all n_b tokens are written to rows 0..n_b-1 of b's slab in EVERY layer,
 * len[l][b] = n_b, pos[b] = n_b; router l's score rho[b][l] and mask[b][l] are formed as in
 * first_prefill_route from the float32 residual stream entering layer l; logits[b] is the
 * distribution after the last prompt token and next_tokens[b] its argmax (or a sampled token,
 * see first_set_sampling) -- the first generated token, to be fed to the first first_decode_step.
 * Whatever the slabs held before is overwritten from row 0.
 *
 * How it runs: the prompt tokens go through the kernels of first_decode_step in chunks of
 * min(max_batch, 256) tokens (option "prefill_rows"), each token a row of its own (its slab is
 * its sequence's slab, its cache length its position), so a context meant for prefill should
 * be created with max_batch of 256 or more.  Weights are streamed once per chunk.  The chunks run without CUDA graphs.
 *   tokens        dev int32 [total], total = cu_seqlens[B]
 *   cu_seqlens    HOST int32 [B+1], cu_seqlens[0] = 0, strictly increasing (no empty prompt);
 *                 every prompt at most max_tokens_per_seq tokens, B at most max_batch
 *   kv            host struct, per_layer = 0 (FIRST_E_UNSUPPORTED otherwise); a slab shorter than
 *                 its prompt sets FIRST_FLAG_KV_FULL and keeps only the tokens that fit
 *   router_w      dev float32 [n_layers][d_model], or NULL: no routing, mask/scores untouched
 *   router_b      dev float32 [n_layers] or NULL (the paper's routers have no bias)
 *   tau, mode     as in first_prefill_route
 *   mask          dev uint8 [B][n_layers] (required with router_w); scores dev float32 [B][n_layers] or NULL
 *   logits        dev float32 [B][vocab] or NULL;  next_tokens  dev int32 [B] or NULL
 * The call waits for the stream before it returns.  It replaces the context's plan: call
 * first_set_mask (with the mask it produced, or any other) before the next first_decode_step.
 * With routers, the first call allocates n_layers*total float32 of token scores (kept, and
 * grown when a later call needs more); must not be called while `stream` is being captured.
 * Errors: FIRST_E_ARG, FIRST_E_CAPACITY, FIRST_E_UNSUPPORTED, FIRST_E_STATE (stream capture),
 * FIRST_E_CUDA; device flags for a full slab or a bad token id. */
int first_prefill(first_ctx *ctx, const int32_t *tokens, const int32_t *cu_seqlens, int32_t B,
                  const first_kv_cache *kv, const float *router_w, const float *router_b, float tau, int32_t mode,
                  uint8_t *mask, float *scores, float *logits, int32_t *next_tokens, void *stream);

/* Fix the skip mask of the current batch and build, per layer, the ascending list of
 * rows that keep it (one decision per sequence per layer, "Adaptive Router Module";
 * fixed for all decode steps, "Inference for FiRST" item 2).  Must be called before
 * first_decode_step and again whenever the batch or its mask changes.  Waits for the
 * stream (the per-layer counts shape the later launches).
 *   mask  dev uint8 [B][n_layers]
 * Errors: FIRST_E_ARG, FIRST_E_CAPACITY (B > max_batch), FIRST_E_DEVICE_FLAG (a mask byte
 * other than 0/1), FIRST_E_CUDA. */
int first_set_mask(first_ctx *ctx, const uint8_t *mask, int32_t B, void *stream);

/* first_set_mask for a mask held in HOST memory, without waiting for the stream (a batch that changes
 * between steps should not stall the device: decisions are per sequence and fixed for its whole decode,
 * "Inference for FiRST" item 2, so sequences come and go independently).  The per-layer counts are taken
 * on the host; the launches of later steps are sized from them rounded up to a multiple of 16 and the
 * kernels read the exact counts from device memory, so a recorded step graph is found again after any
 * change of the batch that leaves every layer's count inside its bucket of 16.
 *   mask  host uint8 [B][n_layers], bytes 0/1 (FIRST_E_ARG otherwise); copied before the call returns
 * Errors: FIRST_E_ARG, FIRST_E_CAPACITY, FIRST_E_STATE (stream being captured), FIRST_E_CUDA. */
int first_set_mask_host(first_ctx *ctx, const uint8_t *mask, int32_t B, void *stream);

/* Read back the plan of the last first_set_mask (for inspection and tests).
 *   idx   host int32 [n_layers][B]: idx[l][0..cnt[l]-1] ascending active rows, rest -1
 *   cnt   host int32 [n_layers]
 *   slot  host int32 [n_layers][B] or NULL: position of row b in idx[l], -1 if skipped */
int first_get_plan(first_ctx *ctx, int32_t *idx, int32_t *cnt, int32_t *slot);

/* One routed decode step for the whole batch (inference rule of "Proposed Solution";
 * "Inference for FiRST" item 2).  For every sequence b: x = embed[tokens[b]]; for each
 * layer l with mask[b][l] = 1: append the token's rotated key and value at row len[l][b]
 * of its slab, attend over the len[l][b]+1 tokens, x += attention, x += SwiGLU FFN; layers
 * with mask 0 leave x, the slab and len untouched.  logits[b] = lm_head . RMSNorm(x).
 * Then pos[b] += 1.
 *   tokens        dev int32 [B]
 *   kv            host struct; see first_kv_cache
 *   logits        dev float32 [B][vocab], or NULL
 *   next_tokens   dev int32 [B] or NULL: argmax of the logits row, lowest index on ties (or a
 *                 sampled token, see first_set_sampling)
 *   layer_inputs  dev float32 [n_layers][B][d_model] or NULL: the residual entering each
 *                 layer (what router l reads when prompts are prefilled token by token
 *                 with an all-keep mask)
 * B is the batch of the last first_set_mask.
 * Errors: FIRST_E_ARG, FIRST_E_STATE (no mask set), FIRST_E_CUDA; device flags for a full
 * slab or a bad token id. */
int first_decode_step(first_ctx *ctx, const int32_t *tokens, const first_kv_cache *kv, float *logits,
                      int32_t *next_tokens, float *layer_inputs, void *stream);

/* Batches whose membership changes between steps ("Inference for FiRST", item 2: a sequence's layer
 * decisions are fixed once its prompt has been routed, and a layer it skips needs no cache).  A pool
 * manages row ranges ("slabs") of caller-owned per-layer cache tensors: a sequence that joins gets a
 * batch row (slot) and, in every layer it KEEPS, a slab of `capacity` token rows; layers it skips get
 * nothing, so the cache memory in use is the sum over kept (sequence, layer) pairs.  The pool keeps the
 * per-layer slab tables of first_kv_cache (per_layer = 1) in device memory and its sequences' masks on
 * the host.  None of these calls waits for the stream; all calls of a pool, and the decode steps on its
 * cache, belong on one stream (a slab freed by first_seq_leave may be handed out by the next join).
 *
 * first_pool_create   max_seqs <= max_batch batch rows; rows_per_layer host int64 [L]: token rows of layer
 *                     l's tensors k[l], v[l] (dev [Hkv][rows_per_layer[l]][hd], caller-owned, borrowed for
 *                     the pool's lifetime).  Allocates the pool's small device tables.
 * first_seq_join      mask_row host uint8 [L] (the sequence's decisions); capacity = slab rows per kept layer
 *                     (<= max_tokens_per_seq).  src != NULL: the keys/values of the sequence's first
 *                     n_tokens tokens are copied, for the kept layers, from sequence src_seq of cache `src`
 *                     (per_layer = 0, e.g. the cache a first_prefill call filled), len = pos = n_tokens;
 *                     src == NULL: nothing is copied; the first n_tokens rows of the new slabs count as
 *                     present, whatever they hold (0 for empty slabs).  *slot = the batch row: the caller
 *                     feeds the sequence's tokens at tokens[slot] and reads its logits at row slot.
 *                     FIRST_E_CAPACITY: no free batch row, or some kept layer has no free range of
 *                     `capacity` rows (nothing is taken then).
 * first_seq_leave     frees the slot and its slabs.
 * first_pool_commit   rebuilds the step's per-layer active-row plan for the sequences now in the pool
 *                     (first_set_mask_host over all max_seqs batch rows; free rows skip every layer).  Call
 *                     after a group of joins and leaves, before the next first_decode_step.
 * first_pool_kv       fills *out with the pool's cache view (per_layer = 1) for first_decode_step; tokens
 *                     and outputs of a step have max_seqs rows; free rows need a valid token id.
 * first_pool_stats    rows_held[l] = token rows handed out in layer l, largest_free[l] = longest free range,
 *                     *live = sequences in the pool (host arrays of L entries, any may be NULL).
 * Errors: FIRST_E_ARG, FIRST_E_CAPACITY, FIRST_E_UNSUPPORTED (more than 96 layers), FIRST_E_STATE (leave of
 * a free slot), FIRST_E_CUDA. */
typedef struct first_pool first_pool;
int first_pool_create(first_ctx *ctx, int32_t max_seqs, const int64_t *rows_per_layer, void *const *k, void *const *v,
                      first_pool **out);
int first_pool_destroy(first_pool *pool);
int first_seq_join(first_pool *pool, const uint8_t *mask_row, int32_t capacity, const first_kv_cache *src,
                   int32_t src_seq, int32_t n_tokens, int32_t *slot, void *stream);
int first_seq_leave(first_pool *pool, int32_t slot, void *stream);
int first_pool_commit(first_pool *pool, void *stream);
int first_pool_kv(first_pool *pool, first_kv_cache *out);
int first_pool_stats(first_pool *pool, int64_t *rows_held, int64_t *largest_free, int32_t *live);

/* The description a context was created with; the number of recorded step graphs it holds. */
int first_get_desc(const first_ctx *ctx, first_model_desc *out);
int64_t first_graph_count(const first_ctx *ctx);

/* Next-token sampling with the paper's generation settings (appendix "Training and Inference
 * Setup", inference settings: temperature 0.8, top-k sampling over 10 tokens).  Per row: the
 * candidates are the top_k largest logits, equal values in index order; their weights are
 * exp((logit - max) / temperature); the token is the first candidate, in that order, whose
 * cumulative weight exceeds u * (sum of weights), u the row's uniform draw.  The draws are an
 * input: the library holds no generator.  Arithmetic is float32.
 *   logits     dev float32 [B][vocab]
 *   top_k      1 .. FIRST_SAMPLE_TOPK_MAX (and <= vocab); 1 is greedy decoding
 *   temperature >= 0; 0 is greedy decoding
 *   uniforms   dev float32 [B], each in [0,1); a value outside selects the last candidate
 *   tokens     dev int32 [B]
 * first_sample_topk is stateless (no context; one launch on `stream`).
 * first_set_sampling makes every later first_decode_step of the context fill next_tokens this
 * way instead of by argmax, reading `uniforms` (borrowed; the caller refreshes its contents
 * before each step, in stream order); top_k <= 1 or temperature 0 restores argmax.
 * Errors: FIRST_E_ARG, FIRST_E_UNSUPPORTED (top_k > FIRST_SAMPLE_TOPK_MAX), FIRST_E_CUDA. */
#define FIRST_SAMPLE_TOPK_MAX 16
int first_set_sampling(first_ctx *ctx, int32_t top_k, float temperature, const float *uniforms);
int first_sample_topk(const float *logits, int32_t B, int32_t vocab, int32_t top_k, float temperature,
                      const float *uniforms, int32_t *tokens, void *stream);

/* Wait for `stream`, read and clear the device flag word.  Returns FIRST_OK with
 * *flags = 0, or FIRST_E_DEVICE_FLAG with the FIRST_FLAG_* bits in *flags. */
int first_last_device_flags(first_ctx *ctx, uint32_t *flags, void *stream);

/* Self-test of the bounded waits (the paper has no counterpart).  Every wait on a copy or on another role
 * inside the kernels gives up after a fixed number of polls, raises FIRST_FLAG_WAIT_EXPIRED and lets the
 * kernel end; a step in which that happened has undefined outputs (first_last_device_flags then also
 * clears the attention merge counters, so later steps are sound).  This call runs that give-up path on
 * purpose, harmlessly: one thread waits `polls` (1 .. 2^20) times on a barrier nothing will ever complete,
 * with no copy in flight.  *returned = what the wait reported (0 = gave up), *abort_word = the CTA's abort
 * word (1); the context's flag word gets FIRST_FLAG_WAIT_EXPIRED.  Waits for `stream`. */
int first_selftest_wait_expiry(first_ctx *ctx, int32_t polls, int32_t *returned, int32_t *abort_word, void *stream);

/* Number of kernels this context has launched so far (for launch accounting). */
int64_t first_launch_count(const first_ctx *ctx);

/* Measurement aid (the paper has no counterpart): per-kernel-class device timing.  While
 * enabled, every launch of this context is bracketed by a CUDA event pair on its stream
 * (this serialises launches slightly; leave it off when timing whole steps).
 * first_profile(ctx, 1) clears the totals and starts; first_profile(ctx, 0) stops.
 * first_profile_read waits for `stream`, folds the pending event pairs into the totals and
 * copies them out: ms[k] = total device milliseconds of class k, launches[k] = its launch
 * count, for k < first_kernel_class_count() (n must be at least that).  Host arrays. */
int first_profile(first_ctx *ctx, int32_t enable);
int first_profile_read(first_ctx *ctx, int32_t n, double *ms, int64_t *launches, void *stream);
int32_t first_kernel_class_count(void);
const char *first_kernel_class_name(int32_t k);

/* Measurement aid (the paper has no counterpart): where a step's time goes WITHOUT serialising it.
 * With option "stamp" = 1 every kernel of a step records, in device memory, when its first CTA
 * started and when its last warp ended (global nanosecond timer); the step runs as it always does
 * (one CUDA graph, programmatic dependent launch).  first_step_trace waits for `stream` and copies
 * out the last step's launches in launch order: cls[i] = kernel class (first_kernel_class_name),
 * t_start[i], t_end[i] in nanoseconds of one clock.  The time from launch i-1's end to launch i's
 * end, summed per class, splits the step's duration among the classes without double counting.
 * Steps with more than 2048 launches are truncated.  Host arrays of max_n entries; *n_out = entries
 * written.  Errors: FIRST_E_ARG, FIRST_E_STATE (option off), FIRST_E_CUDA. */
int first_step_trace(first_ctx *ctx, int32_t max_n, int32_t *cls, uint64_t *t_start, uint64_t *t_end,
                     int32_t *n_out, void *stream);

/* Options (A/B measurements and tuning).  A negative value restores the default.
 *   "max_gemv_rows"  largest active-row count served by the CUDA-core GEMV path; layers with
 *                    more rows use the tensor-core path when the dtype is bfloat16 (default 0: with TMA streaming
 *                    and weight prefetch across kernel boundaries it is the faster path even for one row;
 *                    float32 models always use the GEMV path)
 *   "attn_simple"    1 = always use the general attention kernel
 *   "attn_chunk"     tokens per attention work item (rounded up to 64); default: from the batch
 *   "tc_use_lo"      0 = tensor-core projections use only the bfloat16 hi half of activations
 *   "use_graph"      0 = launch every kernel of a step directly.  Default 1: first_decode_step
 *                    records its launch sequence once per distinct set of pointer arguments
 *                    (tokens, outputs, cache tensors) and per-layer launch rows, as a CUDA graph, and
 *                    replays it; up to 16 such graphs are kept (least recently used dropped), across
 *                    first_set_mask calls: the row lists live in device memory, not in the graph.  Nothing is captured while the
 *                    caller's stream is itself being captured or while first_profile is on.
 *   "tc_lo_max_rows" the hi/lo activation split is used for projections with at most this many
 *                    active rows, the hi half alone above (default: always both halves; the hi
 *                    half alone is bfloat16-activation accuracy and misses the parity bar)
 *   "tc_mt2_min_rows" from this many active rows on a projection CTA takes two weight tiles per
 *                    activation tile (default: when the activation tiles are so wide that only one
 *                    single-tile CTA would fit per SM, i.e. from 96 rows)
 *   "norm_threads"   threads per RMSNorm CTA (one CTA per row), a multiple of 32 up to 1024; default 512
 *   "attn_cluster"   1 = the chunks of a split attention row are launched as a thread-block cluster and merge through
 *                    the first chunk's shared memory (up to 8 chunks) instead of through global memory; default 0
 *   "tc2_min_rows"   from this many active rows on a tensor-core projection launch runs as CTA pairs (two SMs per
 *                    unit, cta_group::2 MMA, each SM holding half of the activation rows); default 96, 0 = never
 *   "tc2_mt2_all"    1 = the CTA-pair kernel takes two weight tiles per unit for the reducing epilogues too
 *   "tc_ksplit_cap"  0 = do not bound the number of K ranges by the reduction traffic
 *   "tc_smem_kb"     shared-memory budget per projection CTA when two CTAs per SM are wanted (110)
 *   "fuse_rope"      0 = a separate kernel rotates q/k and appends the new key/value before attention.
 *                    Default 1: the tuned attention kernel (bfloat16 caches, head_dim 64/128) does both
 *                    itself, from the QKV projection's output.
 *   "prefill_pair"   0 = in first_prefill every prompt token has attention work items of its own.  Default 1:
 *                    two consecutive tokens of a sequence share them (up to 4 query heads per KV head).
 *   "prefill_group"  0 = no groups.  Default 1 (used when "prefill_tc" is 0): in first_prefill up to eight consecutive tokens of a sequence (one
 *                    block of eight positions) share attention work items, so a prefix's keys/values are staged once
 *                    per eight tokens (up to 4 query heads per KV head; otherwise the pair form or single rows)
 *   "prefill_tc"     0 = prompt-chunk attention on the mma.sync kernels ("prefill_group" / "prefill_pair" choose the
 *                    form).  Default 1: causal attention of prompt chunks on the tcgen05 tensor cores, blocks of
 *                    128 / (query heads per KV head) consecutive tokens per work item (bfloat16 caches, head_dim 64
 *                    or 128, 1, 2, 3, 4 or 8 query heads per KV head; otherwise the forms below)
 *   "prefill_lo"     0 = the projections of first_prefill's chunks multiply by the bfloat16 hi half of the
 *                    activations alone (half the tensor work; plain bfloat16-activation accuracy: measured 2.3e-2 of
 *                    the logit range at 32 layers, outside the 2e-2 bar).  Default 1: hi + lo halves as everywhere
 *   "prefill_slack"  0..16, default 8: that kernel keeps its softmax weights relative to a reference maximum which
 *                    moves (and the accumulated output is rescaled) only when a tile's maximum exceeds it by more than
 *                    2^value; 0 = the reference follows the running maximum exactly (the result is the same up to
 *                    rounding; tests use 0 to exercise the rescaling)
 *   "prefill_rows"   prompt tokens per chunk of first_prefill, 1..256 (default 256; never more than max_batch)
 *   "fuse_swiglu"    0 = gate/up projection writes float32 sums and a separate kernel applies
 *                    silu(gate)*up.  Default 1: the tensor-core gate/up projection applies it in
 *                    its epilogue (needs ffn_dim % 64 == 0).
 *   "stamp"          1 = record per-launch start/end times for first_step_trace (default 0)
 *   "use_pdl"        0 = kernels of a step are launched strictly one after another.  Default 1:
 *                    programmatic dependent launch lets a kernel's prologue (and, for the
 *                    projections, its first weight tiles) overlap the previous kernel's tail.
 * Errors: FIRST_E_ARG for an unknown name. */
int first_set_option(first_ctx *ctx, const char *name, int64_t value);

const char *first_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* FIRST_H */
