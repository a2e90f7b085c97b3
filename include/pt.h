/*
 * pt.h - C ABI of the Parallel Track (PT) transformer forward pass for one NVIDIA B200.
 *
 * A PT stack (Section 2.2 and Algorithm 1 of "Parallel Track Transformers: Enabling Fast GPU
 * Inference with Reduced Synchronization") is T independent transformer "tracks", each with
 * its own weights, that run side by side for D layers (one track block) and then meet at a
 * track-sync: h = all-reduce(h_1..h_T), after which every track continues from h.  There are
 * L/D sync points per forward pass, against 2L for tensor parallelism (Sections 2.1, 2.2).
 * On one GPU the tracks are a leading dimension of every kernel and the sync is a reduction
 * in device memory.
 *
 * Conventions
 *  - Every function returns a pt_status (PT_OK = 0) and never throws or aborts.  A failing
 *    call leaves its outputs untouched; pt_last_error() gives a message for the calling thread.
 *  - "device" pointers are CUDA device addresses on the current device, "host" pointers are
 *    ordinary process memory.  The library never allocates device memory: weights, KV pool,
 *    workspace, inputs and outputs are caller-owned buffers that the library only borrows.
 *  - Handles (pt_model, pt_kv_cache) are owned by the library and released by their
 *    destroy / free call.  A handle must not be used from two threads at once.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Compute calls
 *    are asynchronous on it; host arrays passed to them are consumed before the call returns.
 *  - Per-track quantities: hidden, heads, kv_heads and ffn are the sizes of ONE track
 *    (Table 1 lists heads as "total (per track)").
 *  - Layer recipe of a track layer (the workloads' "standard transformer layer"): pre-norm
 *    RMSNorm (eps inside the square root, gain after), rotary embedding on the pairs
 *    (j, j + head_dim/2) with angle pos * rope_base^(-2j/head_dim), causal softmax attention
 *    scaled by 1/sqrt(head_dim) where query head i reads KV head i / (heads/kv_heads),
 *    SwiGLU feed-forward silu(c Wg^T) * (c Wu^T) Wd^T, no biases; residual adds around both.
 */
#ifndef PT_H_
#define PT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PT_OK = 0,
    PT_ERR_INVALID_ARG = 1,      /* null pointer, negative size, index out of range            */
    PT_ERR_BAD_CONFIG = 2,       /* L % D != 0, hidden % heads != 0, heads % kv_heads != 0 ... */
    PT_ERR_UNSUPPORTED = 3,      /* valid architecture the library has no kernel for          */
    PT_ERR_BUFFER_TOO_SMALL = 4, /* caller buffer smaller than the matching *_bytes query      */
    PT_ERR_CACHE_FULL = 5,       /* no free page left                                          */
    PT_ERR_MISALIGNED = 6,       /* device pointer not aligned as documented                   */
    PT_ERR_CUDA = 7,             /* a CUDA runtime / driver call failed                        */
    PT_ERR_DEVICE_BOUNDS = 8,    /* a kernel saw an index outside its buffers and skipped it   */
    PT_ERR_DEVICE_TIMEOUT = 9,   /* a bounded wait inside a kernel ran out                     */
    PT_ERR_STATE = 10            /* call order: weights not bound, sequence unknown ...        */
} pt_status;

typedef enum { PT_F32 = 0, PT_BF16 = 1 } pt_dtype;

/* Storage format of the KV cache.  PT_KV_MODEL keeps K and V in the model dtype.  PT_KV_E4M3 (bf16 models
 * on the tensor-core path, head_dim 128, pages of a multiple of 16 tokens) halves the cache: every cached
 * vector (one token, one KV head, K or V) is stored as head_dim E4M3 codes (1 sign, 4 exponent bits with
 * bias 7, 3 mantissa bits; largest value 448) and one fp32 scale, the smallest power of two s (not below
 * 2^-100) with max|v| / s <= 448 (1 for an all-zero vector); a code is v / s rounded to nearest even,
 * saturating.  Attention reads code * s.  The paper has no cache and no such format: it is this library's
 * own, there so that the ragged decode workload fits one device whole. */
typedef enum { PT_KV_MODEL = 0, PT_KV_E4M3 = 1 } pt_kv_dtype;

typedef enum {
    PT_WQ = 0, PT_WK = 1, PT_WV = 2, PT_WO = 3, PT_WG = 4, PT_WU = 5, PT_WD = 6,
    PT_G1 = 7, /* RMSNorm gain before attention */
    PT_G2 = 8, /* RMSNorm gain before the feed-forward */
    PT_WR = 9  /* router of a PT-MoE layer: [experts][hidden], always fp32 */
} pt_weight_kind;

/* Architecture of a PT stack: Algorithm 1's n (= T), L, D; heads per track as in Table 1. */
typedef struct {
    int32_t T;          /* tracks                                                     */
    int32_t D;          /* track-block depth: a sync after every D layers             */
    int32_t L;          /* layers per track; must be a multiple of D                  */
    int32_t hidden;     /* per-track model width H                                    */
    int32_t heads;      /* query heads per track; head_dim = hidden / heads           */
    int32_t kv_heads;   /* KV heads per track; must divide heads                      */
    int32_t ffn;        /* per-track SwiGLU width F                                   */
    float rope_base;    /* e.g. 10000                                                 */
    float rms_eps;      /* e.g. 1e-6                                                  */
    int32_t dtype;      /* pt_dtype of weights, inputs and the KV cache; accumulation,
                           the residual stream and the output are always fp32         */
    int32_t sync_op;    /* 0 = SUM (the all-reduce of Algorithm 1), 1 = MEAN          */
    int32_t max_pos;    /* positions 0..max_pos-1 are valid (size of the rotary table)*/
    int32_t flags;      /* bit 0: run the plain SIMT kernels even for bf16 (diagnostic
                           cross-check; the fp32 dtype always uses them)
                           bit 1: prefill attention on the warp-level mma.sync kernel
                           instead of the tensor-memory (tcgen05) one (diagnostic; that
                           kernel also serves head_dim 32 and 8-token pages)
                           bit 2: decode attention of an E4M3 cache on the warp-level mma.sync
                           kernel (codes converted to f16) instead of the tcgen05 one
                           (diagnostic)                                                  */
    int32_t experts;    /* 0: the plain SwiGLU feed-forward.  > 0 (at most 16; bf16 models on the
                           tensor-core path): PT-MoE - the feed-forward of every track and layer is a
                           mixture of `experts` SwiGLU experts of width ffn each.  The paper names the
                           combination in one sentence (Section 2.2, "Contrast with MoE": an MoE layer
                           inside each track) and defines nothing else; this library's definition: router
                           logits = rmsnorm(h; g2) Wr^T, the top_k largest logits (the lower index wins a
                           tie) get softmax weights among themselves, the layer's output is the weighted
                           sum of the chosen experts' outputs.  Prefill calls of 512 rows or more copy
                           every token's row to the row groups of the experts it chose and evaluate only
                           those (a grouped GEMM over (track, expert)); smaller calls and decode steps
                           evaluate every expert for every token and weight afterwards (unchosen experts by
                           zero) - the same result, and a decode batch streams every expert's weights
                           either way                                                                */
    int32_t top_k;      /* experts chosen per token, 1 .. experts (0 with experts == 0)              */
} pt_config;

typedef struct pt_model pt_model;
typedef struct pt_kv_cache pt_kv_cache;

/* ---- model ------------------------------------------------------------------------------- */

/* Validate `cfg` (host) and create a model handle (host).  No device work.
 * PT_ERR_BAD_CONFIG: T, D, L < 1; L % D != 0 (Algorithm 1 would drop the trailing layers);
 * hidden % heads; heads % kv_heads; odd head_dim; max_pos < 1.
 * PT_ERR_UNSUPPORTED: head_dim not in {32, 64, 128}; for bf16, hidden or ffn not a multiple
 * of 16. */
pt_status pt_model_create(const pt_config* cfg, pt_model** out);
void pt_model_destroy(pt_model* m);

/* Bytes of the caller-owned device buffer that holds the packed weights, the rotary table
 * and the device status word. */
pt_status pt_model_weight_bytes(const pt_model* m, size_t* bytes);

/* Borrow `dev_buf` (device, 256-byte aligned, >= pt_model_weight_bytes) for the model's
 * lifetime.  Builds the rotary table on the host in double precision and uploads it,
 * zeroes the gains' region and the status word; blocks until done. */
pt_status pt_model_bind_weights(pt_model* m, void* dev_buf, size_t bytes);

/* Copy one weight tensor of (track, layer) into the packed buffer.  `dev_src` (device) is
 * [out, in] row-major in the model dtype (y = x W^T); gains are [hidden] in fp32.
 * Asynchronous on `stream`.  With experts > 0, PT_WR takes the router [experts][hidden] in fp32 and
 * PT_WG / PT_WU / PT_WD go through pt_model_set_expert_weight instead. */
pt_status pt_model_set_weight(pt_model* m, int32_t track, int32_t layer, int32_t kind,
                              const void* dev_src, void* stream);
/* The same for one expert's PT_WG, PT_WU ([ffn, hidden]) or PT_WD ([hidden, ffn]) of a PT-MoE model. */
pt_status pt_model_set_expert_weight(pt_model* m, int32_t track, int32_t layer, int32_t expert, int32_t kind,
                                     const void* dev_src, void* stream);

/* Number of track-sync points of one forward pass: L / D (Section 2.2). */
int32_t pt_sync_count(const pt_model* m);

/* ---- paged KV cache ------------------------------------------------------------------------
 * Pool layout (elements of the model dtype): [T][L][page][K|V][kv_head][slot][head_dim].
 * One page id serves every (track, layer) slab.  K is stored after the rotary embedding, V as
 * projected.  The host-side allocator hands out pages from the front of a free list that
 * starts as 0, 1, 2, ...; released pages go to the back in block-table order. */

pt_status pt_kv_cache_bytes(const pt_model* m, int32_t num_pages, int32_t page_size, size_t* bytes);
/* The same for a cache of the given pt_kv_dtype.  An E4M3 pool is the codes, laid out as above with one byte
 * per element, followed (256-byte aligned) by the fp32 scales [T][L][page][K|V][kv_head][slot]. */
pt_status pt_kv_cache_bytes_ex(const pt_model* m, int32_t num_pages, int32_t page_size, int32_t kv_dtype, size_t* bytes);

/* Wrap the caller-owned device buffer `dev_pool` (256-byte aligned) as a cache of `num_pages`
 * pages of `page_size` tokens (16 is the tuned size; any multiple of 8 up to 64 is accepted).
 * Host only: the pool's contents are left as they are. */
pt_status pt_kv_cache_alloc(const pt_model* m, int32_t num_pages, int32_t page_size,
                            void* dev_pool, size_t bytes, pt_kv_cache** out);
pt_status pt_kv_cache_alloc_ex(const pt_model* m, int32_t num_pages, int32_t page_size, int32_t kv_dtype,
                               void* dev_pool, size_t bytes, pt_kv_cache** out);
void pt_kv_cache_free(pt_kv_cache* c);

/* Replace the free list by `order` (host, a permutation of 0..num_pages-1).  Only while no
 * page is in use (PT_ERR_STATE otherwise). */
pt_status pt_kv_set_free_list(pt_kv_cache* c, const int32_t* order, int32_t n);

/* Make sure sequence `seq` (any non-negative id) owns pages for positions < new_len.
 * PT_ERR_CACHE_FULL leaves the cache unchanged. */
pt_status pt_kv_seq_reserve(pt_kv_cache* c, int32_t seq, int32_t new_len);
/* Give a sequence's pages back and forget it. */
pt_status pt_kv_seq_release(pt_kv_cache* c, int32_t seq);
/* Tokens currently cached for `seq` (0 for an unknown sequence). */
pt_status pt_kv_seq_len(const pt_kv_cache* c, int32_t seq, int32_t* len);
/* Truncate a sequence to `len` <= its current length (pages are kept). */
pt_status pt_kv_seq_truncate(pt_kv_cache* c, int32_t seq, int32_t len);
/* Copy the block table of `seq` into `pages` (host, capacity `cap`); *n = pages owned. */
pt_status pt_kv_block_table(const pt_kv_cache* c, int32_t seq, int32_t* pages, int32_t cap, int32_t* n);
/* Element offset inside the pool of the head_dim values cached for (track, layer, seq, pos,
 * kv = 0 for K / 1 for V, kv_head).  The position must lie inside the reserved pages. */
pt_status pt_kv_slot(const pt_kv_cache* c, int32_t track, int32_t layer, int32_t seq, int32_t pos,
                     int32_t kv, int32_t kv_head, int64_t* elem_offset);

/* E4M3 caches: byte offset, from the start of the pool, of the fp32 scale of the vector that pt_kv_slot
 * addresses (there the offset counts one-byte codes).  PT_ERR_STATE for a cache in the model dtype. */
pt_status pt_kv_scale_slot(const pt_kv_cache* c, int32_t track, int32_t layer, int32_t seq, int32_t pos,
                           int32_t kv, int32_t kv_head, int64_t* byte_offset);

/* ---- forward pass --------------------------------------------------------------------------- */

/* Bytes of workspace (device) that pt_prefill / pt_decode_step need for up to `max_tokens`
 * = B*S tokens and `max_batch` sequences per call. */
pt_status pt_workspace_bytes(const pt_model* m, int64_t max_tokens, int32_t max_batch,
                             int32_t page_size, size_t* bytes);
/* The same for calls on a cache of the given pt_kv_dtype.  With an E4M3 cache the projections' K and V pass
 * through a bf16 staging area on their way into the cache, and a prefill call attends to a bf16 copy of
 * code * scale of every key its sequences hold: `max_context` bounds, over one prefill call, the sum over its
 * sequences of the cached length after the call, each rounded up to 16 (0 = prefill calls only ever start
 * from empty sequences: max_tokens + 16 * max_batch is used).  Decode calls need no such copy. */
pt_status pt_workspace_bytes_ex(const pt_model* m, int64_t max_tokens, int32_t max_batch, int32_t page_size,
                                int32_t kv_dtype, int64_t max_context, size_t* bytes);

/* Algorithm 1 over B sequences of S new tokens each.
 *   x         device, 16-byte aligned, model dtype, [T][B][S][hidden]; track t starts at
 *             x + t*x_track_stride elements (0 = every track starts from the same x,
 *             Algorithm 1's literal case)
 *   seq_ids   host, int32[B], distinct; the S tokens of row b are appended to sequence
 *             seq_ids[b] at positions len..len+S-1 (pages are reserved by the call) and attend
 *             to everything cached for it, themselves included causally
 *   out_h     device, 32-byte aligned, fp32 [B][S][hidden]: the activation h after the last sync
 *   workspace device, 256-byte aligned, >= pt_workspace_bytes(B*S, B, page_size)
 *             (pt_workspace_bytes_ex for an E4M3 cache)
 * On success the sequences' lengths grow by S.  Errors: PT_ERR_CACHE_FULL,
 * PT_ERR_BUFFER_TOO_SMALL, PT_ERR_INVALID_ARG (position >= max_pos, duplicate ids),
 * PT_ERR_STATE (weights not bound), PT_ERR_CUDA.  Kernel-side faults are reported through
 * pt_device_status, not here. */
pt_status pt_prefill(pt_model* m, pt_kv_cache* c, const void* x, int64_t x_track_stride,
                     int32_t B, int32_t S, const int32_t* seq_ids, void* out_h,
                     void* workspace, size_t ws_bytes, void* stream);

/* One new token per sequence: x [T][B][hidden] -> out_h fp32 [B][hidden].  The token of row b
 * is cached at position len(seq_ids[b]) and attends positions 0..len; same rules as
 * pt_prefill with S = 1, with attention split over the KV length. */
pt_status pt_decode_step(pt_model* m, pt_kv_cache* c, const void* x, int64_t x_track_stride,
                         int32_t B, const int32_t* seq_ids, void* out_h,
                         void* workspace, size_t ws_bytes, void* stream);

/* ---- ends of the model (bf16 models) -----------------------------------------------------------
 * Algorithm 1 takes the embedding output x and returns h; the paper's latency tables (time to first
 * token, time per output token: Tables 6-10) need the two ends it leaves to "standard" practice.
 * Conventions of this library: one embedding table [vocab][hidden] shared by every track (Algorithm 1,
 * "Set h_i = x"), a final RMSNorm with its own gain, an untied LM head [vocab][hidden], greedy choice =
 * lowest index among the largest logits.  vocab must be a multiple of 16. */

/* Bytes of, and binding of, the caller-owned device buffer (256-byte aligned) that holds the embedding
 * table, the LM head (both in the model dtype) and the final gain (fp32). */
pt_status pt_lm_bytes(const pt_model* m, int32_t vocab, size_t* bytes);
pt_status pt_lm_bind(pt_model* m, int32_t vocab, void* dev_buf, size_t bytes);
/* Copy one of them from `dev_src` (device, row-major): kind 0 = embedding table, 1 = LM head,
 * 2 = final gain [hidden] fp32. */
pt_status pt_lm_set(pt_model* m, int32_t kind, const void* dev_src, void* stream);

/* x_out[r][:] = table[dev_tokens[r]][:] for r < n (device int32 ids; x_out device, 16-byte aligned,
 * [n][hidden]).  Pass x_out to pt_prefill / pt_decode_step with x_track_stride = 0.  An id outside
 * [0, vocab) is reported through pt_device_status (PT_ERR_DEVICE_BOUNDS) and read as id 0. */
pt_status pt_embed(pt_model* m, const int32_t* dev_tokens, int64_t n, void* x_out, void* stream);

/* logits[r][:] = rmsnorm(h_r; final gain) . head^T for the n rows h_r = h + r*row_stride (fp32, device,
 * 16-byte aligned; row_stride in elements, a multiple of 4 - use S*hidden with h pointing at the last
 * position to take one row per sequence of a prefill output).  logits: device fp32 [n][vocab];
 * next_token (device int32 [n], may be NULL) receives the greedy choice; workspace: device, 256-byte
 * aligned, >= pt_lm_workspace_bytes(n). */
pt_status pt_lm_workspace_bytes(const pt_model* m, int64_t n, size_t* bytes);
pt_status pt_lm_head(pt_model* m, const float* h, int64_t row_stride, int64_t n, float* logits, int32_t* next_token,
                     void* workspace, size_t ws_bytes, void* stream);

/* Greedy generation for B sequences: embed and prefill the prompts (dev_prompt: device int32 [B][S]),
 * take each sequence's next token from its last position, then one decode step per further token, n_new
 * tokens in all.  Token ids never leave the device, so the whole loop is asynchronous on `stream`.
 *   dev_tokens_out  device int32 [B][n_new]
 *   dev_logits_out  device fp32 [B][n_new][vocab] or NULL: the logits each token was chosen from
 *   workspace       device, 256-byte aligned, >= pt_generate_workspace_bytes(B, S, page_size)
 * The sequences seq_ids[b] grow by S + n_new - 1 positions (the last token is not fed back). */
pt_status pt_generate_workspace_bytes(const pt_model* m, int32_t B, int32_t S, int32_t page_size, size_t* bytes);
pt_status pt_generate(pt_model* m, pt_kv_cache* c, const int32_t* dev_prompt, int32_t B, int32_t S, int32_t n_new,
                      const int32_t* seq_ids, int32_t* dev_tokens_out, float* dev_logits_out,
                      void* workspace, size_t ws_bytes, void* stream);

/* ---- track parallelism across GPUs ---------------------------------------------------------------
 * The paper's deployment (Sections 2.2 and 3.3): each GPU holds some of the tracks and the track-sync is
 * one all-reduce per track block, L/D per forward against tensor parallelism's 2L.  A model created
 * with cfg.T = the tracks of THIS rank can be told that it is part of a larger stack of `world_tracks`
 * tracks; at every sync it then sums its own tracks into one fp32 [tokens][hidden] buffer, calls `fn`
 * once, and continues from the result.  `fn(user, dev_buf, count, stream)` must replace the `count`
 * fp32 values at `dev_buf` (device) by their sum over all ranks, enqueued on `stream` (e.g. an NCCL
 * all-reduce), and return 0; any other return value fails the forward call with PT_ERR_CUDA.  With
 * sync_op = MEAN the mean is taken over world_tracks.  Every rank passes the same batch; x holds the
 * rank's own tracks.  While `fn`'s work runs on `stream`, the library pulls the weights of the next layer's
 * first projection into L2 on a stream of its own (created on first use, joined into `stream` before the
 * forward call's work on it ends), so that the next track block does not start from HBM latency.  fn == NULL or world_tracks == 0 returns the model to the single-GPU schedule.
 * bf16 models on the tensor-core path only. */
typedef int32_t (*pt_allreduce_fn)(void* user, void* dev_buf, int64_t count, void* stream);
pt_status pt_model_set_track_group(pt_model* m, int32_t world_tracks, pt_allreduce_fn fn, void* user);

/* Debug tap.  `dev_buf` (device, fp32) receives the residual stream of the following forward
 * calls: for each tapped layer two [T][tokens][hidden] blocks, the first after the attention
 * residual add, the second after the whole layer (after the sync when the layer closes a
 * track block, in which case all T slices are equal).  layer >= 0 taps that layer only
 * (buffer holds 2 blocks), layer == -1 taps all L layers ([L][2][T][tokens][hidden]),
 * dev_buf == NULL switches the tap off. */
pt_status pt_set_debug_tap(pt_model* m, int32_t layer, void* dev_buf);

/* Wait for `stream`, read and clear the device status word: *code = PT_OK,
 * PT_ERR_DEVICE_BOUNDS or PT_ERR_DEVICE_TIMEOUT; *detail (may be NULL) = a kernel-specific
 * location code. */
pt_status pt_device_status(pt_model* m, void* stream, int32_t* code, int32_t* detail);

/* Kernel timing for benchmarks.  With timing on, the bf16 forward calls bracket every kernel
 * with CUDA events on the call's stream.  pt_profile_read waits for those events, ADDS device
 * milliseconds and launch counts per category into ms[] and launches[] (host, PT_PROF_CATEGORIES
 * entries each) and forgets the events.  Categories: 0 attention, 1 QKV GEMM, 2 output-projection
 * GEMM, 3 gate/up GEMM, 4 down GEMM, 5 down GEMM with track-sync, 6 everything else.
 * on = 0: off; on = 1: every category; any other value: bit (c + 1) selects category c (e.g.
 * on = 2 times the attention launches only, which keeps the cost of the events themselves -
 * about 2 us per bracketed launch - out of a measurement of the whole step). */
#define PT_PROF_CATEGORIES 7
pt_status pt_profile_enable(pt_model* m, int32_t on);
pt_status pt_profile_read(pt_model* m, float* ms, int64_t* launches);

/* Kernels launched by this library since the process started (all models). */
int64_t pt_launch_count(void);

/* Message of the last failing call on this thread ("" if none). */
const char* pt_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* PT_H_ */
