/*
 * pt_kernels.h - kernel-level entry points of libpt.so, for unit parity tests and for timing a
 * single kernel of the PT forward pass in isolation.  Same conventions as pt.h: pt_status
 * returns, caller-owned device buffers, asynchronous on `stream`.
 */
#ifndef PT_KERNELS_H_
#define PT_KERNELS_H_

#include "pt.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Track-grouped GEMM, the contraction behind every projection of a track layer (the
 * "standard transformer layers" of Section 2.2, one set of weights per track):
 *   c[t][m][n] = sum_k a[t][m][k] * w[t][n][k]      t < T, m < M, n < N
 *   a  device bf16 [T][M][K] row-major        w  device bf16 [T][N][K] row-major
 *   c  device fp32 [T][M][N]                  status  device int32[16], zeroed by the caller
 * K must be a multiple of 8 and >= 64, N a multiple of 16; bn (N-tile width) is 64, 128 or 256, 0 lets
 * the library choose.  With fold_tracks != 0 the K loop runs over (track, k) and a single
 * c[0][m][n] = sum_t sum_k ... is produced: the contraction of the track-sync (Algorithm 1,
 * h = all-reduce(h_1..h_n)) fused into the last GEMM of a track block. */
pt_status pt_kernel_gemm_bf16(const void* a, const void* w, void* c, int32_t T, int32_t M, int32_t N,
                              int32_t K, int32_t bn, int32_t fold_tracks, void* status, void* stream);

/* Split-KV decode attention over the paged per-track KV cache (one new token per sequence, the
 * attention of a track layer during decode: every query head of every track attends to its KV
 * head's cached keys, tracks never read each other's cache between syncs - Section 2.2):
 *   out[t][b][h] = softmax_j( q[t][b][h] . K[t][b][h / G][j] / sqrt(dh) ) V[t][b][h / G][j],
 *   j < kv_len[b], G = nq / nkv.
 *   q, out        device bf16 [T][B][nq*dh]
 *   pool_l        device bf16: one layer's slabs, track t at pool_l + t*pool_track_stride elements,
 *                 each [num_pages][K|V][nkv][ps][dh]
 *   block_table   device int32 [B][maxp]: page of positions i*ps .. of sequence b
 *   kv_len        host int32 [B] (>= 1): keys to attend to
 *   scratch       device, 256-byte aligned, >= pt_kernel_decode_attn_scratch_bytes: holds the
 *                 split plan and the per-range partial results; contents need not be kept
 *   status        device int32[16], zeroed by the caller; PT_ERR_DEVICE_BOUNDS is recorded there
 *                 when a page id is outside [0, num_pages)
 * dh in {32, 64, 128}, nq/nkv <= 8.  Asynchronous on `stream`; kv_len is consumed before return. */
pt_status pt_kernel_decode_attn_scratch_bytes(int32_t T, int32_t B, int32_t nq, int32_t dh, size_t* bytes);
pt_status pt_kernel_decode_attn(const void* q, const void* pool_l, int64_t pool_track_stride,
                                const int32_t* block_table, int32_t maxp, const int32_t* kv_len,
                                int32_t T, int32_t B, int32_t nq, int32_t nkv, int32_t dh, int32_t ps,
                                int32_t num_pages, void* out, void* scratch, size_t scratch_bytes,
                                void* status, void* stream);

/* Causal prefill attention over the paged per-track KV cache (the attention of a track layer
 * when S new tokens per sequence are processed at once; every track attends only to its own
 * cache - Section 2.2).  The K and V of the new tokens must already be in the cache:
 *   out[t][b*S+s][h] = softmax_{j <= pos}( q[t][b*S+s][h] . K[t][b][h / G][j] / sqrt(dh) ) V[t][b][h / G][j],
 *   pos = kv_len[b] - S + s.
 *   q, out        device bf16 [T][B*S][nq*dh]
 *   pool_l, block_table, status   as for pt_kernel_decode_attn
 *   kv_len        DEVICE int32 [B]: keys cached per sequence, the S new ones included (>= S)
 *   impl          0 = tensor-memory kernel (tcgen05; head_dim 64 or 128, pages of a multiple of
 *                 16 tokens), 1 = warp-level mma.sync kernel (head_dim 32, 64, 128; any page size)
 * Asynchronous on `stream`; nothing is allocated. */
pt_status pt_kernel_prefill_attn(const void* q, const void* pool_l, int64_t pool_track_stride,
                                 const int32_t* block_table, int32_t maxp, const int32_t* kv_len,
                                 int32_t T, int32_t B, int32_t S, int32_t nq, int32_t nkv, int32_t dh, int32_t ps,
                                 int32_t num_pages, void* out, int32_t impl, void* status, void* stream);

/* The same decode attention for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of pt_kernel_decode_attn.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - a real-time or serving loop that
 * must not touch the allocator after start-up, or a host program that handed all device memory to
 * another component and has no pool of its own to carve a scratch buffer from.  Such a caller
 * passes only inputs and outputs; the split plan and the per-range partial results live in a fixed
 * array inside the library image (PT_STATIC_SCRATCH_BYTES, 8 MiB, resident on every GPU that loads
 * the library until the process exits).
 *
 *  - Arguments are those of pt_kernel_decode_attn without scratch / scratch_bytes; results are
 *    identical to it.
 *  - Problems whose scratch need (pt_kernel_decode_attn_scratch_bytes) exceeds
 *    PT_STATIC_SCRATCH_BYTES are refused with PT_ERR_BUFFER_TOO_SMALL and nothing is launched.
 *  - The first call on each device looks up the array's device address (no allocation, but a
 *    driver query): make that first call before any stream capture begins.
 *  - Like pt_kernel_decode_attn, every call builds the split plan on the host from kv_len and
 *    uploads it with an asynchronous copy on `stream`.
 *  - The entry point calls no cudaMalloc, cudaFree or any allocating library routine.
 *  - All calls on a device share the one array, which keeps whatever the previous call left.
 *    Nothing in it has to start at zero - every word a call reads it has written first - but
 *    two calls that overlap on the GPU (different streams, or concurrent host threads) race on
 *    it: serialise them on one stream. */
#define PT_STATIC_SCRATCH_BYTES (8u << 20)
pt_status pt_kernel_decode_attn_static(const void* q, const void* pool_l, int64_t pool_track_stride,
                                       const int32_t* block_table, int32_t maxp, const int32_t* kv_len,
                                       int32_t T, int32_t B, int32_t nq, int32_t nkv, int32_t dh, int32_t ps,
                                       int32_t num_pages, void* out, void* status, void* stream);

/* The quantiser of the E4M3 KV-cache format alone (pt_kv_dtype PT_KV_E4M3 in pt.h; the paper has no cache, the
 * format is this library's): for each of n vectors of 128 bf16 values
 *   scales[i] = the smallest power of two s >= 2^-100 with max|v| / s <= 448 (1 for an all-zero vector)
 *   codes[i][j] = v[j] / s rounded to the nearest E4M3 value, ties to even, saturating at +-448.
 *   src     device bf16 [n][128], 8-byte aligned        codes  device uint8 [n][128]
 *   scales  device fp32 [n]                             status device int32[16], zeroed by the caller
 * Asynchronous on `stream`; nothing is allocated. */
pt_status pt_kernel_kv_quant_e4m3(const void* src, void* codes, float* scales, int64_t n, void* status, void* stream);

/* Decode attention over one layer's slab of an E4M3 cache (pt_kv_dtype PT_KV_E4M3 in pt.h; Algorithm 1's attention of
 * a single-token step, Section 2.1, over the cache format this library defines): for every track, sequence b and
 * query head, softmax(q k^T / sqrt(128)) v over the kv_len[b] cached keys, where a cached vector is its 128 codes
 * times its scale.  Head size 128 only.
 *   q            device bf16 [T][B][nq * 128]
 *   codes_l      device uint8, one layer: [T] slabs codes_track_stride BYTES apart, each [num_pages][K|V][nkv][ps][128];
 *                128-byte aligned, stride a multiple of 128
 *   scales_l     device fp32, the same order without the last dimension; slabs scales_track_stride FLOATS apart
 *   block_table  device int32 [B][maxp]     kv_len  HOST int32 [B], each in [1, maxp * ps]
 *   ps           page size, a multiple of 16 up to 64;  nkv <= 8;  nq / nkv <= 8
 *   out          device bf16 [T][B][nq * 128]
 *   impl         0: the tcgen05 kernel (8-bit MMAs), 1: the mma.sync kernel (codes converted to f16)
 *   scratch      device, 256-byte aligned, at least pt_kernel_decode_attn_scratch_bytes(T, B, nq, 128) bytes
 *   status       device int32[16], zeroed by the caller
 * The key ranges are planned on the host and uploaded with an asynchronous copy on `stream`; everything else is
 * asynchronous on `stream` too.  Nothing is allocated.  Errors: PT_ERR_INVALID_ARG / UNSUPPORTED / MISALIGNED /
 * BUFFER_TOO_SMALL before anything is launched; a page number outside [0, num_pages) is reported in `status`. */
pt_status pt_kernel_decode_attn_e4m3(const void* q, const void* codes_l, int64_t codes_track_stride,
                                     const float* scales_l, int64_t scales_track_stride,
                                     const int32_t* block_table, int32_t maxp, const int32_t* kv_len,
                                     int32_t T, int32_t B, int32_t nq, int32_t nkv, int32_t ps,
                                     int32_t num_pages, void* out, int32_t impl, void* scratch, size_t scratch_bytes,
                                     void* status, void* stream);

/* ---- the bounded wait, exercised ------------------------------------------------------------
 * Every device-side wait of the library (an mbarrier of a TMA -> MMA -> epilogue pipeline) gives up
 * after a time limit (2 s of device time, whatever the iteration counts), records PT_ERR_DEVICE_TIMEOUT with
 * a location code in the status block and lets its kernel wind down, so that the context stays usable.
 * This entry point runs that same wait loop on a barrier at which nothing ever arrives, with the limit
 * given here, in a one-CTA kernel on `stream`:
 *   status    device, int32[16], zeroed by the caller; afterwards status[0] = PT_ERR_DEVICE_TIMEOUT and
 *             status[1] = 20 (the self-test's location code)
 *   limit_ns  how long the wait may last, 1 000 .. 1 000 000 000 (else PT_ERR_INVALID_ARG)
 * Returns PT_OK once the kernel is enqueued (PT_ERR_CUDA if the launch failed). */
pt_status pt_kernel_wait_selftest(void* status, uint64_t limit_ns, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* PT_KERNELS_H_ */
