// Declarations of the bf16 tensor-core path (tcgen05 GEMMs, flash prefill attention, split-KV
// decode attention).
#pragma once
#include <algorithm>
#include <utility>
#include "pt_internal.h"

namespace pt {

enum { EPI_PLAIN = 0, EPI_QKV = 1, EPI_SWIGLU = 2, EPI_RESID = 3 };

// Arguments of one track-grouped GEMM launch: C[t][M][N] = A[t][M][K] * W[t][N][K]^T.
struct GemmP {
    int M, N, K;            // per-track problem
    int T;                  // tracks folded into the grid
    int kt;                 // tracks folded into the K loop (1, or all tracks for the sync GEMM with T = 1)
    int tiles_m, tiles_n;   // filled by the launcher
    int pair;               // 1: CTA-pair kernel (256 x 256 tiles, tb with 128-row boxes); see gemm_pair_ok
    int kps;                // k-blocks per ring stage (1, or 2 / 4 with a 4-D W map from make_w_map; see gemm_kps)
    // filled by the launcher:
    uint32_t a_tx, w_tx;    // bytes a stage's A copy and its W copy deliver
    uint32_t a_bytes;       // shared-memory bytes reserved per k-block of A; the stage's W part follows its kps A pieces
    uint32_t w_kb_bytes;    // shared-memory bytes one k-block of W takes
    int stages;             // ring depth
    int w_static;           // W is written by no kernel of the stream: its first tiles may be fetched before grid_dep_wait()
    // grouped rows (PT-MoE with permuted tokens; one-CTA kernel with kps = 1 only): row tile mt of track t multiplies with
    // expert tile_expert[t * tiles_m + mt]'s weights, found w_row_per_expert rows / w_k_per_expert columns further in W
    const int32_t* tile_expert; int w_row_per_expert, w_k_per_expert;
    int* status;
    // RMSNorm applied as a per-row scale: rinv = rsqrt(sum(ssq_in[row][:]) / K + eps)
    const float* ssq_in; size_t ssq_in_tstride; int ssq_tiles; float eps;
    // EPI_PLAIN
    float* c_out;
    // EPI_QKV
    __nv_bfloat16* q_out;   // [T][M][nq*dh]
    __nv_bfloat16* pool_l;  // KV pool slab of this layer, track 0
    int64_t pool_tstride, slab_elems;
    const int64_t* row_kvoff; const int32_t* row_pos;
    const float* cs; const float* sn;
    const uint32_t* cs16;   // [max_pos][dh/2] (cos, sin) fp16 pairs
    int nq, nkv, dh, ps;
    // EPI_SWIGLU
    __nv_bfloat16* z_out;   // [T][M][N/2]
    const float* gates;     // PT-MoE: [T][M][n_experts] weights; accumulator columns [e * expert_cols, (e + 1) * expert_cols) belong to expert e
    int n_experts, expert_cols;
    // EPI_RESID
    const float* h_in; size_t h_in_tstride; int n_sum; float scale;
    float* h_out; size_t h_out_tstride;
    __nv_bfloat16* hb_out;  // [T][M][N] gain-scaled copy for the next GEMM (may be null)
    const float* gain;      // [T][N] gains of the next RMSNorm
    int n_out;              // tracks that receive hb_out (1 = own track, T = all after a sync)
    float* ssq_out; size_t ssq_out_tstride; int ssq_out_tiles;
};

// Arguments shared by the attention kernels.
struct AttnP {
    const __nv_bfloat16* q;        // [T][M][nq*dh]
    const __nv_bfloat16* pool_l;   // KV slab of this layer, track 0
    int64_t pool_tstride;
    __nv_bfloat16* o;              // [T][M][nq*dh]
    const int32_t* bt; int maxp;
    const int32_t* kvlen;          // [B] keys cached per sequence, this call's tokens included
    int B, S, M, nq, nkv, ps, num_pages;
    float scale_log2;              // log2(e) / sqrt(dh)
    int* status;
    // decode
    const int32_t* items; const int32_t* nsplit; float* part; int max_splits;
};

// Programmatic dependent launch.  A kernel launched with launch_dependent() may start while the
// kernel before it in the stream is still running: its blocks get free SMs as the earlier kernel's
// blocks retire, and run until grid_dep_wait(), which returns once the earlier kernel has completed
// and its writes are visible.  Before that wait a kernel may only touch memory that no kernel of the
// stream writes (weights); everything else, reads and writes, comes after it.  Every block calls
// grid_dep_wait() and only then grid_dep_launch(), so at most two kernels overlap and a kernel past
// its wait sees the results of every launch before it.  In a kernel launched the ordinary way both
// calls do nothing.
#ifdef __CUDACC__
// Every wait in these kernels is a loop of mbarrier.try_wait (which itself suspends the thread for a hardware-chosen
// while) with an iteration limit; the iteration limit alone does not bound the time, so each loop also gives up once
// WaitClock::expired() says that more than kWaitLimitNs have passed since its first slow poll.  A wait that gives up
// records PT_ERR_DEVICE_TIMEOUT and the kernel winds down.
constexpr unsigned long long kWaitLimitNs = 2000000000ull;        // 2 s: far beyond any wait of a healthy launch
struct WaitClock {
    unsigned long long t0 = 0;
    __device__ __forceinline__ static unsigned long long now() { unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
    // call every few hundred polls
    __device__ __forceinline__ bool expired(unsigned long long limit_ns = kWaitLimitNs) {
        const unsigned long long t = now();
        if (t0 == 0) { t0 = t; return false; }
        return t - t0 > limit_ns;
    }
};
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}
#endif

pt_status launch_flash_prefill_p(const AttnP& p, int T, int dh, bool legacy, cudaStream_t st);
pt_status launch_decode_attn_p(const AttnP& p, int T, int dh, int n_items, int max_splits, cudaStream_t st);

// cuTensorMapEncodeTiled, found through the runtime's driver entry point lookup (the library does not link libcuda);
// null when the driver does not offer it
typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeFn get_encode();
pt_status make_map_bf16(CUtensorMap* out, const void* base, int64_t k, int64_t rows, int64_t tracks, int box_rows);
pt_status make_map_bf16_strided(CUtensorMap* out, const void* base, int64_t k, int64_t rows, int64_t tracks,
                                int64_t track_stride_bytes, int box_rows);
int gemm_bn(int N, int M, int T, int epi);
// k-blocks per ring stage for a launch of M rows: more than one when the rows are few, so that a copy of W is 16-32 KB
int gemm_kps(int bn, int M, int K, int kt);
// whether a launch should use the CTA-pair kernel (then W's map is the one with 128-row boxes and kps = 1)
bool gemm_pair_ok(int bn, int M, int N, int T);
// tensor map of W [tracks][rows][k] for tiles of bn rows: 3-D (k, row, track) for kps = 1, else 4-D (64, row, k-block, track)
pt_status make_w_map(CUtensorMap* out, const void* base, int64_t k, int64_t rows, int64_t tracks, int bn, int kps);
// tensor map of A [tracks][rows][k] to go with it: 3-D with a box of min(rows, 128) rows for kps = 1, else 4-D with kps k-blocks per copy
pt_status make_a_map(CUtensorMap* out, const void* base, int64_t k, int64_t rows, int64_t tracks, int kps);
inline int bn_index(int bn) { return bn == 64 ? 0 : (bn == 128 ? 1 : 2); }
pt_status launch_gemm(int epi, int bn, const CUtensorMap& ta, const CUtensorMap& tb, GemmP p, cudaStream_t st);

// pt_simt.cu
void tap_copy(Call& k, int layer, int point, const float* src, size_t src_tstride);
void launch_simt_attn_bf16(Call& k, const __nv_bfloat16* q, int q_row_stride, const __nv_bfloat16* pool_l, __nv_bfloat16* o);

// pt_tc_gemm.cu: a one-CTA kernel that waits on an mbarrier nothing arrives at, with the kernels' own wait loop and a short limit
pt_status launch_wait_selftest(int* status, unsigned long long limit_ns, cudaStream_t st);

// pt_tc_flash.cu
bool flash_tc_supported(int dh, int ps);
pt_status launch_flash_prefill_tc(const AttnP& p, int T, int dh, cudaStream_t st);

// pt_tc_attn.cu
pt_status launch_flash_prefill(Call& k, const __nv_bfloat16* q, const __nv_bfloat16* pool_l, __nv_bfloat16* o);
pt_status launch_decode_attn(Call& k, const __nv_bfloat16* q, const __nv_bfloat16* pool_l, __nv_bfloat16* o);

// pt_tc_moe.cu: the feed-forward of a PT-MoE layer with permuted tokens, from the stream after the attention residual
// (h_in) to what the dense path's down GEMM leaves (h_out, the next operand and statistics, the track-sync when `sync`)
pt_status moe_sparse_ffn(Call& k, int l, bool sync, bool last, float sync_scale, const float* h_in, size_t h_in_tstride,
                         float* h_out, size_t h_out_tstride);

// merges the key ranges of a split decode attention (pt_tc_attn.cu)
pt_status launch_decode_combine(const AttnP& p, int T, int dh, cudaStream_t st);

// pt_tc_kv8.cu: the E4M3 storage format of the KV cache
pt_status launch_kv_quant(Call& k, int layer);
pt_status launch_kv_dequant_ctx(Call& k, int layer);
pt_status launch_flash_prefill_e4m3(Call& k, const __nv_bfloat16* q, __nv_bfloat16* o);
pt_status launch_decode_attn_e4m3(Call& k, const __nv_bfloat16* q, int layer, __nv_bfloat16* o);
// One layer's slab of an E4M3 cache as the decode kernels see it: codes [track][page][K|V][kv_head][slot][128] bytes
// and one fp32 scale per vector in the same order, tracks a fixed stride apart.
struct Kv8Slab {
    const uint8_t* codes_l; int64_t codes_tstride;        // bytes between tracks
    const float* scales_l; int64_t scales_tstride;        // floats between tracks
};
// p holds q, o, the block table, lengths, key ranges (items, nsplit), partial-result buffer, sizes and the status block
pt_status launch_decode_attn_e4m3_p(const AttnP& p, const Kv8Slab& slab, int T, int n_items, int max_splits, bool mma_sync, cudaStream_t st);
// pt_tc_kv8_dec.cu: the same on tcgen05 (the default; the mma.sync kernel serves config flag bit 2)
pt_status launch_decode_attn_e4m3_tc(const AttnP& p, const Kv8Slab& slab, int T, int n_items, int max_splits, cudaStream_t st);

}  // namespace pt
