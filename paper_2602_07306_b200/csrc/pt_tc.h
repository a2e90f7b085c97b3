// Declarations of the bf16 tensor-core path (tcgen05 GEMMs, flash prefill attention, split-KV
// decode attention).
#pragma once
#include <algorithm>
#include "pt_internal.h"

namespace pt {

enum { EPI_PLAIN = 0, EPI_QKV = 1, EPI_SWIGLU = 2, EPI_RESID = 3 };

// Arguments of one track-grouped GEMM launch: C[t][M][N] = A[t][M][K] * W[t][N][K]^T.
struct GemmP {
    int M, N, K;            // per-track problem
    int T;                  // tracks folded into the grid
    int kt;                 // tracks folded into the K loop (1, or all tracks for the sync GEMM with T = 1)
    int tiles_m, tiles_n;   // filled by the launcher
    uint32_t tx_bytes;      // bytes one stage's two TMA loads deliver (filled by the launcher)
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

pt_status launch_flash_prefill_p(const AttnP& p, int T, int dh, bool legacy, cudaStream_t st);
pt_status launch_decode_attn_p(const AttnP& p, int T, int dh, int n_items, int max_splits, cudaStream_t st);

pt_status make_map_bf16(CUtensorMap* out, const void* base, int64_t k, int64_t rows, int64_t tracks, int box_rows);
pt_status make_map_bf16_strided(CUtensorMap* out, const void* base, int64_t k, int64_t rows, int64_t tracks,
                                int64_t track_stride_bytes, int box_rows);
int gemm_bn(int N, int M, int T, int epi);
inline int bn_index(int bn) { return bn == 64 ? 0 : (bn == 128 ? 1 : 2); }
pt_status launch_gemm(int epi, int bn, const CUtensorMap& ta, const CUtensorMap& tb, GemmP p, cudaStream_t st);

// pt_simt.cu
void tap_copy(Call& k, int layer, int point, const float* src, size_t src_tstride);
void launch_simt_attn_bf16(Call& k, const __nv_bfloat16* q, int q_row_stride, const __nv_bfloat16* pool_l, __nv_bfloat16* o);

// pt_tc_flash.cu
bool flash_tc_supported(int dh, int ps);
pt_status launch_flash_prefill_tc(const AttnP& p, int T, int dh, cudaStream_t st);

// pt_tc_attn.cu
pt_status launch_flash_prefill(Call& k, const __nv_bfloat16* q, const __nv_bfloat16* pool_l, __nv_bfloat16* o);
pt_status launch_decode_attn(Call& k, const __nv_bfloat16* q, const __nv_bfloat16* pool_l, __nv_bfloat16* o);

}  // namespace pt
