// Internal declarations shared by the translation units of libpt.so.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda.h>

#include <atomic>
#include <cstdint>
#include <cstdio>
#include <deque>
#include <unordered_map>
#include <vector>

#include "pt.h"

namespace pt {

constexpr int kStatusWords = 16;          // device status word block (int32 each)
constexpr int kSsqTile = 64;              // columns covered by one partial sum of squares
constexpr int kMaxSplits = 16;            // upper bound of KV key ranges per sequence in decode

// Location codes written next to PT_ERR_DEVICE_* in the status block.
enum : int {
    LOC_ROPE_PAGE = 1, LOC_ATTN_PAGE = 2, LOC_GEMM_TMA_WAIT = 3, LOC_GEMM_MMA_WAIT = 4,
    LOC_GEMM_EPI_WAIT = 5, LOC_GEMM_EMPTY_WAIT = 6, LOC_DECODE_PAGE = 7, LOC_FLASH_PAGE = 8,
    LOC_GEMM_ACC_WAIT = 9,
    LOC_FLASH_KEMPTY = 10, LOC_FLASH_VEMPTY = 11, LOC_FLASH_VRAW = 12, LOC_FLASH_KFULL = 13, LOC_FLASH_QFULL = 14,
    LOC_EMBED_TOKEN = 19, LOC_SELFTEST_WAIT = 20,
    LOC_FLASH_PFULL = 15, LOC_FLASH_VFULL = 16, LOC_FLASH_SFULL = 17, LOC_FLASH_OREADY = 18,
};

extern std::atomic<long long> g_launches;
void set_error(const char* fmt, ...);

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Seq {
    std::vector<int32_t> pages;
    int32_t len = 0;
};

// Tensor maps of one layer's packed weights: [qkv, o, gu, d][bn 64, 128, 256][k-blocks per copy 1, 2, 4];
// combinations the GEMM launcher never picks stay unset.
struct WMaps { CUtensorMap m[4][3][3]; };

// Per-device caches (function attributes, SM counts, symbol addresses) are indexed by the current device.
constexpr int kMaxDevices = 64;
inline int current_device() {
    int d = 0;
    if (cudaGetDevice(&d) != cudaSuccess || d < 0 || d >= kMaxDevices) d = 0;
    return d;
}

}  // namespace pt

struct pt_model {
    pt_config cfg;
    int dh, G, QD, KVD, Nqkv;             // head_dim, heads/kv_heads, nq*dh, nkv*dh, QD+2*KVD
    int E, Ftot;                          // experts of a PT-MoE layer (0: plain feed-forward) and the packed width max(E, 1) * ffn
    size_t esz;                           // bytes per element of the model dtype
    bool tc;                              // bf16 tensor-core path (else SIMT)
    // byte offsets inside the bound weight buffer; matrices are [L][T][rows][cols]
    size_t off_wqkv, off_wo, off_wgu, off_wd, off_g1, off_g2, off_cos, off_sin, off_cs16, off_wr, off_status, total_bytes;
    char* wbuf = nullptr;
    char* lm_buf = nullptr;                // embedding table, LM head, final gain (pt_lm_bind)
    int lm_vocab = 0;
    int world_tracks = 0;                  // > 0: this model holds cfg.T of world_tracks tracks (pt_model_set_track_group)
    pt_allreduce_fn ar_fn = nullptr;
    void* ar_user = nullptr;
    // track groups: a side stream and an event (created on first use, destroyed with the model) on which the next
    // layer's first weights are pulled into L2 while the all-reduce of a track-sync runs on the call's stream
    cudaStream_t side_stream = nullptr;
    cudaEvent_t side_event = nullptr;
    int tap_layer = -2;
    float* tap_buf = nullptr;
    std::vector<char> meta_host;          // staging for the per-call metadata upload
    std::vector<pt::WMaps> wmaps;         // [L] tensor maps of the bound weights (tensor-core path)
    // optional per-kernel timing (pt_profile_enable)
    struct ProfEv { cudaEvent_t a, b; int cat; };
    uint32_t prof_mask = 0;               // bit c set: launches of category c are bracketed with events
    std::vector<ProfEv> prof_ev;
    size_t prof_used = 0;

    size_t wqkv_layer() const { return (size_t)cfg.T * Nqkv * cfg.hidden; }     // elements
    size_t wo_layer() const { return (size_t)cfg.T * cfg.hidden * QD; }
    size_t wgu_layer() const { return (size_t)cfg.T * 2 * Ftot * cfg.hidden; }
    size_t wd_layer() const { return (size_t)cfg.T * cfg.hidden * Ftot; }
    // PT-MoE: fp32 router [L][T][E][hidden]
    const float* router(int l) const { return (const float*)(wbuf + off_wr) + (size_t)l * cfg.T * E * cfg.hidden; }
    int* status() const { return (int*)(wbuf + off_status); }
    const float* gain(int which, int l) const {
        return (const float*)(wbuf + (which ? off_g2 : off_g1)) + (size_t)l * cfg.T * cfg.hidden;
    }
    const float* rope_cos() const { return (const float*)(wbuf + off_cos); }
    const float* rope_sin() const { return (const float*)(wbuf + off_sin); }
    const uint32_t* rope_cs16() const { return (const uint32_t*)(wbuf + off_cs16); }   // [max_pos][dh/2] (cos, sin) as fp16 pairs
};

struct pt_kv_cache {
    const pt_model* m;
    int32_t num_pages, ps;
    int32_t kv_dtype;                     // pt_kv_dtype
    size_t esz;                           // bytes per cached element: the model's, or 1 for E4M3 codes
    char* pool;
    float* scales;                        // E4M3: [T][L][page][K|V][kv_head][slot] behind the codes; else null
    size_t bytes;
    int64_t page_elems;                   // 2 * nkv * ps * dh
    int64_t slab_elems;                   // num_pages * page_elems : one (track, layer)
    int64_t slab_vecs() const { return slab_elems / m->dh; }   // cached vectors (= scales) of one (track, layer)
    std::deque<int32_t> free_list;
    std::unordered_map<int32_t, pt::Seq> seqs;
};

namespace pt {

// Per-call device metadata (lives at the head of the workspace).
struct Meta {
    const int64_t* row_kvoff;   // [M] element offset, inside a (track, layer) slab, of K head 0 of the row's slot
    const int32_t* row_pos;     // [M] absolute position of the row's token
    const int32_t* row_b;       // [M] batch row
    const int32_t* kvlen;       // [B] cached length including this call's tokens
    const int32_t* bt;          // [B][maxp] block table rows
    int32_t maxp;
    // E4M3 caches only
    const int64_t* row_stageoff;  // [M] row * head_dim: where the QKV epilogue puts the row's K head 0 in the staging area
    const int64_t* row_attnoff;   // [M] prefill: offset of the row's slot (K head 0) inside a track's slab of the attention copy
    const int32_t* bt_attn;       // [B][maxp_attn] 16-token pages of the attention copy
    const int32_t* ctx_start;     // [B] keys cached before the call (prefill)
    int32_t maxp_attn, attn_pages, max_start;
};

// PT-MoE with permuted tokens: R = moe_rows() rows per track, every (token, chosen expert) one row, experts in runs of
// 128-row tiles.
struct MoeWork {
    int32_t* pos;            // [T][M][E] row of (token, expert), -1 where the token did not choose the expert
    int32_t* tile_expert;    // [T][R / 128]
    __nv_bfloat16* xperm;    // [T][R][H] operand rows
    float* ssq_perm;         // [T][R][H / kSsqTile]
    float* gperm;            // [T][R] routing weight of the row
    __nv_bfloat16* zperm;    // [T][R][ffn]
    float* yperm;            // [T][R][H]
};

// Workspace carve-up for one call.
struct Work {
    Meta meta;
    float* hT;      // [T][M][H] per-track residual stream
    float* hS;      // [M][H] post-sync stream (read with track stride 0)
    void* a;        // [T][M][H] model dtype: normalised activations (SIMT) / gain-scaled bf16 stream (tc)
    void* qkv;      // [T][M][Nqkv]
    void* o;        // [T][M][QD]
    void* gu;       // [T][M][2F] (SIMT only)
    void* z;        // [T][M][F]
    float* ssq;     // [T][M][H/kSsqTile] partial sums of squares (tc)
    float* part;    // decode split-KV partials
    void* kv_stage; // E4M3 caches: [T][K|V][kv_head][M][dh] bf16, this call's K and V as projected
    MoeWork moe;    // PT-MoE, permuted-token path (prefill calls of 512 rows or more)
    float* gates;   // PT-MoE: [T][M][E] routing weights of the current layer (0 for the experts a token did not choose)
    void* attn_kv;  // E4M3 caches, prefill: [T][page][K|V][kv_head][16][dh] bf16 copy of code * scale of every key attended to
    size_t total;
};

struct Call {
    pt_model* m;
    pt_kv_cache* c;
    int B, S, M;
    const void* x;
    int64_t x_stride;
    float* out;
    Work w;
    cudaStream_t st;
    bool decode;
    // decode split plan (host): items of (b, first key, key count)
    int n_items, max_splits;
    const int32_t* items;     // device [n_items][4]: b, start, count, split index
    const int32_t* nsplit;    // device [B]
};

// Brackets one kernel launch with events when timing is on.
struct ProfScope {
    pt_model* m; cudaStream_t st; int idx = -1;
    ProfScope(pt_model* m_, cudaStream_t st_, int cat) : m(m_), st(st_) {
        if (!((m->prof_mask >> cat) & 1u)) return;
        if (m->prof_used == m->prof_ev.size()) {
            pt_model::ProfEv e{};
            if (cudaEventCreate(&e.a) != cudaSuccess || cudaEventCreate(&e.b) != cudaSuccess) return;
            m->prof_ev.push_back(e);
        }
        idx = (int)m->prof_used++;
        m->prof_ev[idx].cat = cat;
        cudaEventRecord(m->prof_ev[idx].a, st);
    }
    ~ProfScope() { if (idx >= 0) cudaEventRecord(m->prof_ev[idx].b, st); }
};

// Split-KV plan of a decode step (host): key ranges are whole pages, longest sequences first.
// items gets 4 ints per range (batch row, first key, key count, range index); nsplit one per row.
void plan_decode_splits(const int32_t* lens, int B, int ps, int64_t units, int32_t* items, int32_t* nsplit,
                        int* n_items, int* max_splits);

// pt_simt.cu
pt_status simt_forward(Call& k);
void launch_pack(const pt_model* m, int kind, const void* src, void* dst_matrix_base, cudaStream_t st, int expert = 0);

// pt_tc_moe.cu
bool moe_sparse_ok(const pt_model* m, int M, bool decode);
int64_t moe_rows(const pt_model* m, int64_t M);

// pt_tc.cu (bf16 tensor-core path)
pt_status tc_build_weight_maps(pt_model* m);
pt_status tc_forward(Call& k);

}  // namespace pt
