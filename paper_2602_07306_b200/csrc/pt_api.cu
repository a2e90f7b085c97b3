// C ABI of libpt.so: configuration checks, packed-weight layout, the host page allocator,
// per-call metadata and dispatch to the kernel paths.  See include/pt.h for the contract.
#include <cmath>
#include <cstdarg>
#include <cstring>
#include <algorithm>
#include <new>
#include <unordered_set>

#include "pt_internal.h"

namespace pt {

std::atomic<long long> g_launches{0};
static thread_local char t_err[512] = "";

void set_error(const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(t_err, sizeof(t_err), fmt, ap);
    va_end(ap);
}

#define PT_FAIL(code, ...) do { pt::set_error(__VA_ARGS__); return (code); } while (0)
#define PT_CUDA(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) { \
    pt::set_error("%s failed: %s", #call, cudaGetErrorString(e_)); return PT_ERR_CUDA; } } while (0)


static size_t meta_bytes(int64_t M, int B, int maxp, bool fp8) {
    size_t b = 0;
    b += align_up((size_t)M * 8, 256);                 // row_kvoff
    b += align_up((size_t)M * 4, 256) * 2;             // row_pos, row_b
    b += align_up((size_t)B * 4, 256) * 2;             // kvlen, nsplit
    b += align_up((size_t)B * maxp * 4, 256);          // block table rows
    b += align_up((size_t)B * kMaxSplits * 16, 256);   // decode work items
    if (fp8) {
        b += align_up((size_t)M * 8, 256) * 2;         // row_stageoff, row_attnoff
        b += align_up((size_t)B * 4, 256);             // ctx_start
        b += align_up((size_t)B * ((size_t)maxp * 4 + 1) * 4, 256);   // pages of the attention copy (16 tokens each; cache pages hold up to 64)
    }
    return b;
}

// Carve the workspace; with base == nullptr only the size is computed.  fp8: the cache holds E4M3 codes;
// ctx_keys: keys of the attention copy a prefill call needs (0 for a decode call).
static size_t carve(const pt_model* m, int64_t M, int B, int maxp, bool fp8, int64_t ctx_keys, char* base, Work* w) {
    const pt_config& c = m->cfg;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes, 256); return base ? base + o : nullptr; };
    char* meta = (char*)take(meta_bytes(M, B, maxp, fp8));
    size_t TMH = (size_t)c.T * M * c.hidden;
    float* hT = (float*)take(TMH * 4);
    float* hS = (float*)take((size_t)M * c.hidden * 4);
    void* a = take(TMH * m->esz);
    void* qkv = take((size_t)c.T * M * m->Nqkv * m->esz);
    void* o = take((size_t)c.T * M * m->QD * m->esz);
    void* gu = m->tc ? nullptr : take((size_t)c.T * M * 2 * m->Ftot * m->esz);
    void* z = take((size_t)c.T * M * m->Ftot * m->esz);
    float* gates = m->E ? (float*)take((size_t)c.T * M * m->E * 4) : nullptr;
    MoeWork mw{};
    if (m->E && moe_sparse_ok(m, (int)std::min<int64_t>(M, 1 << 30), false)) {
        const size_t R = (size_t)moe_rows(m, M);
        mw.pos = (int32_t*)take((size_t)c.T * M * m->E * 4);
        mw.tile_expert = (int32_t*)take((size_t)c.T * (R / 128) * 4);
        mw.xperm = (__nv_bfloat16*)take((size_t)c.T * R * c.hidden * 2);
        mw.ssq_perm = (float*)take((size_t)c.T * R * ((c.hidden + kSsqTile - 1) / kSsqTile) * 4);
        mw.gperm = (float*)take((size_t)c.T * R * 4);
        mw.zperm = (__nv_bfloat16*)take((size_t)c.T * R * c.ffn * 2);
        mw.yperm = (float*)take((size_t)c.T * R * c.hidden * 4);
    }
    float* ssq = m->tc ? (float*)take((size_t)c.T * M * ((c.hidden + kSsqTile - 1) / kSsqTile) * 4) : nullptr;
    float* part = m->tc ? (float*)take((size_t)c.T * B * kMaxSplits * c.heads * (m->dh + 2) * 4) : nullptr;
    void* kv_stage = fp8 ? take((size_t)c.T * 2 * m->KVD * M * 2) : nullptr;
    void* attn_kv = fp8 && ctx_keys > 0 ? take((size_t)c.T * 2 * m->KVD * (size_t)ctx_keys * 2) : nullptr;
    if (w) {
        w->kv_stage = kv_stage; w->attn_kv = attn_kv; w->gates = gates; w->moe = mw;
        w->hT = hT; w->hS = hS; w->a = a; w->qkv = qkv; w->o = o; w->gu = gu; w->z = z;
        w->ssq = ssq; w->part = part; w->total = off;
        (void)meta;
    }
    return off;
}

void plan_decode_splits(const int32_t* lens, int B, int ps, int64_t units, int32_t* items, int32_t* nsplit,
                        int* n_items_out, int* max_splits_out) {
    int n_items = 0, max_splits = 1;
    int64_t total_keys = 0;
    for (int b = 0; b < B; ++b) total_keys += lens[b];
    // aim for >= 4 key ranges per SM over (tracks, kv heads, ranges); never split below 256 keys
    int64_t want_items = std::max<int64_t>(B, (148 * 4 + units - 1) / units);
    int64_t chunk = std::max<int64_t>(256, (total_keys + want_items - 1) / want_items);
    // With eight or more (sequence, track, KV head) triples per SM the machine is full without any split, and every
    // extra key range costs a CTA's start and drain (measured on 256 ragged sequences, 16 triples each: 0.80 -> 0.87
    // of the copy bandwidth in the 8-bit kernel, +2 % in the bf16 one): only sequences of more than twice the mean
    // length are split then.
    if ((int64_t)B * units >= 148 * 8) chunk *= 2;
    chunk = (chunk + ps - 1) / ps * ps;
    std::vector<int> order(B);
    for (int b = 0; b < B; ++b) order[b] = b;
    std::stable_sort(order.begin(), order.end(), [&](int a, int b2) { return lens[a] > lens[b2]; });
    for (int b : order) {
        int ns = (int)std::min<int64_t>(kMaxSplits, (lens[b] + chunk - 1) / chunk);
        ns = std::max(ns, 1);
        int64_t per = ((lens[b] + ns - 1) / ns + ps - 1) / ps * ps;
        per = std::max<int64_t>(per, ps);
        ns = (int)std::max<int64_t>(1, (lens[b] + per - 1) / per);
        nsplit[b] = ns;
        max_splits = std::max(max_splits, ns);
        for (int s2 = 0; s2 < ns; ++s2) {
            int32_t* it = items + (size_t)n_items * 4;
            it[0] = b; it[1] = (int32_t)(s2 * per);
            it[2] = (int32_t)std::min<int64_t>(per, lens[b] - s2 * per); it[3] = s2;
            ++n_items;
        }
    }
    *n_items_out = n_items;
    *max_splits_out = max_splits;
}

}  // namespace pt

using namespace pt;

extern "C" {

const char* pt_last_error(void) { return t_err; }
int64_t pt_launch_count(void) { return g_launches.load(); }

pt_status pt_model_create(const pt_config* cfg, pt_model** out) {
    if (!cfg || !out) PT_FAIL(PT_ERR_INVALID_ARG, "pt_model_create: null argument");
    const pt_config& c = *cfg;
    if (c.T < 1 || c.D < 1 || c.L < 1) PT_FAIL(PT_ERR_BAD_CONFIG, "T, D, L must be >= 1");
    if (c.L % c.D) PT_FAIL(PT_ERR_BAD_CONFIG, "L=%d is not a multiple of D=%d: the trailing layers would never reach a sync", c.L, c.D);
    if (c.hidden < 1 || c.heads < 1 || c.kv_heads < 1 || c.ffn < 1) PT_FAIL(PT_ERR_BAD_CONFIG, "sizes must be >= 1");
    if (c.hidden % c.heads) PT_FAIL(PT_ERR_BAD_CONFIG, "hidden %% heads != 0");
    if (c.heads % c.kv_heads) PT_FAIL(PT_ERR_BAD_CONFIG, "heads %% kv_heads != 0");
    int dh = c.hidden / c.heads;
    if (dh % 2) PT_FAIL(PT_ERR_BAD_CONFIG, "head_dim must be even");
    if (c.max_pos < 1) PT_FAIL(PT_ERR_BAD_CONFIG, "max_pos must be >= 1");
    if (!(c.rope_base > 0.f) || !(c.rms_eps >= 0.f)) PT_FAIL(PT_ERR_BAD_CONFIG, "rope_base must be > 0 and rms_eps >= 0");
    if (c.dtype != PT_F32 && c.dtype != PT_BF16) PT_FAIL(PT_ERR_BAD_CONFIG, "dtype must be PT_F32 or PT_BF16");
    if (c.sync_op != 0 && c.sync_op != 1) PT_FAIL(PT_ERR_BAD_CONFIG, "sync_op must be 0 (sum) or 1 (mean)");
    if (dh != 32 && dh != 64 && dh != 128) PT_FAIL(PT_ERR_UNSUPPORTED, "head_dim %d not in {32, 64, 128}", dh);
    if (c.ffn % 16) PT_FAIL(PT_ERR_UNSUPPORTED, "ffn must be a multiple of 16");
    if (c.hidden % 16) PT_FAIL(PT_ERR_UNSUPPORTED, "hidden must be a multiple of 16");
    if (c.heads / c.kv_heads > 8) PT_FAIL(PT_ERR_UNSUPPORTED, "more than 8 query heads per KV head");
    if (c.experts < 0 || (c.experts == 0 && c.top_k != 0) || (c.experts > 0 && (c.top_k < 1 || c.top_k > c.experts)))
        PT_FAIL(PT_ERR_BAD_CONFIG, "top_k must lie in [1, experts] (and be 0 without experts)");
    if (c.experts > 16) PT_FAIL(PT_ERR_UNSUPPORTED, "more than 16 experts");
    if (c.experts > 0 && (c.dtype != PT_BF16 || (c.flags & 1))) PT_FAIL(PT_ERR_UNSUPPORTED, "PT-MoE needs a bf16 model on the tensor-core path");
    pt_model* m = new (std::nothrow) pt_model();
    if (!m) PT_FAIL(PT_ERR_INVALID_ARG, "out of host memory");
    m->cfg = c;
    m->dh = dh;
    m->G = c.heads / c.kv_heads;
    m->QD = c.heads * dh;
    m->KVD = c.kv_heads * dh;
    m->Nqkv = m->QD + 2 * m->KVD;
    m->esz = c.dtype == PT_BF16 ? 2 : 4;
    m->tc = c.dtype == PT_BF16 && !(c.flags & 1);
    m->E = c.experts;
    m->Ftot = std::max(c.experts, 1) * c.ffn;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes, 256); return o; };
    m->off_wqkv = take(m->wqkv_layer() * c.L * m->esz);
    m->off_wo = take(m->wo_layer() * c.L * m->esz);
    m->off_wgu = take(m->wgu_layer() * c.L * m->esz);
    m->off_wd = take(m->wd_layer() * c.L * m->esz);
    m->off_g1 = take((size_t)c.L * c.T * c.hidden * 4);
    m->off_g2 = take((size_t)c.L * c.T * c.hidden * 4);
    m->off_cos = take((size_t)c.max_pos * (dh / 2) * 4);
    m->off_sin = take((size_t)c.max_pos * (dh / 2) * 4);
    m->off_cs16 = take((size_t)c.max_pos * (dh / 2) * 4);
    m->off_wr = take((size_t)c.L * c.T * m->E * c.hidden * 4);
    m->off_status = take(kStatusWords * 4);
    m->total_bytes = off;
    *out = m;
    return PT_OK;
}

void pt_model_destroy(pt_model* m) {
    if (!m) return;
    for (auto& e : m->prof_ev) { cudaEventDestroy(e.a); cudaEventDestroy(e.b); }
    if (m->side_event) cudaEventDestroy(m->side_event);
    if (m->side_stream) cudaStreamDestroy(m->side_stream);
    delete m;
}

pt_status pt_profile_enable(pt_model* m, int32_t on) {
    if (!m) PT_FAIL(PT_ERR_INVALID_ARG, "null argument");
    m->prof_mask = on == 1 ? 0xffffffffu : (on < 0 ? 0u : ((uint32_t)on >> 1));
    if (!on) m->prof_used = 0;
    return PT_OK;
}

pt_status pt_profile_read(pt_model* m, float* ms, int64_t* launches) {
    if (!m || !ms || !launches) PT_FAIL(PT_ERR_INVALID_ARG, "null argument");
    for (size_t i = 0; i < m->prof_used; ++i) {
        auto& e = m->prof_ev[i];
        PT_CUDA(cudaEventSynchronize(e.b));
        float t = 0.f;
        PT_CUDA(cudaEventElapsedTime(&t, e.a, e.b));
        if (e.cat >= 0 && e.cat < PT_PROF_CATEGORIES) { ms[e.cat] += t; launches[e.cat] += 1; }
    }
    m->prof_used = 0;
    return PT_OK;
}

pt_status pt_model_set_track_group(pt_model* m, int32_t world_tracks, pt_allreduce_fn fn, void* user) {
    if (!m) PT_FAIL(PT_ERR_INVALID_ARG, "null argument");
    if (!fn || world_tracks == 0) { m->world_tracks = 0; m->ar_fn = nullptr; m->ar_user = nullptr; return PT_OK; }
    if (!m->tc) PT_FAIL(PT_ERR_UNSUPPORTED, "track groups are built for bf16 models on the tensor-core path");
    if (world_tracks < m->cfg.T) PT_FAIL(PT_ERR_INVALID_ARG, "world_tracks %d is smaller than this rank's %d tracks", world_tracks, m->cfg.T);
    m->world_tracks = world_tracks; m->ar_fn = fn; m->ar_user = user;
    return PT_OK;
}

int32_t pt_sync_count(const pt_model* m) { return m ? m->cfg.L / m->cfg.D : -1; }

pt_status pt_model_weight_bytes(const pt_model* m, size_t* bytes) {
    if (!m || !bytes) PT_FAIL(PT_ERR_INVALID_ARG, "null argument");
    *bytes = m->total_bytes;
    return PT_OK;
}

pt_status pt_model_bind_weights(pt_model* m, void* dev_buf, size_t bytes) {
    if (!m || !dev_buf) PT_FAIL(PT_ERR_INVALID_ARG, "null argument");
    if (bytes < m->total_bytes) PT_FAIL(PT_ERR_BUFFER_TOO_SMALL, "weight buffer: %zu < %zu bytes", bytes, m->total_bytes);
    if ((uintptr_t)dev_buf % 256) PT_FAIL(PT_ERR_MISALIGNED, "weight buffer must be 256-byte aligned");
    const pt_config& c = m->cfg;
    int half = m->dh / 2;
    std::vector<float> cs((size_t)c.max_pos * half), sn((size_t)c.max_pos * half);
    for (int j = 0; j < half; ++j) {
        double theta = std::pow((double)c.rope_base, -2.0 * j / m->dh);
        for (int p = 0; p < c.max_pos; ++p) {
            double ang = (double)p * theta;
            cs[(size_t)p * half + j] = (float)std::cos(ang);
            sn[(size_t)p * half + j] = (float)std::sin(ang);
        }
    }
    char* b = (char*)dev_buf;
    PT_CUDA(cudaMemcpy(b + m->off_cos, cs.data(), cs.size() * 4, cudaMemcpyHostToDevice));
    PT_CUDA(cudaMemcpy(b + m->off_sin, sn.data(), sn.size() * 4, cudaMemcpyHostToDevice));
    {   // the tensor-core path reads (cos, sin) as fp16 pairs: 2^-12 absolute error, an eighth of the bf16
        // rounding q and k receive right after the rotation, for half the table bytes per token
        std::vector<__half2> cs16(cs.size());
        for (size_t i = 0; i < cs.size(); ++i) cs16[i] = __halves2half2(__float2half_rn(cs[i]), __float2half_rn(sn[i]));
        PT_CUDA(cudaMemcpy(b + m->off_cs16, cs16.data(), cs16.size() * 4, cudaMemcpyHostToDevice));
    }
    PT_CUDA(cudaMemset(b + m->off_g1, 0, (size_t)c.L * c.T * c.hidden * 4));
    PT_CUDA(cudaMemset(b + m->off_g2, 0, (size_t)c.L * c.T * c.hidden * 4));
    PT_CUDA(cudaMemset(b + m->off_status, 0, kStatusWords * 4));
    m->wbuf = b;
    if (m->tc) {
        pt_status s = tc_build_weight_maps(m);
        if (s != PT_OK) { m->wbuf = nullptr; return s; }
    }
    return PT_OK;
}

pt_status pt_model_set_weight(pt_model* m, int32_t track, int32_t layer, int32_t kind,
                              const void* dev_src, void* stream) {
    if (!m || !dev_src) PT_FAIL(PT_ERR_INVALID_ARG, "null argument");
    if (!m->wbuf) PT_FAIL(PT_ERR_STATE, "pt_model_bind_weights has not been called");
    const pt_config& c = m->cfg;
    if (track < 0 || track >= c.T || layer < 0 || layer >= c.L || kind < 0 || kind > PT_WR)
        PT_FAIL(PT_ERR_INVALID_ARG, "track/layer/kind out of range");
    cudaStream_t st = (cudaStream_t)stream;
    if (kind == PT_WR) {
        if (!m->E) PT_FAIL(PT_ERR_INVALID_ARG, "the model has no router (experts == 0)");
        float* dst = (float*)(m->wbuf + m->off_wr) + ((size_t)layer * c.T + track) * m->E * c.hidden;
        PT_CUDA(cudaMemcpyAsync(dst, dev_src, (size_t)m->E * c.hidden * 4, cudaMemcpyDeviceToDevice, st));
        return PT_OK;
    }
    if (m->E && (kind == PT_WG || kind == PT_WU || kind == PT_WD))
        PT_FAIL(PT_ERR_INVALID_ARG, "a PT-MoE model takes its feed-forward weights expert by expert: pt_model_set_expert_weight");
    if (kind == PT_G1 || kind == PT_G2) {
        float* dst = (float*)(m->wbuf + (kind == PT_G1 ? m->off_g1 : m->off_g2)) + ((size_t)layer * c.T + track) * c.hidden;
        PT_CUDA(cudaMemcpyAsync(dst, dev_src, (size_t)c.hidden * 4, cudaMemcpyDeviceToDevice, st));
        return PT_OK;
    }
    char* base;
    switch (kind) {
        case PT_WQ: case PT_WK: case PT_WV:
            base = m->wbuf + m->off_wqkv + ((size_t)layer * c.T + track) * m->Nqkv * c.hidden * m->esz; break;
        case PT_WO:
            base = m->wbuf + m->off_wo + ((size_t)layer * c.T + track) * c.hidden * m->QD * m->esz; break;
        case PT_WG: case PT_WU:
            base = m->wbuf + m->off_wgu + ((size_t)layer * c.T + track) * 2 * m->Ftot * c.hidden * m->esz; break;
        default:
            base = m->wbuf + m->off_wd + ((size_t)layer * c.T + track) * c.hidden * m->Ftot * m->esz; break;
    }
    launch_pack(m, kind, dev_src, base, st);
    PT_CUDA(cudaGetLastError());
    return PT_OK;
}

pt_status pt_model_set_expert_weight(pt_model* m, int32_t track, int32_t layer, int32_t expert, int32_t kind,
                                     const void* dev_src, void* stream) {
    if (!m || !dev_src) PT_FAIL(PT_ERR_INVALID_ARG, "null argument");
    if (!m->wbuf) PT_FAIL(PT_ERR_STATE, "pt_model_bind_weights has not been called");
    const pt_config& c = m->cfg;
    if (!m->E) PT_FAIL(PT_ERR_INVALID_ARG, "the model has no experts");
    if (track < 0 || track >= c.T || layer < 0 || layer >= c.L || expert < 0 || expert >= m->E)
        PT_FAIL(PT_ERR_INVALID_ARG, "track/layer/expert out of range");
    if (kind != PT_WG && kind != PT_WU && kind != PT_WD) PT_FAIL(PT_ERR_INVALID_ARG, "kind must be PT_WG, PT_WU or PT_WD");
    char* base = kind == PT_WD ? m->wbuf + m->off_wd + ((size_t)layer * c.T + track) * c.hidden * m->Ftot * m->esz
                               : m->wbuf + m->off_wgu + ((size_t)layer * c.T + track) * 2 * m->Ftot * c.hidden * m->esz;
    launch_pack(m, kind, dev_src, base, (cudaStream_t)stream, expert);
    PT_CUDA(cudaGetLastError());
    return PT_OK;
}

/* ------------------------------------------------------------------ KV cache (host logic) */

// Bytes of the codes (or model-dtype values) of a pool; an E4M3 pool's scales follow, 256-byte aligned.
static pt_status kv_pool_layout(const pt_model* m, int32_t num_pages, int32_t page_size, int32_t kv_dtype,
                                size_t* codes_bytes, size_t* total) {
    if (!m) PT_FAIL(PT_ERR_INVALID_ARG, "null argument");
    if (num_pages < 1) PT_FAIL(PT_ERR_INVALID_ARG, "num_pages must be >= 1");
    if (page_size < 8 || page_size > 64 || page_size % 8) PT_FAIL(PT_ERR_INVALID_ARG, "page_size must be a multiple of 8 in [8, 64]");
    if (kv_dtype != PT_KV_MODEL && kv_dtype != PT_KV_E4M3) PT_FAIL(PT_ERR_INVALID_ARG, "kv_dtype must be PT_KV_MODEL or PT_KV_E4M3");
    const size_t vecs = (size_t)m->cfg.T * m->cfg.L * num_pages * 2 * m->cfg.kv_heads * page_size;
    if (kv_dtype == PT_KV_E4M3) {
        if (!m->tc) PT_FAIL(PT_ERR_UNSUPPORTED, "an E4M3 cache needs a bf16 model on the tensor-core path");
        if (m->dh != 128 || page_size % 16) PT_FAIL(PT_ERR_UNSUPPORTED, "an E4M3 cache needs head_dim 128 and pages of a multiple of 16 tokens");
        *codes_bytes = align_up(vecs * m->dh, 256);
        *total = *codes_bytes + vecs * 4;
    } else {
        *codes_bytes = vecs * m->dh * m->esz;
        *total = *codes_bytes;
    }
    return PT_OK;
}

pt_status pt_kv_cache_bytes_ex(const pt_model* m, int32_t num_pages, int32_t page_size, int32_t kv_dtype, size_t* bytes) {
    if (!bytes) PT_FAIL(PT_ERR_INVALID_ARG, "null argument");
    size_t codes = 0;
    return kv_pool_layout(m, num_pages, page_size, kv_dtype, &codes, bytes);
}

pt_status pt_kv_cache_bytes(const pt_model* m, int32_t num_pages, int32_t page_size, size_t* bytes) {
    return pt_kv_cache_bytes_ex(m, num_pages, page_size, PT_KV_MODEL, bytes);
}

pt_status pt_kv_cache_alloc(const pt_model* m, int32_t num_pages, int32_t page_size,
                            void* dev_pool, size_t bytes, pt_kv_cache** out) {
    return pt_kv_cache_alloc_ex(m, num_pages, page_size, PT_KV_MODEL, dev_pool, bytes, out);
}

pt_status pt_kv_cache_alloc_ex(const pt_model* m, int32_t num_pages, int32_t page_size, int32_t kv_dtype,
                               void* dev_pool, size_t bytes, pt_kv_cache** out) {
    size_t need = 0, codes = 0;
    if (!out || !dev_pool) PT_FAIL(PT_ERR_INVALID_ARG, "null argument");
    pt_status s = kv_pool_layout(m, num_pages, page_size, kv_dtype, &codes, &need);
    if (s != PT_OK) return s;
    if (bytes < need) PT_FAIL(PT_ERR_BUFFER_TOO_SMALL, "KV pool: %zu < %zu bytes", bytes, need);
    if ((uintptr_t)dev_pool % 256) PT_FAIL(PT_ERR_MISALIGNED, "KV pool must be 256-byte aligned");
    pt_kv_cache* c = new (std::nothrow) pt_kv_cache();
    if (!c) PT_FAIL(PT_ERR_INVALID_ARG, "out of host memory");
    c->m = m; c->num_pages = num_pages; c->ps = page_size; c->pool = (char*)dev_pool; c->bytes = bytes;
    c->kv_dtype = kv_dtype;
    c->esz = kv_dtype == PT_KV_E4M3 ? 1 : m->esz;
    c->scales = kv_dtype == PT_KV_E4M3 ? (float*)((char*)dev_pool + codes) : nullptr;
    c->page_elems = (int64_t)2 * m->cfg.kv_heads * page_size * m->dh;
    c->slab_elems = c->page_elems * num_pages;
    for (int i = 0; i < num_pages; ++i) c->free_list.push_back(i);
    *out = c;
    return PT_OK;
}

void pt_kv_cache_free(pt_kv_cache* c) { delete c; }

pt_status pt_kv_set_free_list(pt_kv_cache* c, const int32_t* order, int32_t n) {
    if (!c || !order) PT_FAIL(PT_ERR_INVALID_ARG, "null argument");
    if ((int)c->free_list.size() != c->num_pages) PT_FAIL(PT_ERR_STATE, "pages are in use");
    if (n != c->num_pages) PT_FAIL(PT_ERR_INVALID_ARG, "order must list all %d pages", c->num_pages);
    std::vector<char> seen(n, 0);
    for (int i = 0; i < n; ++i) {
        if (order[i] < 0 || order[i] >= n || seen[order[i]]) PT_FAIL(PT_ERR_INVALID_ARG, "order is not a permutation");
        seen[order[i]] = 1;
    }
    c->free_list.assign(order, order + n);
    return PT_OK;
}

pt_status pt_kv_seq_reserve(pt_kv_cache* c, int32_t seq, int32_t new_len) {
    if (!c || seq < 0 || new_len < 0) PT_FAIL(PT_ERR_INVALID_ARG, "bad argument");
    auto it = c->seqs.find(seq);
    size_t have = it == c->seqs.end() ? 0 : it->second.pages.size();
    size_t need = ((size_t)new_len + c->ps - 1) / c->ps;
    if (need > have && need - have > c->free_list.size())
        PT_FAIL(PT_ERR_CACHE_FULL, "sequence %d needs %zu more pages, %zu free", seq, need - have, c->free_list.size());
    Seq& s = c->seqs[seq];
    while (s.pages.size() < need) { s.pages.push_back(c->free_list.front()); c->free_list.pop_front(); }
    return PT_OK;
}

pt_status pt_kv_seq_release(pt_kv_cache* c, int32_t seq) {
    if (!c) PT_FAIL(PT_ERR_INVALID_ARG, "null argument");
    auto it = c->seqs.find(seq);
    if (it == c->seqs.end()) PT_FAIL(PT_ERR_STATE, "unknown sequence %d", seq);
    for (int32_t p : it->second.pages) c->free_list.push_back(p);
    c->seqs.erase(it);
    return PT_OK;
}

pt_status pt_kv_seq_len(const pt_kv_cache* c, int32_t seq, int32_t* len) {
    if (!c || !len) PT_FAIL(PT_ERR_INVALID_ARG, "null argument");
    auto it = c->seqs.find(seq);
    *len = it == c->seqs.end() ? 0 : it->second.len;
    return PT_OK;
}

pt_status pt_kv_seq_truncate(pt_kv_cache* c, int32_t seq, int32_t len) {
    if (!c) PT_FAIL(PT_ERR_INVALID_ARG, "null argument");
    auto it = c->seqs.find(seq);
    if (it == c->seqs.end()) PT_FAIL(PT_ERR_STATE, "unknown sequence %d", seq);
    if (len < 0 || len > it->second.len) PT_FAIL(PT_ERR_INVALID_ARG, "len %d outside [0, %d]", len, it->second.len);
    it->second.len = len;
    return PT_OK;
}

pt_status pt_kv_block_table(const pt_kv_cache* c, int32_t seq, int32_t* pages, int32_t cap, int32_t* n) {
    if (!c || !n) PT_FAIL(PT_ERR_INVALID_ARG, "null argument");
    auto it = c->seqs.find(seq);
    int cnt = it == c->seqs.end() ? 0 : (int)it->second.pages.size();
    *n = cnt;
    if (pages) for (int i = 0; i < cnt && i < cap; ++i) pages[i] = it->second.pages[i];
    return PT_OK;
}

// Offset, inside one (track, layer) slab, of the head_dim values of (page, kv, head, slot).
static inline int64_t slab_offset(const pt_kv_cache* c, int32_t page, int kv, int head, int slot) {
    return (((int64_t)page * 2 + kv) * c->m->cfg.kv_heads + head) * c->ps * c->m->dh + (int64_t)slot * c->m->dh;
}

pt_status pt_kv_slot(const pt_kv_cache* c, int32_t track, int32_t layer, int32_t seq, int32_t pos,
                     int32_t kv, int32_t kv_head, int64_t* elem_offset) {
    if (!c || !elem_offset) PT_FAIL(PT_ERR_INVALID_ARG, "null argument");
    const pt_config& g = c->m->cfg;
    if (track < 0 || track >= g.T || layer < 0 || layer >= g.L || kv < 0 || kv > 1 || kv_head < 0 || kv_head >= g.kv_heads || pos < 0)
        PT_FAIL(PT_ERR_INVALID_ARG, "index out of range");
    auto it = c->seqs.find(seq);
    if (it == c->seqs.end()) PT_FAIL(PT_ERR_STATE, "unknown sequence %d", seq);
    if ((size_t)(pos / c->ps) >= it->second.pages.size()) PT_FAIL(PT_ERR_INVALID_ARG, "position %d is outside the reserved pages", pos);
    int32_t page = it->second.pages[pos / c->ps];
    *elem_offset = ((int64_t)track * g.L + layer) * c->slab_elems + slab_offset(c, page, kv, kv_head, pos % c->ps);
    return PT_OK;
}

pt_status pt_kv_scale_slot(const pt_kv_cache* c, int32_t track, int32_t layer, int32_t seq, int32_t pos,
                           int32_t kv, int32_t kv_head, int64_t* byte_offset) {
    if (!c || !byte_offset) PT_FAIL(PT_ERR_INVALID_ARG, "null argument");
    if (c->kv_dtype != PT_KV_E4M3) PT_FAIL(PT_ERR_STATE, "the cache holds no scales");
    int64_t elem = 0;
    pt_status s = pt_kv_slot(c, track, layer, seq, pos, kv, kv_head, &elem);
    if (s != PT_OK) return s;
    *byte_offset = ((char*)c->scales - c->pool) + (elem / c->m->dh) * 4;
    return PT_OK;
}

/* ------------------------------------------------------------------ forward */

pt_status pt_workspace_bytes(const pt_model* m, int64_t max_tokens, int32_t max_batch,
                             int32_t page_size, size_t* bytes) {
    if (!m || !bytes) PT_FAIL(PT_ERR_INVALID_ARG, "null argument");
    if (max_tokens < 1 || max_batch < 1 || max_batch > max_tokens || page_size < 8) PT_FAIL(PT_ERR_INVALID_ARG, "bad sizes");
    return pt_workspace_bytes_ex(m, max_tokens, max_batch, page_size, PT_KV_MODEL, 0, bytes);
}

pt_status pt_workspace_bytes_ex(const pt_model* m, int64_t max_tokens, int32_t max_batch, int32_t page_size,
                                int32_t kv_dtype, int64_t max_context, size_t* bytes) {
    if (!m || !bytes) PT_FAIL(PT_ERR_INVALID_ARG, "null argument");
    if (max_tokens < 1 || max_batch < 1 || max_batch > max_tokens || page_size < 8 || max_context < 0) PT_FAIL(PT_ERR_INVALID_ARG, "bad sizes");
    if (kv_dtype != PT_KV_MODEL && kv_dtype != PT_KV_E4M3) PT_FAIL(PT_ERR_INVALID_ARG, "kv_dtype must be PT_KV_MODEL or PT_KV_E4M3");
    int maxp = (m->cfg.max_pos + page_size - 1) / page_size;
    const bool fp8 = kv_dtype == PT_KV_E4M3;
    const int64_t ctx = fp8 ? std::max<int64_t>(max_context, max_tokens + 16 * (int64_t)max_batch) : 0;
    *bytes = carve(m, max_tokens, max_batch, maxp, fp8, ctx, nullptr, nullptr);
    return PT_OK;
}

static pt_status forward(pt_model* m, pt_kv_cache* c, const void* x, int64_t x_stride, int32_t B, int32_t S,
                         const int32_t* seq_ids, void* out_h, void* workspace, size_t ws_bytes, void* stream,
                         bool decode) {
    if (!m || !c || !x || !seq_ids || !out_h || !workspace) PT_FAIL(PT_ERR_INVALID_ARG, "null argument");
    if (c->m != m) PT_FAIL(PT_ERR_INVALID_ARG, "cache belongs to another model");
    if (!m->wbuf) PT_FAIL(PT_ERR_STATE, "pt_model_bind_weights has not been called");
    if (B < 1 || S < 1) PT_FAIL(PT_ERR_INVALID_ARG, "B and S must be >= 1");
    if (x_stride < 0) PT_FAIL(PT_ERR_INVALID_ARG, "negative track stride");
    if ((uintptr_t)workspace % 256 || (uintptr_t)x % 16 || (uintptr_t)out_h % 32)
        PT_FAIL(PT_ERR_MISALIGNED, "workspace must be 256-byte aligned, x 16-byte and out_h 32-byte aligned");
    const pt_config& g = m->cfg;
    if (x_stride % 8) PT_FAIL(PT_ERR_MISALIGNED, "x_track_stride must be a multiple of 8 elements");
    int64_t M = (int64_t)B * S;
    if (M > (1 << 30)) PT_FAIL(PT_ERR_INVALID_ARG, "too many tokens");
    // validate ids and positions before touching the allocator
    std::unordered_set<int32_t> ids;
    int maxlen = 0;
    size_t pages_needed = 0;
    for (int b = 0; b < B; ++b) {
        if (seq_ids[b] < 0 || !ids.insert(seq_ids[b]).second) PT_FAIL(PT_ERR_INVALID_ARG, "seq_ids must be distinct and non-negative");
        auto it = c->seqs.find(seq_ids[b]);
        int len = it == c->seqs.end() ? 0 : it->second.len;
        size_t have = it == c->seqs.end() ? 0 : it->second.pages.size();
        if ((int64_t)len + S > g.max_pos) PT_FAIL(PT_ERR_INVALID_ARG, "sequence %d would reach position %d >= max_pos %d", seq_ids[b], len + S - 1, g.max_pos);
        size_t need = ((size_t)len + S + c->ps - 1) / c->ps;
        if (need > have) pages_needed += need - have;
        maxlen = std::max(maxlen, len + S);
    }
    if (pages_needed > c->free_list.size()) PT_FAIL(PT_ERR_CACHE_FULL, "call needs %zu new pages, %zu free", pages_needed, c->free_list.size());
    int maxp = (maxlen + c->ps - 1) / c->ps;
    const bool fp8 = c->kv_dtype == PT_KV_E4M3;
    if (fp8 && !m->tc) PT_FAIL(PT_ERR_UNSUPPORTED, "an E4M3 cache needs the tensor-core path");
    // E4M3 cache, prefill: the attention kernel reads a bf16 copy of code * scale of every key of the call's sequences
    int64_t ctx_keys = 0;
    if (fp8 && !decode)
        for (int b = 0; b < B; ++b) {
            auto it = c->seqs.find(seq_ids[b]);
            int len = it == c->seqs.end() ? 0 : it->second.len;
            ctx_keys += ((int64_t)len + S + 15) / 16 * 16;
        }
    Call k{};
    size_t need_ws = carve(m, M, B, maxp, fp8, ctx_keys, (char*)workspace, &k.w);
    if (ws_bytes < need_ws) PT_FAIL(PT_ERR_BUFFER_TOO_SMALL, "workspace: %zu < %zu bytes", ws_bytes, need_ws);
    for (int b = 0; b < B; ++b) {
        auto it = c->seqs.find(seq_ids[b]);
        int len = it == c->seqs.end() ? 0 : it->second.len;
        pt_status s = pt_kv_seq_reserve(c, seq_ids[b], len + S);
        if (s != PT_OK) return s;
    }
    // per-call metadata, one upload
    size_t mb = meta_bytes(M, B, maxp, fp8);
    m->meta_host.assign(mb, 0);
    char* hb = m->meta_host.data();
    char* db = (char*)workspace;
    size_t off = 0;
    auto sect = [&](size_t bytes) { size_t o = off; off += align_up(bytes, 256); return o; };
    size_t o_kvoff = sect((size_t)M * 8), o_pos = sect((size_t)M * 4), o_b = sect((size_t)M * 4);
    size_t o_len = sect((size_t)B * 4), o_nsp = sect((size_t)B * 4), o_bt = sect((size_t)B * maxp * 4);
    size_t o_items = sect((size_t)B * kMaxSplits * 16);
    int64_t* h_kvoff = (int64_t*)(hb + o_kvoff);
    int32_t* h_pos = (int32_t*)(hb + o_pos);
    int32_t* h_b = (int32_t*)(hb + o_b);
    int32_t* h_len = (int32_t*)(hb + o_len);
    int32_t* h_nsp = (int32_t*)(hb + o_nsp);
    int32_t* h_bt = (int32_t*)(hb + o_bt);
    int32_t* h_items = (int32_t*)(hb + o_items);
    for (int b = 0; b < B; ++b) {
        const Seq& s = c->seqs[seq_ids[b]];
        for (size_t i = 0; i < s.pages.size() && i < (size_t)maxp; ++i) h_bt[(size_t)b * maxp + i] = s.pages[i];
        h_len[b] = s.len + S;
        for (int t = 0; t < S; ++t) {
            int pos = s.len + t;
            int64_t r = (int64_t)b * S + t;
            h_pos[r] = pos;
            h_b[r] = b;
            h_kvoff[r] = slab_offset(c, s.pages[pos / c->ps], 0, 0, pos % c->ps);
        }
    }
    size_t o_stageoff = 0, o_attnoff = 0, o_start = 0, o_btattn = 0;
    const int maxp_attn = (maxlen + 15) / 16;
    int max_start = 0;
    if (fp8) {
        o_stageoff = sect((size_t)M * 8); o_attnoff = sect((size_t)M * 8); o_start = sect((size_t)B * 4);
        o_btattn = sect((size_t)B * maxp_attn * 4);
        int64_t* h_stage = (int64_t*)(hb + o_stageoff);
        int64_t* h_attn = (int64_t*)(hb + o_attnoff);
        int32_t* h_start = (int32_t*)(hb + o_start);
        int32_t* h_bta = (int32_t*)(hb + o_btattn);
        int32_t base = 0;                                 // first 16-token page of the sequence in the attention copy
        for (int b = 0; b < B; ++b) {
            const Seq& s = c->seqs[seq_ids[b]];
            h_start[b] = s.len;
            max_start = std::max(max_start, s.len);
            const int np = (s.len + S + 15) / 16;
            for (int i = 0; i < np; ++i) h_bta[(size_t)b * maxp_attn + i] = base + i;
            for (int t = 0; t < S; ++t) {
                const int pos = s.len + t;
                const int64_t r = (int64_t)b * S + t;
                h_stage[r] = r * m->dh;
                h_attn[r] = ((int64_t)(base + pos / 16) * 2 * g.kv_heads) * 16 * m->dh + (int64_t)(pos % 16) * m->dh;
            }
            base += np;
        }
    }
    int n_items = 0, max_splits = 1;
    if (decode) plan_decode_splits(h_len, B, c->ps, (int64_t)g.T * g.kv_heads, h_items, h_nsp, &n_items, &max_splits);
    cudaStream_t st = (cudaStream_t)stream;
    PT_CUDA(cudaMemcpyAsync(db, hb, mb, cudaMemcpyHostToDevice, st));
    k.w.meta.row_kvoff = (const int64_t*)(db + o_kvoff);
    k.w.meta.row_pos = (const int32_t*)(db + o_pos);
    k.w.meta.row_b = (const int32_t*)(db + o_b);
    k.w.meta.kvlen = (const int32_t*)(db + o_len);
    k.w.meta.bt = (const int32_t*)(db + o_bt);
    k.w.meta.maxp = maxp;
    if (fp8) {
        k.w.meta.row_stageoff = (const int64_t*)(db + o_stageoff);
        k.w.meta.row_attnoff = (const int64_t*)(db + o_attnoff);
        k.w.meta.ctx_start = (const int32_t*)(db + o_start);
        k.w.meta.bt_attn = (const int32_t*)(db + o_btattn);
        k.w.meta.maxp_attn = maxp_attn;
        k.w.meta.attn_pages = (int32_t)(ctx_keys / 16);
        k.w.meta.max_start = max_start;
    }
    k.m = m; k.c = c; k.B = B; k.S = S; k.M = (int)M; k.x = x; k.x_stride = x_stride;
    k.out = (float*)out_h; k.st = st; k.decode = decode;
    k.n_items = n_items; k.max_splits = max_splits;
    k.items = (const int32_t*)(db + o_items); k.nsplit = (const int32_t*)(db + o_nsp);
    pt_status s = m->tc ? tc_forward(k) : simt_forward(k);
    if (s != PT_OK) return s;
    for (int b = 0; b < B; ++b) c->seqs[seq_ids[b]].len += S;
    return PT_OK;
}

pt_status pt_prefill(pt_model* m, pt_kv_cache* c, const void* x, int64_t x_track_stride,
                     int32_t B, int32_t S, const int32_t* seq_ids, void* out_h,
                     void* workspace, size_t ws_bytes, void* stream) {
    return forward(m, c, x, x_track_stride, B, S, seq_ids, out_h, workspace, ws_bytes, stream, false);
}

pt_status pt_decode_step(pt_model* m, pt_kv_cache* c, const void* x, int64_t x_track_stride,
                         int32_t B, const int32_t* seq_ids, void* out_h,
                         void* workspace, size_t ws_bytes, void* stream) {
    return forward(m, c, x, x_track_stride, B, 1, seq_ids, out_h, workspace, ws_bytes, stream, true);
}

pt_status pt_set_debug_tap(pt_model* m, int32_t layer, void* dev_buf) {
    if (!m) PT_FAIL(PT_ERR_INVALID_ARG, "null argument");
    if (!dev_buf) { m->tap_layer = -2; m->tap_buf = nullptr; return PT_OK; }
    if (layer < -1 || layer >= m->cfg.L) PT_FAIL(PT_ERR_INVALID_ARG, "layer out of range");
    if ((uintptr_t)dev_buf % 16) PT_FAIL(PT_ERR_MISALIGNED, "tap buffer must be 16-byte aligned");
    m->tap_layer = layer;
    m->tap_buf = (float*)dev_buf;
    return PT_OK;
}

pt_status pt_device_status(pt_model* m, void* stream, int32_t* code, int32_t* detail) {
    if (!m || !code) PT_FAIL(PT_ERR_INVALID_ARG, "null argument");
    if (!m->wbuf) PT_FAIL(PT_ERR_STATE, "pt_model_bind_weights has not been called");
    int32_t w[kStatusWords];
    cudaStream_t st = (cudaStream_t)stream;
    PT_CUDA(cudaStreamSynchronize(st));
    PT_CUDA(cudaMemcpy(w, m->status(), sizeof(w), cudaMemcpyDeviceToHost));
    *code = w[0];
    if (detail) *detail = w[1];
    if (w[0] != 0) PT_CUDA(cudaMemset(m->status(), 0, sizeof(w)));
    return PT_OK;
}

}  // extern "C"
