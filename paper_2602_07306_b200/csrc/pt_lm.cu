// Ends of the model around Algorithm 1 (bf16 models): embedding lookup that produces the shared
// input x, final RMSNorm + LM head + greedy choice on the returned h, and a greedy generate loop
// that keeps the token ids on the device.  The LM head is the track-grouped tcgen05 GEMM with one
// "track" (plain epilogue); everything else here is a small row-per-warp kernel.
#include "pt_tc.h"

namespace pt {

namespace {

// x[r][:] = table[tokens[r]][:]  (16-byte pieces; H is a multiple of 16 elements)
__global__ void k_embed(const __nv_bfloat16* __restrict__ table, const int32_t* __restrict__ tokens, int vocab,
                        __nv_bfloat16* __restrict__ x, int64_t n, int H, int* status) {
    int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    if (row >= n) return;
    int tok = tokens[row];
    if (tok < 0 || tok >= vocab) {                        // reported, and the row is filled from token 0
        if (lane == 0 && atomicCAS(status, 0, PT_ERR_DEVICE_BOUNDS) == 0) status[1] = LOC_EMBED_TOKEN;
        tok = 0;
    }
    const uint4* src = reinterpret_cast<const uint4*>(table + (size_t)tok * H);
    uint4* dst = reinterpret_cast<uint4*>(x + (size_t)row * H);
    for (int i = lane; i < H / 8; i += 32) dst[i] = src[i];
}

// hn[r][:] = bf16( h_row / sqrt(mean(h_row^2) + eps) * gain ), h_row = h + r * row_stride
__global__ void k_final_norm(const float* __restrict__ h, int64_t row_stride, const float* __restrict__ gain,
                             __nv_bfloat16* __restrict__ hn, int64_t n, int H, float eps) {
    int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    if (row >= n) return;
    const float4* src = reinterpret_cast<const float4*>(h + row * row_stride);
    float s = 0.f;
    for (int i = lane; i < H / 4; i += 32) { float4 v = src[i]; s += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w; }
    for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const float rinv = 1.0f / sqrtf(s / (float)H + eps);
    const float4* g4 = reinterpret_cast<const float4*>(gain);
    uint2* dst = reinterpret_cast<uint2*>(hn + (size_t)row * H);
    for (int i = lane; i < H / 4; i += 32) {
        float4 v = src[i], g = g4[i];
        __nv_bfloat162 a = __floats2bfloat162_rn(v.x * rinv * g.x, v.y * rinv * g.y), b = __floats2bfloat162_rn(v.z * rinv * g.z, v.w * rinv * g.w);
        uint2 o;
        o.x = *reinterpret_cast<uint32_t*>(&a); o.y = *reinterpret_cast<uint32_t*>(&b);
        dst[i] = o;
    }
}

// next[r] = lowest index of the largest logit of row r (NaNs never win); also scattered to out[r * out_stride]
__global__ void k_argmax(const float* __restrict__ logits, int vocab, int32_t* __restrict__ next, int32_t* __restrict__ out, int64_t out_stride) {
    __shared__ float sv[32];
    __shared__ int si[32];
    const float* row = logits + (size_t)blockIdx.x * vocab;
    float best = -INFINITY; int idx = 0x7fffffff;
    for (int i = threadIdx.x; i < vocab; i += blockDim.x) { float v = row[i]; if (v > best) { best = v; idx = i; } }
    auto better = [](float v, int i, float bv, int bi) { return v > bv || (v == bv && i < bi); };
    for (int o = 16; o; o >>= 1) {
        float ov = __shfl_xor_sync(0xffffffffu, best, o); int oi = __shfl_xor_sync(0xffffffffu, idx, o);
        if (better(ov, oi, best, idx)) { best = ov; idx = oi; }
    }
    if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = best; si[threadIdx.x >> 5] = idx; }
    __syncthreads();
    if (threadIdx.x < 32) {
        const int nw = blockDim.x >> 5;
        best = threadIdx.x < nw ? sv[threadIdx.x] : -INFINITY; idx = threadIdx.x < nw ? si[threadIdx.x] : 0x7fffffff;
        for (int o = 16; o; o >>= 1) {
            float ov = __shfl_xor_sync(0xffffffffu, best, o); int oi = __shfl_xor_sync(0xffffffffu, idx, o);
            if (better(ov, oi, best, idx)) { best = ov; idx = oi; }
        }
        if (threadIdx.x == 0) {
            if (idx < 0 || idx >= vocab) idx = 0;
            if (next) next[blockIdx.x] = idx;
            if (out) out[(size_t)blockIdx.x * out_stride] = idx;
        }
    }
}

struct LmLayout { size_t off_table, off_head, off_gain, total; };
LmLayout lm_layout(const pt_model* m, int vocab) {
    LmLayout l{};
    size_t off = 0;
    auto take = [&](size_t b) { size_t o = off; off += align_up(b, 256); return o; };
    l.off_table = take((size_t)vocab * m->cfg.hidden * 2);
    l.off_head = take((size_t)vocab * m->cfg.hidden * 2);
    l.off_gain = take((size_t)m->cfg.hidden * 4);
    l.total = off;
    return l;
}

pt_status lm_check(const pt_model* m) {
    if (!m) { set_error("null model"); return PT_ERR_INVALID_ARG; }
    if (!m->tc) { set_error("the model ends are built for bf16 models on the tensor-core path"); return PT_ERR_UNSUPPORTED; }
    if (!m->wbuf) { set_error("pt_model_bind_weights has not been called"); return PT_ERR_STATE; }
    if (!m->lm_buf) { set_error("pt_lm_bind has not been called"); return PT_ERR_STATE; }
    return PT_OK;
}

}  // namespace
}  // namespace pt

using namespace pt;

#define LM_CUDA(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) { \
    set_error("%s failed: %s", #call, cudaGetErrorString(e_)); return PT_ERR_CUDA; } } while (0)

extern "C" {

pt_status pt_lm_bytes(const pt_model* m, int32_t vocab, size_t* bytes) {
    if (!m || !bytes) { set_error("null argument"); return PT_ERR_INVALID_ARG; }
    if (!m->tc) { set_error("the model ends are built for bf16 models on the tensor-core path"); return PT_ERR_UNSUPPORTED; }
    if (vocab < 16 || vocab % 16) { set_error("vocab must be a positive multiple of 16"); return PT_ERR_INVALID_ARG; }
    *bytes = lm_layout(m, vocab).total;
    return PT_OK;
}

pt_status pt_lm_bind(pt_model* m, int32_t vocab, void* dev_buf, size_t bytes) {
    size_t need = 0;
    pt_status s = pt_lm_bytes(m, vocab, &need);
    if (s != PT_OK) return s;
    if (!dev_buf) { set_error("null buffer"); return PT_ERR_INVALID_ARG; }
    if ((uintptr_t)dev_buf % 256) { set_error("buffer must be 256-byte aligned"); return PT_ERR_MISALIGNED; }
    if (bytes < need) { set_error("buffer: %zu < %zu bytes", bytes, need); return PT_ERR_BUFFER_TOO_SMALL; }
    m->lm_buf = (char*)dev_buf;
    m->lm_vocab = vocab;
    return PT_OK;
}

pt_status pt_lm_set(pt_model* m, int32_t kind, const void* dev_src, void* stream) {
    pt_status s = lm_check(m);
    if (s != PT_OK) return s;
    if (!dev_src || kind < 0 || kind > 2) { set_error("bad argument"); return PT_ERR_INVALID_ARG; }
    LmLayout l = lm_layout(m, m->lm_vocab);
    const size_t mat = (size_t)m->lm_vocab * m->cfg.hidden * 2;
    char* dst = m->lm_buf + (kind == 0 ? l.off_table : kind == 1 ? l.off_head : l.off_gain);
    LM_CUDA(cudaMemcpyAsync(dst, dev_src, kind == 2 ? (size_t)m->cfg.hidden * 4 : mat, cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
    return PT_OK;
}

pt_status pt_embed(pt_model* m, const int32_t* dev_tokens, int64_t n, void* x_out, void* stream) {
    pt_status s = lm_check(m);
    if (s != PT_OK) return s;
    if (!dev_tokens || !x_out || n < 1) { set_error("bad argument"); return PT_ERR_INVALID_ARG; }
    if ((uintptr_t)x_out % 16) { set_error("x_out must be 16-byte aligned"); return PT_ERR_MISALIGNED; }
    LmLayout l = lm_layout(m, m->lm_vocab);
    k_embed<<<(unsigned)((n * 32 + 255) / 256), 256, 0, (cudaStream_t)stream>>>(
        (const __nv_bfloat16*)(m->lm_buf + l.off_table), dev_tokens, m->lm_vocab, (__nv_bfloat16*)x_out, n, m->cfg.hidden, m->status());
    g_launches.fetch_add(1, std::memory_order_relaxed);
    LM_CUDA(cudaGetLastError());
    return PT_OK;
}

pt_status pt_lm_workspace_bytes(const pt_model* m, int64_t n, size_t* bytes) {
    if (!m || !bytes || n < 1) { set_error("bad argument"); return PT_ERR_INVALID_ARG; }
    *bytes = align_up((size_t)n * m->cfg.hidden * 2, 256);
    return PT_OK;
}

pt_status pt_lm_head(pt_model* m, const float* h, int64_t row_stride, int64_t n, float* logits, int32_t* next_token,
                     void* workspace, size_t ws_bytes, void* stream) {
    pt_status s = lm_check(m);
    if (s != PT_OK) return s;
    if (!h || !logits || !workspace || n < 1 || n > (1 << 30) || row_stride < m->cfg.hidden) { set_error("bad argument"); return PT_ERR_INVALID_ARG; }
    if ((uintptr_t)h % 16 || row_stride % 4 || (uintptr_t)logits % 16 || (uintptr_t)workspace % 256) { set_error("h, logits 16-byte, workspace 256-byte aligned"); return PT_ERR_MISALIGNED; }
    size_t need = 0;
    pt_lm_workspace_bytes(m, n, &need);
    if (ws_bytes < need) { set_error("workspace: %zu < %zu bytes", ws_bytes, need); return PT_ERR_BUFFER_TOO_SMALL; }
    const int H = m->cfg.hidden, V = m->lm_vocab;
    if (H < 64) { set_error("hidden must be at least 64"); return PT_ERR_UNSUPPORTED; }
    cudaStream_t st = (cudaStream_t)stream;
    LmLayout l = lm_layout(m, V);
    __nv_bfloat16* hn = (__nv_bfloat16*)workspace;
    k_final_norm<<<(unsigned)((n * 32 + 255) / 256), 256, 0, st>>>(h, row_stride, (const float*)(m->lm_buf + l.off_gain), hn, n, H, m->cfg.rms_eps);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    const int bn = gemm_bn(V, (int)n, 1, EPI_PLAIN);
    CUtensorMap ta, tb;
    const int kps = gemm_kps(bn, (int)n, H, 1);
    const bool pair = gemm_pair_ok(bn, (int)n, V, 1);
    if ((s = make_a_map(&ta, hn, H, n, 1, kps)) != PT_OK) return s;
    if ((s = make_w_map(&tb, m->lm_buf + l.off_head, H, V, 1, pair ? 128 : bn, kps)) != PT_OK) return s;
    GemmP p{};
    p.kps = kps; p.pair = pair;
    p.M = (int)n; p.N = V; p.K = H; p.T = 1; p.kt = 1; p.status = m->status(); p.c_out = logits; p.scale = 1.f; p.n_sum = 1; p.n_out = 1;
    if ((s = launch_gemm(EPI_PLAIN, bn, ta, tb, p, st)) != PT_OK) return s;
    if (next_token) {
        k_argmax<<<(unsigned)n, 256, 0, st>>>(logits, V, next_token, nullptr, 0);
        g_launches.fetch_add(1, std::memory_order_relaxed);
    }
    LM_CUDA(cudaGetLastError());
    return PT_OK;
}


/* Workspace of pt_generate: the forward workspace first, then the embedded inputs, the forward's output,
 * the normalised rows for the LM head, one step's logits and the current tokens. */
static size_t gen_carve(const pt_model* m, int32_t B, int32_t S, int32_t page_size, char* base,
                        char** fwd, size_t* fwd_bytes, char** x, char** h, char** hn, char** logits, char** tok) {
    size_t off = 0;
    auto take = [&](size_t b) { size_t o = off; off += align_up(b, 256); return base ? base + o : nullptr; };
    size_t fb = 0;
    pt_workspace_bytes(m, (int64_t)B * S, B, page_size, &fb);
    size_t fb1 = 0;
    pt_workspace_bytes(m, B, B, page_size, &fb1);
    fb = std::max(fb, fb1);
    char* f = (char*)take(fb);
    char* xx = (char*)take((size_t)B * S * m->cfg.hidden * 2);
    char* hh = (char*)take((size_t)B * S * m->cfg.hidden * 4);
    char* nn = (char*)take((size_t)B * m->cfg.hidden * 2);
    char* lg = (char*)take((size_t)B * m->lm_vocab * 4);
    char* tk = (char*)take((size_t)B * 4);
    if (fwd) { *fwd = f; *fwd_bytes = fb; *x = xx; *h = hh; *hn = nn; *logits = lg; *tok = tk; }
    return off;
}

pt_status pt_generate_workspace_bytes(const pt_model* m, int32_t B, int32_t S, int32_t page_size, size_t* bytes) {
    pt_status s = lm_check(m);
    if (s != PT_OK) return s;
    if (!bytes || B < 1 || S < 1) { set_error("bad argument"); return PT_ERR_INVALID_ARG; }
    *bytes = gen_carve(m, B, S, page_size, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr);
    return PT_OK;
}

pt_status pt_generate(pt_model* m, pt_kv_cache* c, const int32_t* dev_prompt, int32_t B, int32_t S, int32_t n_new,
                      const int32_t* seq_ids, int32_t* dev_tokens_out, float* dev_logits_out,
                      void* workspace, size_t ws_bytes, void* stream) {
    pt_status s = lm_check(m);
    if (s != PT_OK) return s;
    if (!c || !dev_prompt || !seq_ids || !dev_tokens_out || !workspace || B < 1 || S < 1 || n_new < 1) { set_error("bad argument"); return PT_ERR_INVALID_ARG; }
    if ((uintptr_t)workspace % 256) { set_error("workspace must be 256-byte aligned"); return PT_ERR_MISALIGNED; }
    if (c->kv_dtype != PT_KV_MODEL) { set_error("pt_generate sizes its workspace for a cache in the model dtype: drive pt_prefill / pt_decode_step directly with an E4M3 cache"); return PT_ERR_UNSUPPORTED; }
    char *fwd, *x, *h, *hn, *logits, *tok;
    size_t fwd_bytes;
    size_t need = gen_carve(m, B, S, c->ps, (char*)workspace, &fwd, &fwd_bytes, &x, &h, &hn, &logits, &tok);
    if (ws_bytes < need) { set_error("workspace: %zu < %zu bytes", ws_bytes, need); return PT_ERR_BUFFER_TOO_SMALL; }
    cudaStream_t st = (cudaStream_t)stream;
    const int H = m->cfg.hidden, V = m->lm_vocab;
    const size_t hn_bytes = align_up((size_t)B * H * 2, 256);
    // prompt: every track starts from the same embedding (track stride 0); the next token comes from the
    // last position of every sequence
    if ((s = pt_embed(m, dev_prompt, (int64_t)B * S, x, stream)) != PT_OK) return s;
    if ((s = pt_prefill(m, c, x, 0, B, S, seq_ids, h, fwd, fwd_bytes, stream)) != PT_OK) return s;
    if ((s = pt_lm_head(m, (const float*)h + (size_t)(S - 1) * H, (int64_t)S * H, B, (float*)logits, nullptr, hn, hn_bytes, stream)) != PT_OK) return s;
    for (int i = 0; i < n_new; ++i) {
        k_argmax<<<B, 256, 0, st>>>((const float*)logits, V, (int32_t*)tok, dev_tokens_out + i, n_new);
        g_launches.fetch_add(1, std::memory_order_relaxed);
        if (dev_logits_out)
            LM_CUDA(cudaMemcpy2DAsync(dev_logits_out + (size_t)i * V, (size_t)n_new * V * 4, logits, (size_t)V * 4, (size_t)V * 4, B, cudaMemcpyDeviceToDevice, st));
        if (i + 1 == n_new) break;
        if ((s = pt_embed(m, (const int32_t*)tok, B, x, stream)) != PT_OK) return s;
        if ((s = pt_decode_step(m, c, x, 0, B, seq_ids, h, fwd, fwd_bytes, stream)) != PT_OK) return s;
        if ((s = pt_lm_head(m, (const float*)h, H, B, (float*)logits, nullptr, hn, hn_bytes, stream)) != PT_OK) return s;
    }
    LM_CUDA(cudaGetLastError());
    return PT_OK;
}

}  // extern "C"
