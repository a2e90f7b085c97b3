// Forward pass of the bf16 tensor-core path: five launches per layer for all tracks at once
// (QKV GEMM, attention, output-projection GEMM, gate/up GEMM, down GEMM); the track-sync of
// Algorithm 1 is the down GEMM of every D-th layer run with its K loop over (track, k).
#include "pt_tc.h"

namespace pt {

namespace {

// x (bf16) -> fp32 residual stream, gain-scaled bf16 GEMM operand, partial sums of squares.
// One warp per (row, track).
__global__ void k_tc_prep(const __nv_bfloat16* __restrict__ x, int64_t x_stride, const float* __restrict__ gain,
                          float* __restrict__ h, __nv_bfloat16* __restrict__ hb, float* __restrict__ ssq,
                          int M, int H, int tiles) {
    int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    int t = blockIdx.y;
    if (warp >= M) return;
    const __nv_bfloat16* xr = x + (size_t)t * x_stride + (size_t)warp * H;
    size_t ro = ((size_t)t * M + warp) * H;
    // 128 columns per pass: lanes 0-15 cover one kSsqTile-column group, lanes 16-31 the next
    for (int g = 0; g * 128 < H; ++g) {
        int c = g * 128 + lane * 4;
        float s = 0.f;
        if (c < H) {
            uint2 raw = *reinterpret_cast<const uint2*>(xr + c);
            __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&raw.x), b = *reinterpret_cast<__nv_bfloat162*>(&raw.y);
            float v0 = __low2float(a), v1 = __high2float(a), v2 = __low2float(b), v3 = __high2float(b);
            *reinterpret_cast<float4*>(h + ro + c) = make_float4(v0, v1, v2, v3);
            float4 gn = *reinterpret_cast<const float4*>(gain + (size_t)t * H + c);
            __nv_bfloat162 o0 = __floats2bfloat162_rn(v0 * gn.x, v1 * gn.y), o1 = __floats2bfloat162_rn(v2 * gn.z, v3 * gn.w);
            uint2 ov;
            ov.x = *reinterpret_cast<uint32_t*>(&o0); ov.y = *reinterpret_cast<uint32_t*>(&o1);
            *reinterpret_cast<uint2*>(hb + ro + c) = ov;
            s = v0 * v0 + v1 * v1 + v2 * v2 + v3 * v3;
        }
        for (int o = 8; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        int tile = g * 2 + (lane >> 4);
        if ((lane & 15) == 0 && tile < tiles) ssq[((size_t)t * M + warp) * tiles + tile] = s;
    }
}

// Track-sync outside a GEMM epilogue: h = scale * sum of T input streams in order, the synced stream, the
// gain-scaled bf16 operand of each of the T_out tracks that continue from it and the partial sums of
// squares.  One warp per (row, 128-column group), so a single decoded row still spreads over H / 128 warps.
// Used for a decode step's few rows and after the all-reduce of a track group.  (With few rows the
// K-concatenated sync GEMM would run on N/128 CTAs only; the per-track down GEMM fills the machine and this
// kernel finishes the reduction.)
__global__ void k_track_sync(const float* __restrict__ hT, size_t tstride, int T, int T_out, float scale,
                             float* __restrict__ h_out, __nv_bfloat16* __restrict__ hb, const float* __restrict__ gain,
                             float* __restrict__ ssq, int M, int H, int tiles) {
    grid_dep_wait();              // a dependent launch: the GEMM after it may fetch its first weight tiles while this runs
    grid_dep_launch();
    const int groups = (H + 127) / 128;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= M * groups) return;
    const int row = warp / groups, g = warp % groups;
    const size_t ro = (size_t)row * H;
    const int c = g * 128 + lane * 4;
    float s = 0.f;
    if (c < H) {
        float4 a = *reinterpret_cast<const float4*>(hT + ro + c);
#pragma unroll 4
        for (int t = 1; t < T; ++t) {
            float4 b = *reinterpret_cast<const float4*>(hT + (size_t)t * tstride + ro + c);
            a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
        }
        a.x *= scale; a.y *= scale; a.z *= scale; a.w *= scale;
        *reinterpret_cast<float4*>(h_out + ro + c) = a;
        s = a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w;
        if (hb) {
            for (int t = 0; t < T_out; ++t) {
                float4 gn = *reinterpret_cast<const float4*>(gain + (size_t)t * H + c);
                __nv_bfloat162 o0 = __floats2bfloat162_rn(a.x * gn.x, a.y * gn.y), o1 = __floats2bfloat162_rn(a.z * gn.z, a.w * gn.w);
                uint2 ov;
                ov.x = *reinterpret_cast<uint32_t*>(&o0); ov.y = *reinterpret_cast<uint32_t*>(&o1);
                *reinterpret_cast<uint2*>(hb + (size_t)t * M * H + ro + c) = ov;
            }
        }
    }
    for (int o = 8; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const int tile = g * 2 + (lane >> 4);
    if (ssq && (lane & 15) == 0 && tile < tiles) ssq[(size_t)row * tiles + tile] = s;
}

// Asks L2 for `bytes` bytes from `base` (128-byte lines, a grid-stride loop of prefetch hints: nothing is read into the SM).
__global__ void k_l2_prefetch(const char* __restrict__ base, size_t bytes) {
    const size_t lines = (bytes + 127) / 128;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < lines; i += (size_t)gridDim.x * blockDim.x)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(base + i * 128));
}

// PT-MoE routing weights of one layer: one warp per (token, track).  The normalised stream is the gain-scaled bf16
// copy times 1/rms (the operand the gate/up GEMM sees); the router itself is fp32.  logits[e] = c . Wr[e]; the top_k
// largest logits (the lower index wins a tie) get softmax weights among themselves, every other expert 0.
__global__ void k_moe_route(const __nv_bfloat16* __restrict__ hb, const float* __restrict__ ssq, int tiles, float eps,
                            const float* __restrict__ wr, float* __restrict__ gates, int M, int H, int E, int top_k) {
    grid_dep_wait();
    grid_dep_launch();
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    const int t = blockIdx.y;
    if (warp >= M) return;
    const size_t row = (size_t)t * M + warp;
    float ss = 0.f;
    for (int i = lane; i < tiles; i += 32) ss += ssq[row * tiles + i];
#pragma unroll
    for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    const float rinv = 1.0f / sqrtf(ss / (float)H + eps);
    float logit[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) logit[e] = 0.f;
    const __nv_bfloat16* hr = hb + row * H;
    const float* w = wr + (size_t)t * E * H;
    for (int c = lane * 2; c < H; c += 64) {
        const float2 hv = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(hr + c));
#pragma unroll
        for (int e = 0; e < 16; ++e)
            if (e < E) {
                const float2 wv = *reinterpret_cast<const float2*>(w + (size_t)e * H + c);
                logit[e] = fmaf(hv.x, wv.x, fmaf(hv.y, wv.y, logit[e]));
            }
    }
#pragma unroll
    for (int e = 0; e < 16; ++e) {
#pragma unroll
        for (int o = 16; o; o >>= 1) logit[e] += __shfl_xor_sync(0xffffffffu, logit[e], o);
        logit[e] *= rinv;
    }
    // every lane holds all logits: choose top_k (lowest index among equals first), softmax over the chosen
    unsigned chosen = 0;
    float top = 0.f;
    for (int k = 0; k < top_k; ++k) {
        int best = -1;
        float bv = 0.f;
#pragma unroll
        for (int e = 0; e < 16; ++e)
            if (e < E && !((chosen >> e) & 1u) && (best < 0 || logit[e] > bv)) { best = e; bv = logit[e]; }
        chosen |= 1u << best;
        if (k == 0) top = bv;
    }
    float sum = 0.f, wgt[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) { wgt[e] = ((chosen >> e) & 1u) ? __expf(logit[e] - top) : 0.f; sum += wgt[e]; }
    const float inv = 1.0f / sum;
    float mine = 0.f;
#pragma unroll
    for (int e = 0; e < 16; ++e) mine = lane == e ? wgt[e] * inv : mine;
    if (lane < E) gates[row * E + lane] = mine;
}

inline int kps_index(int kps) { return kps == 4 ? 2 : (kps == 2 ? 1 : 0); }

}  // namespace

pt_status tc_build_weight_maps(pt_model* m) {
    const pt_config& c = m->cfg;
    if (c.hidden < 64 || c.ffn < 64) { set_error("the tensor-core path needs hidden >= 64 and ffn >= 64"); return PT_ERR_UNSUPPORTED; }
    std::vector<WMaps> v(c.L);
    const __nv_bfloat16* wqkv = (const __nv_bfloat16*)(m->wbuf + m->off_wqkv);
    const __nv_bfloat16* wo = (const __nv_bfloat16*)(m->wbuf + m->off_wo);
    const __nv_bfloat16* wgu = (const __nv_bfloat16*)(m->wbuf + m->off_wgu);
    const __nv_bfloat16* wd = (const __nv_bfloat16*)(m->wbuf + m->off_wd);
    for (int l = 0; l < c.L; ++l)
        for (int b = 0; b < 3; ++b)
            for (int kp = 0; kp < 3; ++kp) {
                const int bn = 64 << b, kps = 1 << kp;
                if (bn * kps > 256) continue;
                const void* base[4] = {wqkv + (size_t)l * m->wqkv_layer(), wo + (size_t)l * m->wo_layer(),
                                       wgu + (size_t)l * m->wgu_layer(), wd + (size_t)l * m->wd_layer()};
                const int64_t kk[4] = {c.hidden, m->QD, c.hidden, m->Ftot}, nn[4] = {m->Nqkv, c.hidden, 2 * m->Ftot, c.hidden};
                for (int i = 0; i < 4; ++i) {
                    if (kps > 1 && (kk[i] % 64 || (kk[i] / 64) % kps)) continue;
                    pt_status s = make_w_map(&v[l].m[i][b][kp], base[i], kk[i], nn[i], c.T, bn, kps);
                    if (s != PT_OK) return s;
                }
            }
    m->wmaps = std::move(v);
    return PT_OK;
}

pt_status tc_forward(Call& k) {
    pt_model* m = k.m;
    pt_kv_cache* c = k.c;
    const pt_config& g = m->cfg;
    const int T = g.T, M = k.M, H = g.hidden, F = m->Ftot;        // with experts: all of a track's experts side by side
    const size_t MH = (size_t)M * H;
    cudaStream_t st = k.st;
    Work& w = k.w;
    if ((int)m->wmaps.size() != g.L) { set_error("weights not bound"); return PT_ERR_STATE; }
    const std::vector<WMaps>& wm = m->wmaps;
    const bool fp8 = c->kv_dtype == PT_KV_E4M3;       // K and V go through a bf16 staging area into 8-bit codes
    __nv_bfloat16* pool = (__nv_bfloat16*)c->pool;
    const int64_t pool_tstride = (int64_t)g.L * c->slab_elems;
    const int tiles = (H + kSsqTile - 1) / kSsqTile;
    __nv_bfloat16* hb = (__nv_bfloat16*)w.a;
    __nv_bfloat16* q = (__nv_bfloat16*)w.qkv;
    __nv_bfloat16* o = (__nv_bfloat16*)w.o;
    __nv_bfloat16* z = (__nv_bfloat16*)w.z;

    // A operands (normalised stream, attention output, SwiGLU output): one map per copy shape a GEMM of this call uses
    struct AMaps { CUtensorMap m[3]; bool have[3] = {false, false, false}; } ta_h, ta_o, ta_z;
    pt_status s;
    auto a_map = [&](AMaps& am, const void* base, int64_t kk, int kps, const CUtensorMap** out) -> pt_status {
        const int i = kps_index(kps);
        if (!am.have[i]) {
            pt_status r = make_a_map(&am.m[i], base, kk, M, T, kps);
            if (r != PT_OK) return r;
            am.have[i] = true;
        }
        *out = &am.m[i];
        return PT_OK;
    };
    const CUtensorMap* ta = nullptr;

    { ProfScope ps(m, st, 6);
    k_tc_prep<<<dim3((M * 32 + 255) / 256, T), 256, 0, st>>>((const __nv_bfloat16*)k.x, k.x_stride, m->gain(0, 0), w.hT, hb, w.ssq, M, H, tiles);
    g_launches.fetch_add(1, std::memory_order_relaxed); }

    const float* hin = w.hT;
    size_t hin_stride = MH;
    size_t ssq_tstride = (size_t)M * tiles;
    for (int l = 0; l < g.L; ++l) {
        __nv_bfloat16* pool_l = pool + (size_t)l * c->slab_elems;
        GemmP base{};
        base.M = M; base.status = m->status(); base.eps = g.rms_eps; base.kt = 1; base.T = T;
        base.scale = 1.0f; base.n_sum = 1; base.n_out = 1; base.w_static = 1;
        {   // QKV: RMSNorm-1 scale, RoPE, KV append
            GemmP p = base;
            p.N = m->Nqkv; p.K = H;
            p.ssq_in = w.ssq; p.ssq_in_tstride = ssq_tstride; p.ssq_tiles = tiles;
            p.q_out = q; p.pool_l = pool_l; p.pool_tstride = pool_tstride; p.slab_elems = c->slab_elems;
            p.row_kvoff = w.meta.row_kvoff; p.row_pos = w.meta.row_pos; p.cs = m->rope_cos(); p.sn = m->rope_sin(); p.cs16 = m->rope_cs16();
            p.nq = g.heads; p.nkv = g.kv_heads; p.dh = m->dh; p.ps = c->ps;
            if (fp8) {          // the staging area looks like one page of M slots: [K|V][kv_head][row][dh] per track
                p.pool_l = (__nv_bfloat16*)w.kv_stage; p.pool_tstride = (int64_t)2 * m->KVD * M; p.slab_elems = (int64_t)2 * m->KVD * M;
                p.row_kvoff = w.meta.row_stageoff; p.ps = M;
            }
            int bn = gemm_bn(p.N, M, T, EPI_QKV);
            p.kps = gemm_kps(bn, M, p.K, 1);
            p.pair = gemm_pair_ok(bn, M, p.N, p.T);
            if ((s = a_map(ta_h, hb, H, p.kps, &ta)) != PT_OK) return s;
            ProfScope ps(m, st, 1);
            if ((s = launch_gemm(EPI_QKV, bn, *ta, wm[l].m[0][bn_index(p.pair ? 128 : bn)][kps_index(p.kps)], p, st)) != PT_OK) return s;
        }
        if (fp8) {
            ProfScope ps(m, st, 6);
            if (!k.decode && (s = launch_kv_dequant_ctx(k, l)) != PT_OK) return s;
            if ((s = launch_kv_quant(k, l)) != PT_OK) return s;
        }
        {
            ProfScope ps(m, st, 0);
            if (fp8) s = k.decode ? launch_decode_attn_e4m3(k, q, l, o) : launch_flash_prefill_e4m3(k, q, o);
            else if (k.decode) s = launch_decode_attn(k, q, pool_l, o);
            else s = launch_flash_prefill(k, q, pool_l, o);
        }
        if (s != PT_OK) return s;
        {   // output projection + residual; emits the operand and statistics of RMSNorm-2
            GemmP p = base;
            p.N = H; p.K = m->QD;
            p.h_in = hin; p.h_in_tstride = hin_stride; p.h_out = w.hT; p.h_out_tstride = MH;
            p.hb_out = hb; p.gain = m->gain(1, l);
            p.ssq_out = w.ssq; p.ssq_out_tstride = (size_t)M * tiles; p.ssq_out_tiles = tiles;
            int bn = gemm_bn(p.N, M, T, EPI_RESID);
            p.kps = gemm_kps(bn, M, p.K, 1);
            p.pair = gemm_pair_ok(bn, M, p.N, p.T);
            if ((s = a_map(ta_o, o, m->QD, p.kps, &ta)) != PT_OK) return s;
            ProfScope ps(m, st, 2);
            if ((s = launch_gemm(EPI_RESID, bn, *ta, wm[l].m[1][bn_index(p.pair ? 128 : bn)][kps_index(p.kps)], p, st)) != PT_OK) return s;
            ssq_tstride = (size_t)M * tiles;
        }
        tap_copy(k, l, 0, w.hT, MH);
        if (m->E) {   // PT-MoE: the routing weights of this layer, from the operand and statistics the out-projection just wrote
            ProfScope ps(m, st, 6);
            launch_dependent(k_moe_route, dim3((M * 32 + 255) / 256, T), dim3(256), (size_t)0, st, (const __nv_bfloat16*)hb, (const float*)w.ssq, tiles,
                             g.rms_eps, m->router(l), w.gates, M, H, m->E, g.top_k);
            g_launches.fetch_add(1, std::memory_order_relaxed);
        }
        if (moe_sparse_ok(m, M, k.decode)) {   // PT-MoE on permuted tokens: only the chosen experts are evaluated
            const bool sync = (l + 1) % g.D == 0, last = l + 1 == g.L;
            float* ho = last ? k.out : w.hS;
            const float sync_scale = g.sync_op ? 1.0f / (float)T : 1.0f;
            if ((s = moe_sparse_ffn(k, l, sync, last, sync_scale, w.hT, MH, sync ? ho : w.hT, sync ? 0 : MH)) != PT_OK) return s;
            if (sync) { ssq_tstride = 0; hin = ho; hin_stride = 0; }
            else { ssq_tstride = (size_t)M * tiles; hin = w.hT; hin_stride = MH; }
            tap_copy(k, l, 1, hin, hin_stride);
            continue;
        }
        {   // gate/up + SwiGLU (PT-MoE: every expert's, each column block weighted by its expert's routing weight)
            GemmP p = base;
            p.N = 2 * F; p.K = H;
            p.gates = w.gates; p.n_experts = m->E; p.expert_cols = 2 * g.ffn;
            p.ssq_in = w.ssq; p.ssq_in_tstride = ssq_tstride; p.ssq_tiles = tiles;
            p.z_out = z;
            int bn = gemm_bn(p.N, M, T, EPI_SWIGLU);
            p.kps = gemm_kps(bn, M, p.K, 1);
            p.pair = gemm_pair_ok(bn, M, p.N, p.T);
            if ((s = a_map(ta_h, hb, H, p.kps, &ta)) != PT_OK) return s;
            ProfScope ps(m, st, 3);
            if ((s = launch_gemm(EPI_SWIGLU, bn, *ta, wm[l].m[2][bn_index(p.pair ? 128 : bn)][kps_index(p.kps)], p, st)) != PT_OK) return s;
        }
        {   // down projection + residual (+ track-sync when the layer closes a track block)
            const bool sync = (l + 1) % g.D == 0, last = l + 1 == g.L;
            GemmP p = base;
            p.N = H; p.K = F;
            p.h_in = w.hT; p.h_in_tstride = MH;
            if (!last) { p.hb_out = hb; p.gain = m->gain(0, l + 1); p.ssq_out = w.ssq; p.ssq_out_tiles = tiles; }
            // a decode step (few rows): per-track down GEMM on the whole machine, then a small reduction kernel;
            // many rows (prefill): one GEMM whose K loop runs over (track, k) and whose epilogue is the sync
            const bool split_sync = sync && k.decode && M <= 256;
            const bool grouped = sync && m->ar_fn != nullptr;          // tracks of other ranks join through an all-reduce
            const float sync_scale = g.sync_op ? 1.0f / (float)(grouped ? m->world_tracks : T) : 1.0f;
            if (sync && !split_sync) {
                p.T = 1; p.kt = T; p.n_sum = T; p.n_out = T;
                p.scale = grouped ? 1.0f : sync_scale;
                p.h_out = (last && !grouped) ? k.out : w.hS; p.h_out_tstride = 0;
                p.ssq_out_tstride = 0;
                if (grouped) { p.hb_out = nullptr; p.ssq_out = nullptr; }
            } else {
                p.h_out = w.hT; p.h_out_tstride = MH;
                p.ssq_out_tstride = (size_t)M * tiles;
                if (split_sync) { p.hb_out = nullptr; p.ssq_out = nullptr; }
            }
            int bn = gemm_bn(p.N, M, p.T, EPI_RESID);
            p.kps = gemm_kps(bn, M, p.K, p.kt);
            p.pair = gemm_pair_ok(bn, M, p.N, p.T);
            if ((s = a_map(ta_z, z, F, p.kps, &ta)) != PT_OK) return s;
            ProfScope ps(m, st, sync ? 5 : 4);
            if ((s = launch_gemm(EPI_RESID, bn, *ta, wm[l].m[3][bn_index(p.pair ? 128 : bn)][kps_index(p.kps)], p, st)) != PT_OK) return s;
            float* ho = last ? k.out : w.hS;
            __nv_bfloat16* hb_next = last ? nullptr : hb;
            const float* gain_next = last ? nullptr : m->gain(0, l + 1);
            float* ssq_next = last ? nullptr : w.ssq;
            const unsigned sync_grid = (unsigned)(((size_t)M * ((H + 127) / 128) * 32 + 255) / 256);
            if (split_sync) {       // local tracks -> one stream (the final one unless other ranks still have to join)
                launch_dependent(k_track_sync, dim3(sync_grid), dim3(256), (size_t)0, st, (const float*)w.hT, MH, T, T, grouped ? 1.0f : sync_scale,
                                 grouped ? w.hS : ho, grouped ? (__nv_bfloat16*)nullptr : hb_next, grouped ? (const float*)nullptr : gain_next,
                                 grouped ? (float*)nullptr : ssq_next, M, H, tiles);
                g_launches.fetch_add(1, std::memory_order_relaxed);
            }
            if (grouped) {
                // w.hS holds this rank's partial sum: one all-reduce per track block, then every local track's
                // next operand from the total.  While the all-reduce runs on the call's stream, a side stream pulls the
                // weights of the next layer's QKV projection (at most 48 MB of them) into L2, so that the first GEMM of
                // the next track block does not start from HBM latency: the side stream only waits for the sync GEMM
                // (an event), nothing waits for it.
                if (!last) {
                    if (!m->side_stream && (cudaStreamCreateWithFlags(&m->side_stream, cudaStreamNonBlocking) != cudaSuccess ||
                                            cudaEventCreateWithFlags(&m->side_event, cudaEventDisableTiming) != cudaSuccess)) {
                        set_error("side stream for the weight prefetch: %s", cudaGetErrorString(cudaGetLastError()));
                        return PT_ERR_CUDA;
                    }
                    const size_t wbytes = std::min<size_t>(m->wqkv_layer() * 2, (size_t)48 << 20);
                    cudaEventRecord(m->side_event, st);
                    cudaStreamWaitEvent(m->side_stream, m->side_event, 0);
                    k_l2_prefetch<<<148, 256, 0, m->side_stream>>>(m->wbuf + m->off_wqkv + (size_t)(l + 1) * m->wqkv_layer() * 2, wbytes);
                    g_launches.fetch_add(1, std::memory_order_relaxed);
                }
                if (m->ar_fn(m->ar_user, w.hS, (int64_t)M * H, (void*)st) != 0) { set_error("the all-reduce hook failed at layer %d", l); return PT_ERR_CUDA; }
                launch_dependent(k_track_sync, dim3(sync_grid), dim3(256), (size_t)0, st, (const float*)w.hS, (size_t)0, 1, T, sync_scale, ho, hb_next,
                                 gain_next, ssq_next, M, H, tiles);
                g_launches.fetch_add(1, std::memory_order_relaxed);
            }
            if (sync) { ssq_tstride = 0; hin = ho; hin_stride = 0; }
            else { ssq_tstride = (size_t)M * tiles; hin = w.hT; hin_stride = MH; }
        }
        tap_copy(k, l, 1, hin, hin_stride);
    }
    if (m->ar_fn && m->side_stream) {      // the call's stream ends after the side stream's last prefetch: a wait on it covers both
        cudaEventRecord(m->side_event, m->side_stream);
        cudaStreamWaitEvent(st, m->side_event, 0);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("kernel launch failed: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
    return PT_OK;
}

}  // namespace pt

#include "pt_kernels.h"

extern "C" pt_status pt_kernel_gemm_bf16(const void* a, const void* w, void* c, int32_t T, int32_t M, int32_t N,
                                         int32_t K, int32_t bn, int32_t fold_tracks, void* status, void* stream) {
    using namespace pt;
    if (!a || !w || !c || !status) { set_error("null argument"); return PT_ERR_INVALID_ARG; }
    if (T < 1 || M < 1 || N < 16 || N % 16 || K < 64 || K % 8) { set_error("unsupported GEMM shape"); return PT_ERR_INVALID_ARG; }
    if (bn == 0) bn = gemm_bn(N, M, fold_tracks ? 1 : T, EPI_PLAIN);
    if (bn != 64 && bn != 128 && bn != 256) { set_error("bn must be 0, 64, 128 or 256"); return PT_ERR_INVALID_ARG; }
    CUtensorMap ta, tb;
    pt_status s;
    const int kps = gemm_kps(bn, M, K, fold_tracks ? T : 1);
    const bool pair = gemm_pair_ok(bn, M, N, fold_tracks ? 1 : T);
    if ((s = make_a_map(&ta, a, K, M, T, kps)) != PT_OK) return s;
    if ((s = make_w_map(&tb, w, K, N, T, pair ? 128 : bn, kps)) != PT_OK) return s;
    GemmP p{};
    p.M = M; p.N = N; p.K = K; p.T = fold_tracks ? 1 : T; p.kt = fold_tracks ? T : 1; p.kps = kps; p.pair = pair;
    p.status = (int*)status; p.c_out = (float*)c; p.scale = 1.f; p.n_sum = 1; p.n_out = 1;
    if ((s = launch_gemm(EPI_PLAIN, bn, ta, tb, p, (cudaStream_t)stream)) != PT_OK) return s;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("kernel launch failed: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
    return PT_OK;
}

namespace pt {

// Scratch layout of the kernel-level decode attention: plan first, partials after.
struct DecodeScratch { size_t o_items, o_nsplit, o_len, o_part, total; };
static DecodeScratch decode_scratch_layout(int T, int B, int nq, int dh) {
    DecodeScratch d{};
    size_t off = 0;
    auto take = [&](size_t b) { size_t o = off; off += align_up(b, 256); return o; };
    d.o_items = take((size_t)B * kMaxSplits * 16);
    d.o_nsplit = take((size_t)B * 4);
    d.o_len = take((size_t)B * 4);
    d.o_part = take((size_t)T * B * kMaxSplits * nq * (dh + 2) * 4);
    d.total = off;
    return d;
}

// Shared by the caller-scratch and the static-scratch entry points.
pt_status decode_attn_with_scratch(const void* q, const void* pool_l, int64_t pool_track_stride,
                                   const int32_t* block_table, int32_t maxp, const int32_t* kv_len,
                                   int32_t T, int32_t B, int32_t nq, int32_t nkv, int32_t dh, int32_t ps,
                                   int32_t num_pages, void* out, char* scratch, void* status, cudaStream_t st) {
    DecodeScratch d = decode_scratch_layout(T, B, nq, dh);
    std::vector<int32_t> host((d.o_part) / 4, 0);
    int32_t* items = host.data() + d.o_items / 4;
    int32_t* nsplit = host.data() + d.o_nsplit / 4;
    int32_t* lens = host.data() + d.o_len / 4;
    for (int b = 0; b < B; ++b) lens[b] = kv_len[b];
    int n_items = 0, max_splits = 1;
    plan_decode_splits(lens, B, ps, (int64_t)T * nkv, items, nsplit, &n_items, &max_splits);
    cudaError_t e = cudaMemcpyAsync(scratch, host.data(), d.o_part, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) { set_error("cudaMemcpyAsync: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
    AttnP p{};
    p.q = (const __nv_bfloat16*)q; p.pool_l = (const __nv_bfloat16*)pool_l; p.pool_tstride = pool_track_stride;
    p.o = (__nv_bfloat16*)out; p.bt = block_table; p.maxp = maxp; p.kvlen = (const int32_t*)(scratch + d.o_len);
    p.B = B; p.S = 1; p.M = B; p.nq = nq; p.nkv = nkv; p.ps = ps; p.num_pages = num_pages;
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)dh);
    p.status = (int*)status;
    p.items = (const int32_t*)(scratch + d.o_items); p.nsplit = (const int32_t*)(scratch + d.o_nsplit);
    p.part = (float*)(scratch + d.o_part); p.max_splits = kMaxSplits;
    pt_status s = launch_decode_attn_p(p, T, dh, n_items, max_splits, st);
    if (s != PT_OK) return s;
    e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("kernel launch failed: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
    return PT_OK;
}

pt_status decode_attn_check_args(const void* q, const void* pool_l, const int32_t* block_table, int32_t maxp,
                                 const int32_t* kv_len, int32_t T, int32_t B, int32_t nq, int32_t nkv, int32_t dh,
                                 int32_t ps, int32_t num_pages, const void* out, const void* status) {
    if (!q || !pool_l || !block_table || !kv_len || !out || !status) { set_error("null argument"); return PT_ERR_INVALID_ARG; }
    if (T < 1 || B < 1 || nq < 1 || nkv < 1 || nq % nkv || nq / nkv > 8 || maxp < 1 || num_pages < 1) { set_error("bad sizes"); return PT_ERR_INVALID_ARG; }
    if (dh != 32 && dh != 64 && dh != 128) { set_error("head_dim %d not in {32, 64, 128}", dh); return PT_ERR_UNSUPPORTED; }
    if (ps < 8 || ps > 64 || ps % 8) { set_error("page size must be a multiple of 8 in [8, 64]"); return PT_ERR_INVALID_ARG; }
    for (int b = 0; b < B; ++b)
        if (kv_len[b] < 1 || (int64_t)kv_len[b] > (int64_t)maxp * ps) { set_error("kv_len[%d] = %d outside [1, maxp*ps]", b, kv_len[b]); return PT_ERR_INVALID_ARG; }
    return PT_OK;
}

}  // namespace pt

extern "C" pt_status pt_kernel_prefill_attn(const void* q, const void* pool_l, int64_t pool_track_stride,
                                            const int32_t* block_table, int32_t maxp, const int32_t* kv_len,
                                            int32_t T, int32_t B, int32_t S, int32_t nq, int32_t nkv, int32_t dh, int32_t ps,
                                            int32_t num_pages, void* out, int32_t impl, void* status, void* stream) {
    using namespace pt;
    if (!q || !pool_l || !block_table || !kv_len || !out || !status) { set_error("null argument"); return PT_ERR_INVALID_ARG; }
    if (T < 1 || B < 1 || S < 1 || nq < 1 || nkv < 1 || nq % nkv || maxp < 1 || num_pages < 1 || (int64_t)B * S > (1 << 30)) { set_error("bad sizes"); return PT_ERR_INVALID_ARG; }
    if (dh != 32 && dh != 64 && dh != 128) { set_error("head_dim %d not in {32, 64, 128}", dh); return PT_ERR_UNSUPPORTED; }
    if (ps < 8 || ps > 64 || ps % 8) { set_error("page size must be a multiple of 8 in [8, 64]"); return PT_ERR_INVALID_ARG; }
    if (impl != 0 && impl != 1) { set_error("impl must be 0 or 1"); return PT_ERR_INVALID_ARG; }
    if (impl == 0 && !flash_tc_supported(dh, ps)) { set_error("impl 0 needs head_dim 64 or 128 and pages of a multiple of 16 tokens"); return PT_ERR_UNSUPPORTED; }
    AttnP p{};
    p.q = (const __nv_bfloat16*)q; p.pool_l = (const __nv_bfloat16*)pool_l; p.pool_tstride = pool_track_stride;
    p.o = (__nv_bfloat16*)out; p.bt = block_table; p.maxp = maxp; p.kvlen = kv_len;
    p.B = B; p.S = S; p.M = B * S; p.nq = nq; p.nkv = nkv; p.ps = ps; p.num_pages = num_pages;
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)dh);
    p.status = (int*)status;
    pt_status s = launch_flash_prefill_p(p, T, dh, impl == 1, (cudaStream_t)stream);
    if (s != PT_OK) return s;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("kernel launch failed: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
    return PT_OK;
}

extern "C" pt_status pt_kernel_decode_attn_scratch_bytes(int32_t T, int32_t B, int32_t nq, int32_t dh, size_t* bytes) {
    using namespace pt;
    if (!bytes || T < 1 || B < 1 || nq < 1 || dh < 1) { set_error("bad argument"); return PT_ERR_INVALID_ARG; }
    *bytes = decode_scratch_layout(T, B, nq, dh).total;
    return PT_OK;
}

extern "C" pt_status pt_kernel_decode_attn(const void* q, const void* pool_l, int64_t pool_track_stride,
                                           const int32_t* block_table, int32_t maxp, const int32_t* kv_len,
                                           int32_t T, int32_t B, int32_t nq, int32_t nkv, int32_t dh, int32_t ps,
                                           int32_t num_pages, void* out, void* scratch, size_t scratch_bytes,
                                           void* status, void* stream) {
    using namespace pt;
    pt_status s = decode_attn_check_args(q, pool_l, block_table, maxp, kv_len, T, B, nq, nkv, dh, ps, num_pages, out, status);
    if (s != PT_OK) return s;
    if (!scratch) { set_error("null scratch"); return PT_ERR_INVALID_ARG; }
    if ((uintptr_t)scratch % 256) { set_error("scratch must be 256-byte aligned"); return PT_ERR_MISALIGNED; }
    size_t need = decode_scratch_layout(T, B, nq, dh).total;
    if (scratch_bytes < need) { set_error("scratch: %zu < %zu bytes", scratch_bytes, need); return PT_ERR_BUFFER_TOO_SMALL; }
    return decode_attn_with_scratch(q, pool_l, pool_track_stride, block_table, maxp, kv_len, T, B, nq, nkv, dh, ps,
                                    num_pages, out, (char*)scratch, status, (cudaStream_t)stream);
}

extern "C" pt_status pt_kernel_decode_attn_e4m3(const void* q, const void* codes_l, int64_t codes_track_stride,
                                                const float* scales_l, int64_t scales_track_stride,
                                                const int32_t* block_table, int32_t maxp, const int32_t* kv_len,
                                                int32_t T, int32_t B, int32_t nq, int32_t nkv, int32_t ps,
                                                int32_t num_pages, void* out, int32_t impl, void* scratch, size_t scratch_bytes,
                                                void* status, void* stream) {
    using namespace pt;
    const int dh = 128;
    pt_status s = decode_attn_check_args(q, codes_l, block_table, maxp, kv_len, T, B, nq, nkv, dh, ps, num_pages, out, status);
    if (s != PT_OK) return s;
    if (!scales_l || !scratch) { set_error("null argument"); return PT_ERR_INVALID_ARG; }
    if (ps % 16 || nkv > 8) { set_error("an E4M3 cache needs pages of a multiple of 16 tokens and at most 8 KV heads"); return PT_ERR_UNSUPPORTED; }
    if (impl != 0 && impl != 1) { set_error("impl must be 0 or 1"); return PT_ERR_INVALID_ARG; }
    if ((uintptr_t)codes_l % 128 || codes_track_stride % 128 || (uintptr_t)scales_l % 4 || (uintptr_t)scratch % 256) {
        set_error("codes must be 128-byte, scales 4-byte, scratch 256-byte aligned"); return PT_ERR_MISALIGNED;
    }
    DecodeScratch d = decode_scratch_layout(T, B, nq, dh);
    if (scratch_bytes < d.total) { set_error("scratch: %zu < %zu bytes", scratch_bytes, d.total); return PT_ERR_BUFFER_TOO_SMALL; }
    cudaStream_t st = (cudaStream_t)stream;
    std::vector<int32_t> host((d.o_part) / 4, 0);
    int32_t* items = host.data() + d.o_items / 4;
    int32_t* nsplit = host.data() + d.o_nsplit / 4;
    int32_t* lens = host.data() + d.o_len / 4;
    for (int b = 0; b < B; ++b) lens[b] = kv_len[b];
    int n_items = 0, max_splits = 1;
    plan_decode_splits(lens, B, ps, (int64_t)T * nkv, items, nsplit, &n_items, &max_splits);
    cudaError_t e = cudaMemcpyAsync(scratch, host.data(), d.o_part, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) { set_error("cudaMemcpyAsync: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
    char* sc = (char*)scratch;
    AttnP p{};
    p.q = (const __nv_bfloat16*)q; p.o = (__nv_bfloat16*)out; p.bt = block_table; p.maxp = maxp; p.kvlen = (const int32_t*)(sc + d.o_len);
    p.B = B; p.S = 1; p.M = B; p.nq = nq; p.nkv = nkv; p.ps = ps; p.num_pages = num_pages;
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)dh);
    p.status = (int*)status;
    p.items = (const int32_t*)(sc + d.o_items); p.nsplit = (const int32_t*)(sc + d.o_nsplit);
    p.part = (float*)(sc + d.o_part); p.max_splits = kMaxSplits;
    Kv8Slab slab{};
    slab.codes_l = (const uint8_t*)codes_l; slab.codes_tstride = codes_track_stride;
    slab.scales_l = scales_l; slab.scales_tstride = scales_track_stride;
    s = launch_decode_attn_e4m3_p(p, slab, T, n_items, max_splits, impl == 1, st);
    if (s != PT_OK) return s;
    e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("kernel launch failed: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
    return PT_OK;
}

// ---- decode attention with built-in scratch -------------------------------------------------
// The array lives in the library image, once per device that loads it.  In host code its name
// is only a handle: the device address comes from cudaGetSymbolAddress, looked up once per
// device with that device current.
static __device__ __align__(256) unsigned char g_static_scratch[PT_STATIC_SCRATCH_BYTES];

namespace pt {
static void* g_static_scratch_addr[kMaxDevices] = {};
}

extern "C" pt_status pt_kernel_decode_attn_static(const void* q, const void* pool_l, int64_t pool_track_stride,
                                                  const int32_t* block_table, int32_t maxp, const int32_t* kv_len,
                                                  int32_t T, int32_t B, int32_t nq, int32_t nkv, int32_t dh, int32_t ps,
                                                  int32_t num_pages, void* out, void* status, void* stream) {
    using namespace pt;
    pt_status s = decode_attn_check_args(q, pool_l, block_table, maxp, kv_len, T, B, nq, nkv, dh, ps, num_pages, out, status);
    if (s != PT_OK) return s;
    size_t need = decode_scratch_layout(T, B, nq, dh).total;
    if (need > PT_STATIC_SCRATCH_BYTES) {
        set_error("problem needs %zu bytes of scratch, the built-in array holds %u: use pt_kernel_decode_attn with a caller buffer",
                  need, (unsigned)PT_STATIC_SCRATCH_BYTES);
        return PT_ERR_BUFFER_TOO_SMALL;
    }
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) { set_error("cudaGetDevice: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
    if (!g_static_scratch_addr[dev]) {
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess || !ptr) { set_error("cudaGetSymbolAddress: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
        g_static_scratch_addr[dev] = ptr;
    }
    return decode_attn_with_scratch(q, pool_l, pool_track_stride, block_table, maxp, kv_len, T, B, nq, nkv, dh, ps,
                                    num_pages, out, (char*)g_static_scratch_addr[dev], status, (cudaStream_t)stream);
}

extern "C" pt_status pt_kernel_wait_selftest(void* status, uint64_t limit_ns, void* stream) {
    using namespace pt;
    if (!status) { set_error("null status"); return PT_ERR_INVALID_ARG; }
    if (limit_ns < 1000 || limit_ns > 1000000000ull) { set_error("limit_ns must be in [1e3, 1e9]"); return PT_ERR_INVALID_ARG; }
    return launch_wait_selftest((int*)status, (unsigned long long)limit_ns, (cudaStream_t)stream);
}
