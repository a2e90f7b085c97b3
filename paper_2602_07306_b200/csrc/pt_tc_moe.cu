// PT-MoE feed-forward with permuted tokens: every token's row is copied to the row groups of the top_k experts it
// chose, so that the two GEMMs of the feed-forward only multiply tokens with the experts they use - a grouped GEMM
// over (track, expert) whose groups are runs of 128-row tiles of one row space.
//   k_moe_plan      per track: tokens per expert, each expert's first row (a multiple of 128, so a row tile belongs to
//                   one expert), every (token, chosen expert)'s row (token order is kept: deterministic), and the
//                   expert of every row tile
//   k_moe_dispatch  one warp per (token, track): the token's bf16 operand row, its partial sums of squares and its
//                   routing weight to each of its rows
//   gemm_tc         gate/up with the SwiGLU epilogue (the routing weight multiplies z), then the down projection into
//                   fp32 rows; the producer warp shifts the W coordinates by the row tile's expert
//   k_moe_combine   per token: residual + the token's top_k rows, then exactly what the dense path's down-GEMM epilogue
//                   does - the track-sync when the layer closes a block, the next layer's bf16 operand and statistics
// Rows between an expert's last token and its next 128-row boundary hold whatever the buffer held: they are
// multiplied and never read.
#include "pt_tc.h"

namespace pt {

namespace {

__global__ void __launch_bounds__(1024)
k_moe_plan(const float* __restrict__ gates, int M, int E, int tiles_m, int32_t* __restrict__ pos, int32_t* __restrict__ tile_expert) {
    __shared__ int warp_sums[32];
    __shared__ int base_sh, run_sh;
    const int t = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float* g = gates + (size_t)t * M * E;
    int32_t* ps = pos + (size_t)t * M * E;
    if (threadIdx.x == 0) base_sh = 0;
    __syncthreads();
    for (int e = 0; e < E; ++e) {
        if (threadIdx.x == 0) run_sh = 0;
        __syncthreads();
        const int base = base_sh;
        for (int m0 = 0; m0 < M; m0 += 1024) {
            const int m = m0 + threadIdx.x;
            const int flag = (m < M && g[(size_t)m * E + e] > 0.f) ? 1 : 0;
            int incl = flag;                                   // inclusive scan of the flags over the block
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += v; }
            if (lane == 31) warp_sums[warp] = incl;
            __syncthreads();
            if (warp == 0) {
                int w = warp_sums[lane];
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, w, o); if (lane >= o) w += v; }
                warp_sums[lane] = w;
            }
            __syncthreads();
            const int before = run_sh + (warp ? warp_sums[warp - 1] : 0) + incl - flag;
            if (m < M) ps[(size_t)m * E + e] = flag ? base + before : -1;
            __syncthreads();
            if (threadIdx.x == 0) run_sh += warp_sums[31];
            __syncthreads();
        }
        const int count = run_sh;
        const int tiles = (count + 127) >> 7;
        for (int i = threadIdx.x; i < tiles; i += 1024) tile_expert[(size_t)t * tiles_m + (base >> 7) + i] = e;
        __syncthreads();
        if (threadIdx.x == 0) base_sh = base + tiles * 128;
        __syncthreads();
    }
    for (int i = (base_sh >> 7) + threadIdx.x; i < tiles_m; i += 1024) tile_expert[(size_t)t * tiles_m + i] = 0;   // unused tiles
}

__global__ void k_moe_dispatch(const __nv_bfloat16* __restrict__ hb, const float* __restrict__ ssq, int tiles,
                               const float* __restrict__ gates, const int32_t* __restrict__ pos,
                               __nv_bfloat16* __restrict__ xperm, float* __restrict__ ssq_perm, float* __restrict__ gperm,
                               int M, int H, int E, int R) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    const int t = blockIdx.y;
    if (warp >= M) return;
    const size_t row = (size_t)t * M + warp;
    for (int e = 0; e < E; ++e) {
        const int r = pos[row * E + e];
        if (r < 0) continue;
        const size_t dst = (size_t)t * R + r;
        for (int c = lane * 8; c < H; c += 256)
            *reinterpret_cast<uint4*>(xperm + dst * H + c) = *reinterpret_cast<const uint4*>(hb + row * H + c);
        for (int i = lane; i < tiles; i += 32) ssq_perm[dst * tiles + i] = ssq[row * tiles + i];
        if (lane == 0) gperm[dst] = gates[row * E + e];
    }
}

// h = h_in + sum over the token's rows of y; then as k_track_sync: one warp per (token, 128 columns).
__global__ void k_moe_combine(const float* __restrict__ h_in, size_t h_in_tstride, const float* __restrict__ y, const int32_t* __restrict__ pos,
                              int T, int sync, float scale, float* __restrict__ h_out, size_t h_out_tstride,
                              __nv_bfloat16* __restrict__ hb, const float* __restrict__ gain, float* __restrict__ ssq,
                              int M, int H, int E, int R, int tiles) {
    const int groups = (H + 127) / 128;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= M * groups) return;
    const int row = warp / groups, gidx = warp % groups;
    const int c = gidx * 128 + lane * 4;
    const bool in = c < H;
    float4 total = make_float4(0.f, 0.f, 0.f, 0.f);
    const int tile = gidx * 2 + (lane >> 4);
    for (int t = 0; t < T; ++t) {
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
        if (in) {
            a = *reinterpret_cast<const float4*>(h_in + (size_t)t * h_in_tstride + (size_t)row * H + c);
            for (int e = 0; e < E; ++e) {
                const int r = pos[((size_t)t * M + row) * E + e];
                if (r < 0) continue;
                const float4 b = *reinterpret_cast<const float4*>(y + ((size_t)t * R + r) * H + c);
                a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
            }
        }
        if (sync) { total.x += a.x; total.y += a.y; total.z += a.z; total.w += a.w; continue; }
        // no sync after this layer: every track keeps its own stream
        float s = 0.f;
        if (in) {
            *reinterpret_cast<float4*>(h_out + (size_t)t * h_out_tstride + (size_t)row * H + c) = a;
            s = a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w;
            if (hb) {
                const float4 gn = *reinterpret_cast<const float4*>(gain + (size_t)t * H + c);
                uint2 ov;
                __nv_bfloat162 o0 = __floats2bfloat162_rn(a.x * gn.x, a.y * gn.y), o1 = __floats2bfloat162_rn(a.z * gn.z, a.w * gn.w);
                ov.x = *reinterpret_cast<uint32_t*>(&o0); ov.y = *reinterpret_cast<uint32_t*>(&o1);
                *reinterpret_cast<uint2*>(hb + ((size_t)t * M + row) * H + c) = ov;
            }
        }
        for (int o = 8; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (ssq && (lane & 15) == 0 && tile < tiles) ssq[((size_t)t * M + row) * tiles + tile] = s;
    }
    if (!sync) return;
    float s = 0.f;
    if (in) {
        total.x *= scale; total.y *= scale; total.z *= scale; total.w *= scale;
        *reinterpret_cast<float4*>(h_out + (size_t)row * H + c) = total;
        s = total.x * total.x + total.y * total.y + total.z * total.z + total.w * total.w;
        if (hb) {
            for (int t = 0; t < T; ++t) {
                const float4 gn = *reinterpret_cast<const float4*>(gain + (size_t)t * H + c);
                uint2 ov;
                __nv_bfloat162 o0 = __floats2bfloat162_rn(total.x * gn.x, total.y * gn.y), o1 = __floats2bfloat162_rn(total.z * gn.z, total.w * gn.w);
                ov.x = *reinterpret_cast<uint32_t*>(&o0); ov.y = *reinterpret_cast<uint32_t*>(&o1);
                *reinterpret_cast<uint2*>(hb + ((size_t)t * M + row) * H + c) = ov;
            }
        }
    }
    for (int o = 8; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (ssq && (lane & 15) == 0 && tile < tiles) ssq[(size_t)row * tiles + tile] = s;
}

}  // namespace

bool moe_sparse_ok(const pt_model* m, int M, bool decode) {
    // permuting pays when a 128-row tile of an expert fills: prefills; a decode step streams every expert's weights anyway
    return m->E > 0 && !decode && M >= 512 && !m->ar_fn && m->cfg.ffn >= 64;
}

int64_t moe_rows(const pt_model* m, int64_t M) { return ((int64_t)m->cfg.top_k * M + 127) / 128 * 128 + (int64_t)m->E * 128; }

pt_status moe_sparse_ffn(Call& k, int l, bool sync, bool last, float sync_scale, const float* h_in, size_t h_in_tstride,
                         float* h_out, size_t h_out_tstride) {
    pt_model* m = k.m;
    const pt_config& g = m->cfg;
    Work& w = k.w;
    cudaStream_t st = k.st;
    const int T = g.T, M = k.M, H = g.hidden, F = g.ffn, E = m->E;
    const int R = (int)moe_rows(m, M), tiles_m = R / 128;
    const int tiles = (H + kSsqTile - 1) / kSsqTile;
    MoeWork& mw = w.moe;
    k_moe_plan<<<T, 1024, 0, st>>>(w.gates, M, E, tiles_m, mw.pos, mw.tile_expert);
    k_moe_dispatch<<<dim3((M * 32 + 255) / 256, T), 256, 0, st>>>((const __nv_bfloat16*)w.a, w.ssq, tiles, w.gates, mw.pos, mw.xperm, mw.ssq_perm,
                                                                    mw.gperm, M, H, E, R);
    g_launches.fetch_add(2, std::memory_order_relaxed);
    pt_status s;
    GemmP base{};
    base.M = R; base.status = m->status(); base.eps = g.rms_eps; base.kt = 1; base.T = T;
    base.scale = 1.0f; base.n_sum = 1; base.n_out = 1; base.w_static = 0; base.kps = 1; base.pair = 0;
    base.tile_expert = mw.tile_expert;
    {   // gate/up of the row's expert + SwiGLU, weighted by the row's routing weight
        GemmP p = base;
        p.N = 2 * F; p.K = H;
        p.ssq_in = mw.ssq_perm; p.ssq_in_tstride = (size_t)R * tiles; p.ssq_tiles = tiles;
        p.z_out = mw.zperm;
        p.gates = mw.gperm; p.n_experts = 1; p.expert_cols = 1 << 30;
        p.w_row_per_expert = 2 * F; p.w_k_per_expert = 0;
        const int bn = 2 * F >= 256 ? 256 : 128;
        CUtensorMap ta;
        if ((s = make_a_map(&ta, mw.xperm, H, R, T, 1)) != PT_OK) return s;
        ProfScope ps(m, st, 3);
        if ((s = launch_gemm(EPI_SWIGLU, bn, ta, m->wmaps[l].m[2][bn_index(bn)][0], p, st)) != PT_OK) return s;
    }
    {   // down projection of the row's expert, fp32 rows
        GemmP p = base;
        p.N = H; p.K = F;
        p.c_out = mw.yperm;
        p.w_row_per_expert = 0; p.w_k_per_expert = F;
        const int bn = H >= 256 ? 256 : (H >= 128 ? 128 : 64);
        CUtensorMap ta;
        if ((s = make_a_map(&ta, mw.zperm, F, R, T, 1)) != PT_OK) return s;
        ProfScope ps(m, st, sync ? 5 : 4);
        if ((s = launch_gemm(EPI_PLAIN, bn, ta, m->wmaps[l].m[3][bn_index(bn)][0], p, st)) != PT_OK) return s;
    }
    const unsigned grid = (unsigned)(((size_t)M * ((H + 127) / 128) * 32 + 255) / 256);
    ProfScope ps(m, st, 6);
    k_moe_combine<<<grid, 256, 0, st>>>(h_in, h_in_tstride, mw.yperm, mw.pos, T, sync ? 1 : 0, sync_scale, h_out, h_out_tstride,
                                        last ? nullptr : (__nv_bfloat16*)w.a, last ? nullptr : m->gain(0, l + 1), last ? nullptr : w.ssq,
                                        M, H, E, R, tiles);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return PT_OK;
}

}  // namespace pt
