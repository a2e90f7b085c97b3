// Plain SIMT kernels for every step of a PT layer, templated on the storage type.
// They are the fp32 path (accumulating in fp32 FMA, no tensor cores, no tf32) and, with
// pt_config.flags bit 0, a slow cross-check of the bf16 tensor-core path.  The track index is
// a grid dimension of every kernel.
#include "pt_tc.h"
#include "pt_ptx.cuh"

namespace pt {

#define LAUNCH_COUNT() (g_launches.fetch_add(1, std::memory_order_relaxed))

template <class E> __device__ __forceinline__ float ldf(const E* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
template <class E> __device__ __forceinline__ void stf(E* p, float v);
template <> __device__ __forceinline__ void stf<float>(float* p, float v) { *p = v; }
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }


// ---- weight packing: rows of one [rows, cols] source matrix go to mapped rows of the packed matrix.
// kind: PT_WQ/PT_WK/PT_WV -> rows offset inside [Nqkv, H]; PT_WG/PT_WU -> interleaved in groups
// of 16 rows (gate rows 32g..32g+15, up rows 32g+16..32g+31); others -> identity.
// A PT-MoE model packs its experts side by side: expert e's gate/up rows follow those of expert e - 1 (row_off),
// its down-projection columns sit at e * ffn of rows that are Ftot wide (dst_cols, col_off).
template <class E>
__global__ void k_pack(const E* __restrict__ src, E* __restrict__ dst, int rows, int cols, int row_off, int interleave,
                       int dst_cols, int col_off) {
    size_t n = (size_t)rows * cols;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        int r = (int)(i / cols), c = (int)(i % cols);
        int dr = (interleave ? (r / 16) * 32 + (interleave - 1) * 16 + r % 16 : r) + row_off;
        dst[(size_t)dr * dst_cols + col_off + c] = src[i];
    }
}

void launch_pack(const pt_model* m, int kind, const void* src, void* dst, cudaStream_t st, int expert) {
    const pt_config& c = m->cfg;
    int rows, cols, row_off = 0, il = 0, dst_cols = 0, col_off = 0;
    switch (kind) {
        case PT_WQ: rows = m->QD; cols = c.hidden; break;
        case PT_WK: rows = m->KVD; cols = c.hidden; row_off = m->QD; break;
        case PT_WV: rows = m->KVD; cols = c.hidden; row_off = m->QD + m->KVD; break;
        case PT_WO: rows = c.hidden; cols = m->QD; break;
        case PT_WG: rows = c.ffn; cols = c.hidden; il = 1; row_off = expert * 2 * c.ffn; break;
        case PT_WU: rows = c.ffn; cols = c.hidden; il = 2; row_off = expert * 2 * c.ffn; break;
        default: rows = c.hidden; cols = c.ffn; dst_cols = m->Ftot; col_off = expert * c.ffn; break;
    }
    if (!dst_cols) dst_cols = cols;
    size_t n = (size_t)rows * cols;
    int grid = (int)std::min<size_t>((n + 255) / 256, 148 * 8);
    if (m->esz == 2) k_pack<<<grid, 256, 0, st>>>((const __nv_bfloat16*)src, (__nv_bfloat16*)dst, rows, cols, row_off, il, dst_cols, col_off);
    else k_pack<<<grid, 256, 0, st>>>((const float*)src, (float*)dst, rows, cols, row_off, il, dst_cols, col_off);
    LAUNCH_COUNT();
}

// ---- x -> fp32 residual stream
template <class E>
__global__ void k_prep(const E* __restrict__ x, int64_t x_stride, float* __restrict__ h, size_t MH) {
    int t = blockIdx.y;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < MH; i += (size_t)gridDim.x * blockDim.x)
        h[(size_t)t * MH + i] = ldf(x + (size_t)t * x_stride + i);
}

// ---- RMSNorm: a = h * rsqrt(mean(h^2) + eps) * g ; one block per (row, track)
template <class E>
__global__ void k_rmsnorm(const float* __restrict__ h, size_t h_stride, const float* __restrict__ g,
                          E* __restrict__ a, int M, int H, float eps) {
    int m = blockIdx.x, t = blockIdx.y;
    const float* row = h + (size_t)t * h_stride + (size_t)m * H;
    float s = 0.f;
    for (int i = threadIdx.x; i < H; i += blockDim.x) s += row[i] * row[i];
    __shared__ float red[32];
    for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x < 32) {
        float v = threadIdx.x < (blockDim.x >> 5) ? red[threadIdx.x] : 0.f;
        for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (threadIdx.x == 0) red[0] = v;
    }
    __syncthreads();
    float rinv = 1.0f / sqrtf(red[0] / (float)H + eps);
    for (int i = threadIdx.x; i < H; i += blockDim.x)
        stf(a + ((size_t)t * M + m) * H + i, row[i] * rinv * g[(size_t)t * H + i]);
}

// ---- GEMM  C[t,m,n] = sum_k A[t,m,k] * W[t,n,k]  (64x64x16 tiles, 4x4 per thread)
// RESID = 0: C stored in E.  RESID = 1: hout[t,m,n] = hin[t*hin_stride + m*N + n] + acc (fp32).
template <class E, int RESID>
__global__ void __launch_bounds__(256)
k_gemm(const E* __restrict__ A, const E* __restrict__ W, void* Cout,
       const float* hin, size_t hin_stride, int M, int N, int K) {
    __shared__ float As[16][64 + 4], Ws[16][64 + 4];
    int t = blockIdx.z;
    const E* At = A + (size_t)t * M * K;
    const E* Wt = W + (size_t)t * N * K;
    int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
    int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < K; k0 += 16) {
        for (int i = threadIdx.x; i < 64 * 16; i += 256) {
            int r = i / 16, kk = i % 16;
            int gm = m0 + r, gn = n0 + r, gk = k0 + kk;
            As[kk][r] = (gm < M && gk < K) ? ldf(At + (size_t)gm * K + gk) : 0.f;
            Ws[kk][r] = (gn < N && gk < K) ? ldf(Wt + (size_t)gn * K + gk) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = As[kk][ty * 4 + i]; b[i] = Ws[kk][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int gm = m0 + ty * 4 + i;
        if (gm >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int gn = n0 + tx * 4 + j;
            if (gn >= N) continue;
            size_t idx = ((size_t)t * M + gm) * N + gn;
            if (RESID) ((float*)Cout)[idx] = hin[(size_t)t * hin_stride + (size_t)gm * N + gn] + acc[i][j];
            else stf((E*)Cout + idx, acc[i][j]);
        }
    }
}

// ---- RoPE on q and k (in place) + KV-cache append.  One thread per (t, row, head slot, pair j).
template <class E>
__global__ void k_rope_kv(E* __restrict__ qkv, E* __restrict__ pool_l, int64_t pool_tstride, int64_t slab_elems,
                          const int64_t* __restrict__ row_kvoff, const int32_t* __restrict__ row_pos,
                          const float* __restrict__ cs, const float* __restrict__ sn,
                          int M, int nq, int nkv, int dh, int ps, int* status) {
    int half = dh / 2, slots = nq + 2 * nkv;
    size_t per_t = (size_t)M * slots * half;
    int t = blockIdx.y;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < per_t; i += (size_t)gridDim.x * blockDim.x) {
        int j = (int)(i % half);
        int hs = (int)((i / half) % slots);
        int m = (int)(i / ((size_t)half * slots));
        E* v = qkv + ((size_t)t * M + m) * (size_t)(slots * dh) + (size_t)hs * dh;
        int pos = row_pos[m];
        float lo = ldf(v + j), hi = ldf(v + j + half);
        if (hs < nq + nkv) {
            float c = cs[(size_t)pos * half + j], s = sn[(size_t)pos * half + j];
            float rlo = lo * c - hi * s, rhi = hi * c + lo * s;
            lo = rlo; hi = rhi;
            if (hs < nq) { stf(v + j, lo); stf(v + j + half, hi); }
        }
        if (hs >= nq) {
            int kv = hs >= nq + nkv, head = hs - nq - kv * nkv;
            int64_t off = row_kvoff[m] + ((int64_t)kv * nkv + head) * ps * dh;
            if (off < 0 || off + dh > slab_elems) { report(status, PT_ERR_DEVICE_BOUNDS, LOC_ROPE_PAGE); continue; }
            E* dst = pool_l + (size_t)t * pool_tstride + off;
            stf(dst + j, lo); stf(dst + j + half, hi);
        }
    }
}

// ---- attention: one warp per (row, q head, track); online softmax over keys 0..pos read
// from the paged cache through the block table.
template <class E, int DH>
__global__ void k_attn(const E* __restrict__ qkv, int q_row_stride, const E* __restrict__ pool_l,
                       int64_t pool_tstride, const int32_t* __restrict__ bt, int maxp,
                       const int32_t* __restrict__ row_pos, const int32_t* __restrict__ row_b,
                       E* __restrict__ o, int M, int nq, int nkv, int ps, int num_pages, int* status) {
    constexpr int PER = DH / 32;
    int warp = (blockIdx.x * blockDim.x + threadIdx.x) / 32, lane = threadIdx.x & 31;
    int t = blockIdx.y;
    if (warp >= M * nq) return;
    int m = warp / nq, head = warp % nq, kvh = head / (nq / nkv);
    const E* q = qkv + ((size_t)t * M + m) * q_row_stride + (size_t)head * DH;
    float qv[PER], acc[PER];
    float scale = 1.0f / sqrtf((float)DH);
#pragma unroll
    for (int i = 0; i < PER; ++i) { qv[i] = ldf(q + lane + 32 * i) * scale; acc[i] = 0.f; }
    float mx = -INFINITY, den = 0.f;
    int pos = row_pos[m], b = row_b[m];
    const E* slab = pool_l + (size_t)t * pool_tstride;
    for (int j = 0; j <= pos; ++j) {
        int page = bt[(size_t)b * maxp + j / ps];
        if (page < 0 || page >= num_pages) { if (lane == 0) report(status, PT_ERR_DEVICE_BOUNDS, LOC_ATTN_PAGE); return; }
        const E* kp = slab + (((size_t)page * 2 + 0) * nkv + kvh) * ps * DH + (size_t)(j % ps) * DH;
        const E* vp = slab + (((size_t)page * 2 + 1) * nkv + kvh) * ps * DH + (size_t)(j % ps) * DH;
        float s = 0.f;
#pragma unroll
        for (int i = 0; i < PER; ++i) s += qv[i] * ldf(kp + lane + 32 * i);
        for (int d = 16; d; d >>= 1) s += __shfl_xor_sync(0xffffffffu, s, d);
        float nm = fmaxf(mx, s);
        float corr = expf(mx - nm), p = expf(s - nm);
        den = den * corr + p;
#pragma unroll
        for (int i = 0; i < PER; ++i) acc[i] = acc[i] * corr + p * ldf(vp + lane + 32 * i);
        mx = nm;
    }
#pragma unroll
    for (int i = 0; i < PER; ++i) stf(o + ((size_t)t * M + m) * (size_t)(nq * DH) + (size_t)head * DH + lane + 32 * i, acc[i] / den);
}

// ---- SwiGLU on the interleaved gate/up product: gu[.., 32g + r] gate, gu[.., 32g + 16 + r] up
template <class E>
__global__ void k_swiglu(const E* __restrict__ gu, E* __restrict__ z, size_t rows, int F) {
    size_t n = rows * F;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        size_t r = i / F;
        int f = (int)(i % F);
        const E* p = gu + r * 2 * F + (f / 16) * 32 + f % 16;
        float g = ldf(p), u = ldf(p + 16);
        stf(z + i, g / (1.0f + expf(-g)) * u);
    }
}

// ---- track-sync: out[m, :] = scale * sum_t h[t, m, :], tracks added in index order
__global__ void k_sync(const float* __restrict__ h, float* __restrict__ out, size_t MH, int T, float scale) {
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < MH; i += (size_t)gridDim.x * blockDim.x) {
        float s = h[i];
        for (int t = 1; t < T; ++t) s += h[(size_t)t * MH + i];
        out[i] = s * scale;
    }
}

__global__ void k_bcast(const float* __restrict__ src, size_t src_tstride, float* __restrict__ dst, size_t MH) {
    int t = blockIdx.y;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < MH; i += (size_t)gridDim.x * blockDim.x)
        dst[(size_t)t * MH + i] = src[(size_t)t * src_tstride + i];
}

static inline int grid1d(size_t n, int block = 256) { return (int)std::min<size_t>((n + block - 1) / block, 148 * 16); }

void tap_copy(Call& k, int layer, int point, const float* src, size_t src_tstride) {
    pt_model* m = k.m;
    if (!m->tap_buf || (m->tap_layer != -1 && m->tap_layer != layer)) return;
    size_t MH = (size_t)k.M * m->cfg.hidden;
    size_t block = (size_t)m->cfg.T * MH;
    float* dst = m->tap_buf + ((m->tap_layer == -1 ? (size_t)layer * 2 : 0) + point) * block;
    k_bcast<<<dim3(grid1d(MH), m->cfg.T), 256, 0, k.st>>>(src, src_tstride, dst, MH);
    LAUNCH_COUNT();
}

void launch_simt_attn_bf16(Call& k, const __nv_bfloat16* q, int q_row_stride, const __nv_bfloat16* pool_l, __nv_bfloat16* o) {
    pt_model* m = k.m;
    pt_kv_cache* c = k.c;
    const pt_config& g = m->cfg;
    using E = __nv_bfloat16;
    const int64_t pool_tstride = (int64_t)g.L * c->slab_elems;
    dim3 ag(((size_t)k.M * g.heads * 32 + 127) / 128, g.T);
#define ATTN(DH_) k_attn<E, DH_><<<ag, 128, 0, k.st>>>(q, q_row_stride, pool_l, pool_tstride, k.w.meta.bt, k.w.meta.maxp, \
        k.w.meta.row_pos, k.w.meta.row_b, o, k.M, g.heads, g.kv_heads, c->ps, c->num_pages, m->status())
    if (m->dh == 32) ATTN(32); else if (m->dh == 64) ATTN(64); else ATTN(128);
#undef ATTN
    LAUNCH_COUNT();
}

template <class E>
static pt_status simt_forward_t(Call& k) {
    pt_model* m = k.m;
    pt_kv_cache* c = k.c;
    const pt_config& g = m->cfg;
    const int T = g.T, M = k.M, H = g.hidden, F = g.ffn, dh = m->dh;
    const size_t MH = (size_t)M * H;
    cudaStream_t st = k.st;
    Work& w = k.w;
    E* pool = (E*)c->pool;
    const int64_t pool_tstride = (int64_t)g.L * c->slab_elems;

    k_prep<E><<<dim3(grid1d(MH), T), 256, 0, st>>>((const E*)k.x, k.x_stride, w.hT, MH);
    LAUNCH_COUNT();
    const float* hin = w.hT;
    size_t hin_stride = MH;
    for (int l = 0; l < g.L; ++l) {
        const E* Wqkv = (const E*)(m->wbuf + m->off_wqkv) + (size_t)l * m->wqkv_layer();
        const E* Wo = (const E*)(m->wbuf + m->off_wo) + (size_t)l * m->wo_layer();
        const E* Wgu = (const E*)(m->wbuf + m->off_wgu) + (size_t)l * m->wgu_layer();
        const E* Wd = (const E*)(m->wbuf + m->off_wd) + (size_t)l * m->wd_layer();
        E* pool_l = pool + (size_t)l * c->slab_elems;
        k_rmsnorm<E><<<dim3(M, T), 128, 0, st>>>(hin, hin_stride, m->gain(0, l), (E*)w.a, M, H, g.rms_eps);
        LAUNCH_COUNT();
        k_gemm<E, 0><<<dim3((m->Nqkv + 63) / 64, (M + 63) / 64, T), 256, 0, st>>>((const E*)w.a, Wqkv, w.qkv, nullptr, 0, M, m->Nqkv, H);
        LAUNCH_COUNT();
        k_rope_kv<E><<<dim3(grid1d((size_t)M * (g.heads + 2 * g.kv_heads) * (dh / 2)), T), 256, 0, st>>>(
            (E*)w.qkv, pool_l, pool_tstride, c->slab_elems, w.meta.row_kvoff, w.meta.row_pos,
            m->rope_cos(), m->rope_sin(), M, g.heads, g.kv_heads, dh, c->ps, m->status());
        LAUNCH_COUNT();
        dim3 ag(((size_t)M * g.heads * 32 + 127) / 128, T);
#define ATTN(DH_) k_attn<E, DH_><<<ag, 128, 0, st>>>((const E*)w.qkv, m->Nqkv, pool_l, pool_tstride, w.meta.bt, w.meta.maxp, \
            w.meta.row_pos, w.meta.row_b, (E*)w.o, M, g.heads, g.kv_heads, c->ps, c->num_pages, m->status())
        if (dh == 32) ATTN(32); else if (dh == 64) ATTN(64); else ATTN(128);
#undef ATTN
        LAUNCH_COUNT();
        k_gemm<E, 1><<<dim3((H + 63) / 64, (M + 63) / 64, T), 256, 0, st>>>((const E*)w.o, Wo, w.hT, hin, hin_stride, M, H, m->QD);
        LAUNCH_COUNT();
        tap_copy(k, l, 0, w.hT, MH);
        k_rmsnorm<E><<<dim3(M, T), 128, 0, st>>>(w.hT, MH, m->gain(1, l), (E*)w.a, M, H, g.rms_eps);
        LAUNCH_COUNT();
        k_gemm<E, 0><<<dim3((2 * F + 63) / 64, (M + 63) / 64, T), 256, 0, st>>>((const E*)w.a, Wgu, w.gu, nullptr, 0, M, 2 * F, H);
        LAUNCH_COUNT();
        k_swiglu<E><<<grid1d((size_t)T * M * F), 256, 0, st>>>((const E*)w.gu, (E*)w.z, (size_t)T * M, F);
        LAUNCH_COUNT();
        k_gemm<E, 1><<<dim3((H + 63) / 64, (M + 63) / 64, T), 256, 0, st>>>((const E*)w.z, Wd, w.hT, w.hT, MH, M, H, F);
        LAUNCH_COUNT();
        if ((l + 1) % g.D == 0) {
            float* dst = (l + 1 == g.L) ? k.out : w.hS;
            k_sync<<<grid1d(MH), 256, 0, st>>>(w.hT, dst, MH, T, g.sync_op ? 1.0f / T : 1.0f);
            LAUNCH_COUNT();
            hin = dst; hin_stride = 0;
        } else {
            hin = w.hT; hin_stride = MH;
        }
        tap_copy(k, l, 1, hin, hin_stride);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("kernel launch failed: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
    return PT_OK;
}

pt_status simt_forward(Call& k) {
    return k.m->esz == 2 ? simt_forward_t<__nv_bfloat16>(k) : simt_forward_t<float>(k);
}

}  // namespace pt
