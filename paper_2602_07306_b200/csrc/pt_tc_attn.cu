// Attention kernels of the bf16 path, both reading K and V straight from the paged per-track
// KV cache through the block table.
//   k_flash_prefill  causal flash-style attention: a CTA owns 64 query rows of one (track,
//                    sequence, head); KV tiles of 64 keys are staged in shared memory with 16-byte
//                    cp.async copies (XOR-swizzled rows), scores and P*V run on mma.sync m16n8k16,
//                    the online softmax keeps its row statistics in registers and reduces them
//                    with quad shuffles.
//   k_decode_attn    split-KV decode: a CTA owns one (track, sequence, KV head, key range); the G
//                    query heads that share the KV head are the rows of one 16-row MMA tile, each
//                    of the 4 warps takes one 16-token page of every 64-key tile, and the warps'
//                    partial (max, sum, output) triples are merged in shared memory.  Key ranges
//                    of one sequence are merged by k_decode_combine.
// Softmax runs in base 2: scores are scaled by log2(e)/sqrt(head_dim) once.
#include "pt_tc.h"
#include "pt_ptx.cuh"

namespace pt {

namespace {

constexpr int kTileKeys = 64;
constexpr int kThreads = 128;


__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    int sz = valid ? 16 : 0;                         // 0 source bytes: the 16 destination bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Byte offset of 16-byte chunk `chunk` of row `row` in a [rows][DH] bf16 tile whose chunks are
// XOR-swizzled so that 8 consecutive rows of one chunk column fall into 8 different bank groups.
template <int DH> __device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
    constexpr int CPR = DH / 8;
    int sw = CPR >= 8 ? (row & 7) : ((row >> 1) & 3);
    return (uint32_t)(row * (DH * 2) + ((chunk ^ sw) << 4));
}


// Stage `rows` keys starting at key `key0` of sequence b (K and V of one KV head) into a tile.
// Keys at or beyond `key_end` are zero-filled.
template <int DH>
__device__ __forceinline__ void load_kv_tile(const AttnP& p, const __nv_bfloat16* slab, int b, int kvh, int key0, int key_end,
                                             uint8_t* sk, uint8_t* sv, bool& bad_page) {
    constexpr int CPR = DH / 8;
    constexpr int ROWS_PER_PASS = kThreads / CPR;
    const int chunk = threadIdx.x % CPR;
    const int r0 = threadIdx.x / CPR;
    const uint32_t k_base = smem_u32(sk), v_base = smem_u32(sv);
#pragma unroll
    for (int r = r0; r < kTileKeys; r += ROWS_PER_PASS) {
        int key = key0 + r;
        bool valid = key < key_end;
        int page = valid ? p.bt[(size_t)b * p.maxp + key / p.ps] : 0;
        if (page < 0 || page >= p.num_pages) { bad_page = true; valid = false; page = 0; }
        const __nv_bfloat16* kp = slab + (((size_t)page * 2) * p.nkv + kvh) * p.ps * DH + (size_t)(key % p.ps) * DH + chunk * 8;
        const __nv_bfloat16* vp = kp + (size_t)p.nkv * p.ps * DH;
        uint32_t off = tile_off<DH>(r, chunk);
        cp_async16(k_base + off, valid ? kp : slab, valid);
        cp_async16(v_base + off, valid ? vp : slab, valid);
    }
}

// A-operand fragments of 16 query rows read directly from global memory.  row_ptr_lo / row_ptr_hi
// point at the head_dim values of rows lane/4 and lane/4 + 8 (nullptr = a zero row).
template <int DH>
__device__ __forceinline__ void load_q_frags(uint32_t (*qf)[4], const __nv_bfloat16* lo, const __nv_bfloat16* hi, int lane) {
    const int c = (lane & 3) * 2;
#pragma unroll
    for (int ks = 0; ks < DH / 16; ++ks) {
        qf[ks][0] = lo ? *reinterpret_cast<const uint32_t*>(lo + ks * 16 + c) : 0u;
        qf[ks][1] = hi ? *reinterpret_cast<const uint32_t*>(hi + ks * 16 + c) : 0u;
        qf[ks][2] = lo ? *reinterpret_cast<const uint32_t*>(lo + ks * 16 + 8 + c) : 0u;
        qf[ks][3] = hi ? *reinterpret_cast<const uint32_t*>(hi + ks * 16 + 8 + c) : 0u;
    }
}

// S[16 x 16] += Q[16 x DH] * K[16 keys x DH]^T for the 16 keys starting at tile row `krow`.
template <int DH>
__device__ __forceinline__ void qk_16keys(float (*s)[4], const uint32_t (*qf)[4], uint32_t k_base, int krow, int lane) {
    const int row = krow + (lane >> 4) * 8 + (lane & 7);
    const int cofs = (lane >> 3) & 1;
#pragma unroll
    for (int ks = 0; ks < DH / 16; ++ks) {
        uint32_t b0, b1, b2, b3;
        ldsm_x4(k_base + tile_off<DH>(row, ks * 2 + cofs), b0, b1, b2, b3);
        mma_bf16(s[0], qf[ks], b0, b1);
        mma_bf16(s[1], qf[ks], b2, b3);
    }
}

// O[16 x DH] += P[16 x 16] * V[16 keys x DH] for the 16 keys starting at tile row `krow`.
template <int DH>
__device__ __forceinline__ void pv_16keys(float (*o)[4], const uint32_t* pf, uint32_t v_base, int krow, int lane) {
    const int row = krow + ((lane >> 3) & 1) * 8 + (lane & 7);
    const int cofs = lane >> 4;
#pragma unroll
    for (int dc = 0; dc < DH / 16; ++dc) {
        uint32_t b0, b1, b2, b3;
        ldsm_x4_t(v_base + tile_off<DH>(row, dc * 2 + cofs), b0, b1, b2, b3);
        mma_bf16(o[dc * 2], pf, b0, b1);
        mma_bf16(o[dc * 2 + 1], pf, b2, b3);
    }
}

// ------------------------------------------------------------------------------------ prefill

template <int DH>
__global__ void __launch_bounds__(kThreads)
k_flash_prefill(const AttnP p) {
    constexpr int STAGES = 2;
    constexpr int TILE_BYTES = kTileKeys * DH * 2;
    extern __shared__ __align__(128) uint8_t smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int qtiles = (p.S + 63) / 64;
    const int qt = qtiles - 1 - blockIdx.x;                  // longest rows first
    const int head = blockIdx.y, kvh = head / (p.nq / p.nkv);
    const int t = blockIdx.z / p.B, b = blockIdx.z % p.B;
    const int start = p.kvlen[b] - p.S;                      // position of the sequence's first new token
    const __nv_bfloat16* slab = p.pool_l + (size_t)t * p.pool_tstride;

    const int s_lo = qt * 64 + warp * 16 + (lane >> 2), s_hi = s_lo + 8;     // rows inside the sequence
    const size_t rowbase = ((size_t)t * p.M + (size_t)b * p.S) * (size_t)(p.nq * DH) + (size_t)head * DH;
    uint32_t qf[DH / 16][4];
    load_q_frags<DH>(qf, s_lo < p.S ? p.q + rowbase + (size_t)s_lo * (p.nq * DH) : nullptr,
                     s_hi < p.S ? p.q + rowbase + (size_t)s_hi * (p.nq * DH) : nullptr, lane);

    float o[DH / 8][4];
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

    const int q_end = min(p.S, qt * 64 + 64);                // rows of this CTA: [qt*64, q_end)
    const int key_end = start + q_end;                       // keys any row of the CTA may see
    const int ntiles = (key_end + kTileKeys - 1) / kTileKeys;
    const int pos_lo = start + s_lo, pos_hi = start + s_hi;
    const int warp_pos_max = start + min(q_end, qt * 64 + warp * 16 + 16) - 1;
    bool bad_page = false;

    load_kv_tile<DH>(p, slab, b, kvh, 0, key_end, smem, smem + TILE_BYTES, bad_page);
    cp_async_commit();
    for (int j = 0; j < ntiles; ++j) {
        uint8_t* sk = smem + (j % STAGES) * 2 * TILE_BYTES;
        if (j + 1 < ntiles) {
            uint8_t* nk = smem + ((j + 1) % STAGES) * 2 * TILE_BYTES;
            load_kv_tile<DH>(p, slab, b, kvh, (j + 1) * kTileKeys, key_end, nk, nk + TILE_BYTES, bad_page);
        }
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();
        const uint32_t k_base = smem_u32(sk), v_base = k_base + TILE_BYTES;
        const int key0 = j * kTileKeys;
        if (key0 <= warp_pos_max) {                          // the warp's rows see part of this tile
            float s[8][4];
#pragma unroll
            for (int i = 0; i < 8; ++i) { s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f; }
#pragma unroll
            for (int kb = 0; kb < 4; ++kb) qk_16keys<DH>(&s[kb * 2], qf, k_base, kb * 16, lane);
            const bool diag = key0 + kTileKeys - 1 > start + qt * 64 + warp * 16;   // some key may be masked
            float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float v = s[i][e] * p.scale_log2;
                    if (diag) {
                        int key = key0 + i * 8 + (lane & 3) * 2 + (e & 1);
                        if (key > ((e & 2) ? pos_hi : pos_lo)) v = -INFINITY;
                    }
                    s[i][e] = v;
                }
                mx_lo = fmaxf(mx_lo, fmaxf(s[i][0], s[i][1]));
                mx_hi = fmaxf(mx_hi, fmaxf(s[i][2], s[i][3]));
            }
            mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
            mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
            mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
            mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
            const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
            const float ref_lo = mn_lo == -INFINITY ? 0.f : mn_lo, ref_hi = mn_hi == -INFINITY ? 0.f : mn_hi;
            const float c_lo = exp2f(m_lo - ref_lo), c_hi = exp2f(m_hi - ref_hi);
            m_lo = mn_lo; m_hi = mn_hi;
            float sum_lo = 0.f, sum_hi = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                s[i][0] = exp2f(s[i][0] - ref_lo); s[i][1] = exp2f(s[i][1] - ref_lo);
                s[i][2] = exp2f(s[i][2] - ref_hi); s[i][3] = exp2f(s[i][3] - ref_hi);
                sum_lo += s[i][0] + s[i][1];
                sum_hi += s[i][2] + s[i][3];
            }
            l_lo = l_lo * c_lo + sum_lo;
            l_hi = l_hi * c_hi + sum_hi;
#pragma unroll
            for (int i = 0; i < DH / 8; ++i) { o[i][0] *= c_lo; o[i][1] *= c_lo; o[i][2] *= c_hi; o[i][3] *= c_hi; }
#pragma unroll
            for (int kb = 0; kb < 4; ++kb) {
                uint32_t pf[4];
                pf[0] = pack_bf16(s[kb * 2][0], s[kb * 2][1]);
                pf[1] = pack_bf16(s[kb * 2][2], s[kb * 2][3]);
                pf[2] = pack_bf16(s[kb * 2 + 1][0], s[kb * 2 + 1][1]);
                pf[3] = pack_bf16(s[kb * 2 + 1][2], s[kb * 2 + 1][3]);
                pv_16keys<DH>(o, pf, v_base, kb * 16, lane);
            }
        }
        __syncthreads();
    }
    if (bad_page && lane == 0) report(p.status, PT_ERR_DEVICE_BOUNDS, LOC_FLASH_PAGE);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1); l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1); l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
    const float inv_lo = l_lo > 0.f ? 1.f / l_lo : 0.f, inv_hi = l_hi > 0.f ? 1.f / l_hi : 0.f;
    const int c = (lane & 3) * 2;
    if (s_lo < p.S) {
        __nv_bfloat16* dst = p.o + rowbase + (size_t)s_lo * (p.nq * DH);
#pragma unroll
        for (int i = 0; i < DH / 8; ++i) *reinterpret_cast<uint32_t*>(dst + i * 8 + c) = pack_bf16(o[i][0] * inv_lo, o[i][1] * inv_lo);
    }
    if (s_hi < p.S) {
        __nv_bfloat16* dst = p.o + rowbase + (size_t)s_hi * (p.nq * DH);
#pragma unroll
        for (int i = 0; i < DH / 8; ++i) *reinterpret_cast<uint32_t*>(dst + i * 8 + c) = pack_bf16(o[i][2] * inv_hi, o[i][3] * inv_hi);
    }
}

// ------------------------------------------------------------------------------------ decode

// Merge the four warps' partial (max, sum, output) of the G query heads through shared memory
// and store either the final output (one key range) or this range's partial.  All threads of
// the CTA call it after a __syncthreads() that retired every use of `mg`.
template <int DH>
__device__ __forceinline__ void decode_merge_store(const AttnP& p, float* mg, float (*o)[4], float m_run, float l_run,
                                                   int t, int b, int kvh, int split) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = p.nq / p.nkv;
    const int g_lo = lane >> 2;
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    if (g_lo < G) {                                           // per-warp partials: [warp][g][DH + 2] floats
        float* dst = mg + ((size_t)warp * 8 + g_lo) * (DH + 2);
        const int c = (lane & 3) * 2;
#pragma unroll
        for (int i = 0; i < DH / 8; ++i) { dst[i * 8 + c] = o[i][0]; dst[i * 8 + c + 1] = o[i][1]; }
        if ((lane & 3) == 0) { dst[DH] = m_run; dst[DH + 1] = l_run; }
    }
    __syncthreads();
    const int ns = p.nsplit[b];
    for (int idx = threadIdx.x; idx < G * DH; idx += kThreads) {
        const int g = idx / DH, d = idx % DH;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < 4; ++w) M = fmaxf(M, mg[((size_t)w * 8 + g) * (DH + 2) + DH]);
        float L = 0.f, acc = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const float* src = mg + ((size_t)w * 8 + g) * (DH + 2);
            float f = src[DH] == -INFINITY ? 0.f : exp2f(src[DH] - M);
            L += src[DH + 1] * f;
            acc += src[d] * f;
        }
        const int head = kvh * G + g;
        if (ns == 1) {
            p.o[((size_t)t * p.M + b) * (size_t)(p.nq * DH) + (size_t)head * DH + d] = __float2bfloat16_rn(L > 0.f ? acc / L : 0.f);
        } else {
            float* dst = p.part + ((((size_t)t * p.B + b) * p.nq + head) * p.max_splits + split) * (DH + 2);
            dst[d] = acc;
            if (d == 0) { dst[DH] = M; dst[DH + 1] = L; }
        }
    }
}

// ---- TMA-fed decode attention (page size a multiple of 16, head_dim 64 or 128) ----------------
// Each warp streams its own pages: lane 0 issues one tensor-map load per 128-byte-wide half of
// the K and V blocks of a 16-token page (hardware 128-byte swizzle, so ldmatrix reads are
// conflict-free) into the warp's private ring of kDecStages slots and waits on the slot's
// mbarrier; no CTA-wide barrier is taken until the final merge.  Waits are bounded.
constexpr int kDecStages = 3;
constexpr uint32_t kDecSpin = 1u << 24;


// Byte offset of 16-byte chunk `chunk` of row `row` (0..15) inside one page block as the tensor
// map lays it out: 128-byte-wide halves of 16 rows each, chunks XOR-swizzled with row % 8.
template <int DH> __device__ __forceinline__ uint32_t page_off(int row, int chunk) {
    return (uint32_t)((chunk >> 3) * 2048 + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

template <int DH>
__global__ void __launch_bounds__(kThreads)
k_decode_attn_tma(const __grid_constant__ CUtensorMap kvmap, const AttnP p) {
    constexpr int PAGE_BYTES = 16 * DH * 2;                   // one K or V block of 16 tokens
    constexpr int SLOT_BYTES = 2 * PAGE_BYTES;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = (uint64_t*)(smem + 4 * kDecStages * SLOT_BYTES);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    grid_dep_wait();                                          // q and this step's K/V rows come from the QKV GEMM before it
    grid_dep_launch();
    const int32_t* item = p.items + (size_t)blockIdx.x * 4;
    const int b = item[0], kstart = item[1], kcount = item[2], split = item[3];
    const int kvh = blockIdx.y, t = blockIdx.z;
    const int G = p.nq / p.nkv;
    const int key_end = min(kstart + kcount, p.kvlen[b]);
    const int npages = (key_end - kstart + 15) >> 4;          // 16-token groups of this key range

    if (threadIdx.x == 0) {
        for (int i = 0; i < 4 * kDecStages; ++i) mbar_init(&bars[i], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    uint8_t* ring = smem + warp * kDecStages * SLOT_BYTES;
    uint64_t* wbar = bars + warp * kDecStages;
    bool bad_page = false;
    // lane 0: fetch the K and V blocks of local 16-token group `g` into slot g % kDecStages
    auto issue = [&](int gidx) {
        const int key0 = kstart + gidx * 16;
        int page = p.bt[(size_t)b * p.maxp + key0 / p.ps];
        if (page < 0 || page >= p.num_pages) { bad_page = true; page = 0; }
        const int slot = (gidx >> 2) % kDecStages;
        const uint32_t dst = smem_u32(ring + slot * SLOT_BYTES);
        const int row_k = ((page * 2 + 0) * p.nkv + kvh) * p.ps + key0 % p.ps;
        const int row_v = row_k + p.nkv * p.ps;
        mbar_expect_tx(&wbar[slot], SLOT_BYTES);
#pragma unroll
        for (int h = 0; h < DH / 64; ++h) {
            tma_load_3d(dst + h * 2048, &kvmap, &wbar[slot], h * 64, row_k, t);
            tma_load_3d(dst + PAGE_BYTES + h * 2048, &kvmap, &wbar[slot], h * 64, row_v, t);
        }
    };

    const int g_lo = lane >> 2;
    const __nv_bfloat16* qrow = p.q + ((size_t)t * p.M + b) * (size_t)(p.nq * DH) + (size_t)(kvh * G) * DH;
    uint32_t qf[DH / 16][4];
    load_q_frags<DH>(qf, g_lo < G ? qrow + (size_t)g_lo * DH : nullptr, nullptr, lane);
    float o[DH / 8][4];
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m_run = -INFINITY, l_run = 0.f;

    // warp w owns local groups w, w + 4, w + 8, ...
    if (lane == 0)
        for (int s = 0; s < kDecStages; ++s) { int gi = warp + 4 * s; if (gi < npages) issue(gi); }
    bool timed_out = false;
    int it = 0;
    for (int gi = warp; gi < npages; gi += 4, ++it) {
        const int slot = it % kDecStages;
        const uint32_t parity = (it / kDecStages) & 1;
        bool ok = false;
        {
            WaitClock clock;
            for (uint32_t spin = 0; spin < kDecSpin; ++spin) {
                if (mbar_try(&wbar[slot], parity)) { ok = true; break; }
                if ((spin & 255) == 255 && clock.expired()) break;
            }
        }
        if (!__all_sync(0xffffffffu, ok)) { timed_out = true; break; }
        const uint32_t k_base = smem_u32(ring + slot * SLOT_BYTES), v_base = k_base + PAGE_BYTES;
        const int key0 = kstart + gi * 16;
        const int nvalid = key_end - key0;                    // >= 1
        if (nvalid < 16) {                                    // tail of the sequence: unused slots may hold anything
            for (int i = lane; i < (16 - nvalid) * (DH / 8); i += 32) {
                int row = nvalid + i / (DH / 8), chunk = i % (DH / 8);
                *reinterpret_cast<uint4*>(ring + slot * SLOT_BYTES + PAGE_BYTES + page_off<DH>(row, chunk)) = make_uint4(0, 0, 0, 0);
            }
            __syncwarp();
        }
        float s[2][4] = {};
        {
            const int row = (lane >> 4) * 8 + (lane & 7);
            const int cofs = (lane >> 3) & 1;
#pragma unroll
            for (int ks = 0; ks < DH / 16; ++ks) {
                uint32_t b0, b1, b2, b3;
                ldsm_x4(k_base + page_off<DH>(row, ks * 2 + cofs), b0, b1, b2, b3);
                mma_bf16(s[0], qf[ks], b0, b1);
                mma_bf16(s[1], qf[ks], b2, b3);
            }
        }
        float mx = -INFINITY;
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                int key = i * 8 + (lane & 3) * 2 + e;
                float v = key < nvalid ? s[i][e] * p.scale_log2 : -INFINITY;
                s[i][e] = v;
                mx = fmaxf(mx, v);
            }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float mn = fmaxf(m_run, mx);
        const float corr = exp2f(m_run - mn);
        m_run = mn;
        float sum = 0.f;
#pragma unroll
        for (int i = 0; i < 2; ++i) { s[i][0] = exp2f(s[i][0] - mn); s[i][1] = exp2f(s[i][1] - mn); sum += s[i][0] + s[i][1]; }
        l_run = l_run * corr + sum;
        if (__any_sync(0xffffffffu, corr != 1.f)) {
#pragma unroll
            for (int i = 0; i < DH / 8; ++i) { o[i][0] *= corr; o[i][1] *= corr; }
        }
        uint32_t pf[4];
        pf[0] = pack_bf16(s[0][0], s[0][1]); pf[1] = 0u;
        pf[2] = pack_bf16(s[1][0], s[1][1]); pf[3] = 0u;
        {
            const int row = ((lane >> 3) & 1) * 8 + (lane & 7);
            const int cofs = lane >> 4;
#pragma unroll
            for (int dc = 0; dc < DH / 16; ++dc) {
                uint32_t b0, b1, b2, b3;
                ldsm_x4_t(v_base + page_off<DH>(row, dc * 2 + cofs), b0, b1, b2, b3);
                mma_bf16(o[dc * 2], pf, b0, b1);
                mma_bf16(o[dc * 2 + 1], pf, b2, b3);
            }
        }
        __syncwarp();                                         // every lane is done reading the slot
        if (lane == 0) {
            int gn = gi + 4 * kDecStages;
            if (gn < npages) { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); issue(gn); }
        }
    }
    if (timed_out) {
        // give the copies this warp still has in flight a bounded chance to land, then give up
        WaitClock clock;
        for (int s2 = 0; s2 < kDecStages; ++s2)
            for (uint32_t spin = 0; spin < (1u << 16); ++spin) {
                if (mbar_try(&wbar[s2], 0) || mbar_try(&wbar[s2], 1)) break;
                if ((spin & 63) == 63 && clock.expired(100000000ull)) break;
            }
        if (lane == 0) report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_DECODE_PAGE);
    }
    if (bad_page) report(p.status, PT_ERR_DEVICE_BOUNDS, LOC_DECODE_PAGE);
    __syncthreads();                                          // every warp has drained its ring
    decode_merge_store<DH>(p, reinterpret_cast<float*>(smem), o, m_run, l_run, t, b, kvh, split);
}


template <int DH>
__global__ void __launch_bounds__(kThreads)
k_decode_attn(const AttnP p) {
    constexpr int STAGES = 3;
    constexpr int TILE_BYTES = kTileKeys * DH * 2;
    extern __shared__ __align__(128) uint8_t smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int32_t* item = p.items + (size_t)blockIdx.x * 4;
    const int b = item[0], kstart = item[1], kcount = item[2], split = item[3];
    const int kvh = blockIdx.y, t = blockIdx.z;
    const int G = p.nq / p.nkv;
    const __nv_bfloat16* slab = p.pool_l + (size_t)t * p.pool_tstride;
    const int key_end = min(kstart + kcount, p.kvlen[b]);

    const int g_lo = lane >> 2;                               // query head of the group held in the "lo" rows
    const __nv_bfloat16* qrow = p.q + ((size_t)t * p.M + b) * (size_t)(p.nq * DH) + (size_t)(kvh * G) * DH;
    uint32_t qf[DH / 16][4];
    load_q_frags<DH>(qf, g_lo < G ? qrow + (size_t)g_lo * DH : nullptr, nullptr, lane);

    float o[DH / 8][4];
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m_run = -INFINITY, l_run = 0.f;

    const int ntiles = (key_end - kstart + kTileKeys - 1) / kTileKeys;
    bool bad_page = false;
#pragma unroll
    for (int j = 0; j < STAGES - 1; ++j) {
        if (j < ntiles) load_kv_tile<DH>(p, slab, b, kvh, kstart + j * kTileKeys, key_end, smem + j * 2 * TILE_BYTES, smem + j * 2 * TILE_BYTES + TILE_BYTES, bad_page);
        cp_async_commit();
    }
    for (int j = 0; j < ntiles; ++j) {
        cp_async_wait<STAGES - 2>();
        __syncthreads();
        {
            int jn = j + STAGES - 1;
            if (jn < ntiles) {
                uint8_t* nk = smem + (jn % STAGES) * 2 * TILE_BYTES;
                load_kv_tile<DH>(p, slab, b, kvh, kstart + jn * kTileKeys, key_end, nk, nk + TILE_BYTES, bad_page);
            }
            cp_async_commit();
        }
        const uint32_t k_base = smem_u32(smem + (j % STAGES) * 2 * TILE_BYTES), v_base = k_base + TILE_BYTES;
        const int key0 = kstart + j * kTileKeys + warp * 16;  // this warp's 16 keys of the tile
        if (key0 < key_end) {
            float s[2][4] = {};
            qk_16keys<DH>(s, qf, k_base, warp * 16, lane);
            float mx = -INFINITY;
#pragma unroll
            for (int i = 0; i < 2; ++i)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    int key = key0 + i * 8 + (lane & 3) * 2 + e;
                    float v = key < key_end ? s[i][e] * p.scale_log2 : -INFINITY;
                    s[i][e] = v;
                    mx = fmaxf(mx, v);
                }
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float mn = fmaxf(m_run, mx);                // finite: key0 < key_end
            const float corr = exp2f(m_run - mn);
            m_run = mn;
            float sum = 0.f;
#pragma unroll
            for (int i = 0; i < 2; ++i) { s[i][0] = exp2f(s[i][0] - mn); s[i][1] = exp2f(s[i][1] - mn); sum += s[i][0] + s[i][1]; }
            l_run = l_run * corr + sum;
            if (__any_sync(0xffffffffu, corr != 1.f)) {
#pragma unroll
                for (int i = 0; i < DH / 8; ++i) { o[i][0] *= corr; o[i][1] *= corr; }
            }
            uint32_t pf[4];
            pf[0] = pack_bf16(s[0][0], s[0][1]); pf[1] = 0u;
            pf[2] = pack_bf16(s[1][0], s[1][1]); pf[3] = 0u;
            pv_16keys<DH>(o, pf, v_base, warp * 16, lane);
        }
    }
    cp_async_wait<0>();
    __syncthreads();                                          // tiles are dead: reuse shared memory for the merge
    if (bad_page && lane == 0) report(p.status, PT_ERR_DEVICE_BOUNDS, LOC_DECODE_PAGE);
    decode_merge_store<DH>(p, reinterpret_cast<float*>(smem), o, m_run, l_run, t, b, kvh, split);
}

// Merge the key ranges of one (track, sequence, head): one warp each.
template <int DH>
__global__ void k_decode_combine(const AttnP p) {
    grid_dep_wait();
    grid_dep_launch();
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    const int t = blockIdx.y;
    if (warp >= p.B * p.nq) return;
    const int b = warp / p.nq, head = warp % p.nq;
    const int ns = p.nsplit[b];
    if (ns == 1) return;                                       // written by the attention kernel itself
    const float* src = p.part + (((size_t)t * p.B + b) * p.nq + head) * p.max_splits * (DH + 2);
    float M = -INFINITY;
    for (int s = 0; s < ns; ++s) M = fmaxf(M, src[(size_t)s * (DH + 2) + DH]);
    float L = 0.f, acc[DH / 32];
#pragma unroll
    for (int i = 0; i < DH / 32; ++i) acc[i] = 0.f;
    for (int s = 0; s < ns; ++s) {
        const float* ps = src + (size_t)s * (DH + 2);
        float f = ps[DH] == -INFINITY ? 0.f : exp2f(ps[DH] - M);
        L += ps[DH + 1] * f;
#pragma unroll
        for (int i = 0; i < DH / 32; ++i) acc[i] += ps[lane + 32 * i] * f;
    }
    __nv_bfloat16* dst = p.o + ((size_t)t * p.M + b) * (size_t)(p.nq * DH) + (size_t)head * DH;
#pragma unroll
    for (int i = 0; i < DH / 32; ++i) dst[lane + 32 * i] = __float2bfloat16_rn(L > 0.f ? acc[i] / L : 0.f);
}

AttnP make_params(Call& k, const __nv_bfloat16* q, const __nv_bfloat16* pool_l, __nv_bfloat16* o) {
    const pt_config& g = k.m->cfg;
    AttnP p{};
    p.q = q; p.pool_l = pool_l; p.pool_tstride = (int64_t)g.L * k.c->slab_elems; p.o = o;
    p.bt = k.w.meta.bt; p.maxp = k.w.meta.maxp; p.kvlen = k.w.meta.kvlen;
    p.B = k.B; p.S = k.S; p.M = k.M; p.nq = g.heads; p.nkv = g.kv_heads; p.ps = k.c->ps; p.num_pages = k.c->num_pages;
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)k.m->dh);
    p.status = k.m->status();
    p.items = k.items; p.nsplit = k.nsplit; p.part = k.w.part; p.max_splits = kMaxSplits;
    return p;
}

template <class F>
pt_status set_smem(F* fn, int bytes) {
    cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e != cudaSuccess) { set_error("cudaFuncSetAttribute: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
    return PT_OK;
}

}  // namespace

pt_status launch_flash_prefill_p(const AttnP& p, int T, int dh, bool legacy, cudaStream_t st) {
    if (flash_tc_supported(dh, p.ps) && !legacy) return launch_flash_prefill_tc(p, T, dh, st);
    dim3 grid((p.S + 63) / 64, p.nq, T * p.B);
    const int smem = 2 * 2 * kTileKeys * dh * 2;
    pt_status s = PT_OK;
#define GO(DH_) { static bool done_[kMaxDevices] = {}; bool& done = done_[current_device()]; if (!done) { if ((s = set_smem(k_flash_prefill<DH_>, smem)) != PT_OK) return s; done = true; } \
                  k_flash_prefill<DH_><<<grid, kThreads, smem, st>>>(p); }
    if (dh == 32) GO(32) else if (dh == 64) GO(64) else GO(128)
#undef GO
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return PT_OK;
}

pt_status launch_flash_prefill(Call& k, const __nv_bfloat16* q, const __nv_bfloat16* pool_l, __nv_bfloat16* o) {
    AttnP p = make_params(k, q, pool_l, o);
    return launch_flash_prefill_p(p, k.m->cfg.T, k.m->dh, (k.m->cfg.flags & 2) != 0, k.st);
}

pt_status launch_decode_attn_p(const AttnP& p, int T, int dh, int n_items, int max_splits, cudaStream_t st) {
    dim3 grid(n_items, p.nkv, T);
    if (p.ps % 16 == 0 && (dh == 64 || dh == 128)) {
        // tensor map over one layer's slabs: (head_dim, rows of a slab, track); a box is 16 tokens x 128 bytes
        CUtensorMap kvmap;
        pt_status s = make_map_bf16_strided(&kvmap, p.pool_l, dh, (int64_t)p.num_pages * 2 * p.nkv * p.ps, T,
                                            p.pool_tstride * 2, 16);
        if (s != PT_OK) return s;
        const int smem = 1024 + 4 * kDecStages * 2 * 16 * dh * 2 + 4 * kDecStages * 8;
#define GOT(DH_) { static bool done_[kMaxDevices] = {}; bool& done = done_[current_device()]; if (!done) { if ((s = set_smem(k_decode_attn_tma<DH_>, smem)) != PT_OK) return s; done = true; } \
                   launch_dependent(k_decode_attn_tma<DH_>, grid, dim3(kThreads), (size_t)smem, st, kvmap, p); \
                   if (max_splits > 1) { launch_dependent(k_decode_combine<DH_>, dim3((p.B * p.nq * 32 + 127) / 128, T), dim3(128), (size_t)0, st, p); \
                                         g_launches.fetch_add(1, std::memory_order_relaxed); } }
        if (dh == 64) GOT(64) else GOT(128)
#undef GOT
        g_launches.fetch_add(1, std::memory_order_relaxed);
        return PT_OK;
    }
    const int smem = std::max(3 * 2 * kTileKeys * dh * 2, 4 * 8 * (dh + 2) * 4);
    pt_status s = PT_OK;
#define GO(DH_) { static bool done_[kMaxDevices] = {}; bool& done = done_[current_device()]; if (!done) { if ((s = set_smem(k_decode_attn<DH_>, smem)) != PT_OK) return s; done = true; } \
                  k_decode_attn<DH_><<<grid, kThreads, smem, st>>>(p); \
                  if (max_splits > 1) { k_decode_combine<DH_><<<dim3((p.B * p.nq * 32 + 127) / 128, T), 128, 0, st>>>(p); g_launches.fetch_add(1, std::memory_order_relaxed); } }
    if (dh == 32) GO(32) else if (dh == 64) GO(64) else GO(128)
#undef GO
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return PT_OK;
}

pt_status launch_decode_combine(const AttnP& p, int T, int dh, cudaStream_t st) {
    const dim3 grid((p.B * p.nq * 32 + 127) / 128, T);
    cudaError_t e;
    if (dh == 64) e = launch_dependent(k_decode_combine<64>, grid, dim3(128), (size_t)0, st, p);
    else if (dh == 128) e = launch_dependent(k_decode_combine<128>, grid, dim3(128), (size_t)0, st, p);
    else { set_error("no combine kernel for head_dim %d", dh); return PT_ERR_UNSUPPORTED; }
    if (e != cudaSuccess) { set_error("k_decode_combine launch: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return PT_OK;
}

pt_status launch_decode_attn(Call& k, const __nv_bfloat16* q, const __nv_bfloat16* pool_l, __nv_bfloat16* o) {
    AttnP p = make_params(k, q, pool_l, o);
    return launch_decode_attn_p(p, k.m->cfg.T, k.m->dh, k.n_items, k.max_splits, k.st);
}

}  // namespace pt
