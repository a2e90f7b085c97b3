// The E4M3 storage format of the KV cache (pt_kv_dtype PT_KV_E4M3): every cached vector (one token, one KV
// head, K or V) is head_dim 8-bit codes and one power-of-two fp32 scale.
//   k_kv_quant         this call's K and V, as the QKV GEMM left them in the bf16 staging area, into the cache:
//                      one warp per vector finds max|v|, the scale, the codes; for a prefill it also writes
//                      code * scale (exact in bf16: a code has four significant bits) into the bf16 copy the
//                      prefill attention kernel reads
//   k_kv_dequant_ctx   the keys a prefill call's sequences held before the call, code * scale into that copy
//   k_decode_attn_e4m3 split-KV decode attention from the codes on mma.sync (config flag bit 2; the default kernel is the
//                      tcgen05 one in pt_tc_kv8_dec.cu)
#include <cuda_fp8.h>

#include "pt_tc.h"
#include "pt_ptx.cuh"

namespace pt {

namespace {

constexpr int kDh = 128;                   // the format's kernels are written for head_dim 128

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&v);
}
// two codes (low byte first) -> two floats
__device__ __forceinline__ float2 codes_to_float2(uint32_t two) {
    const __half2_raw h = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)two, __NV_E4M3);
    return __half22float2(*reinterpret_cast<const __half2*>(&h));
}

struct QuantP {
    const __nv_bfloat16* stage; int64_t stage_tstride;   // [T][K|V][kv_head][M][dh]
    uint8_t* codes_l; int64_t codes_tstride;             // this layer's slab of track 0; bytes between tracks
    float* scales_l; int64_t scales_tstride;
    const int64_t* row_kvoff;                            // [M] offset of the row's slot (K head 0) inside a slab, in elements
    __nv_bfloat16* attn; int64_t attn_tstride;           // prefill: the attention copy (null for a decode step)
    const int64_t* row_attnoff;
    int M, nvec, ps;                                     // nvec = 2 * kv_heads vectors per row
    int64_t slab_elems;
    int* status;
};

__global__ void k_kv_quant(const QuantP p) {
    grid_dep_wait();
    grid_dep_launch();
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    const int t = blockIdx.y;
    const int nvec = p.nvec;
    if (warp >= p.M * nvec) return;
    const int row = warp / nvec, kvh = warp % nvec;       // kvh = (K|V) * nkv + head
    const uint2 raw = *reinterpret_cast<const uint2*>(p.stage + (size_t)t * p.stage_tstride + ((size_t)kvh * p.M + row) * kDh + lane * 4);
    const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&raw.x), b = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
    const float v0 = __low2float(a), v1 = __high2float(a), v2 = __low2float(b), v3 = __high2float(b);
    float amax = fmaxf(fmaxf(fabsf(v0), fabsf(v1)), fmaxf(fabsf(v2), fabsf(v3)));
#pragma unroll
    for (int o = 16; o; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    // the smallest power of two 2^e >= 2^-100 with amax / 2^e <= 448 = 1.75 * 2^8: with amax = f * 2^x, 1 <= f < 2,
    // e = x - 8, one more when f > 1.75
    const uint32_t bits = __float_as_uint(amax);
    const int xf = (int)(bits >> 23) & 0xff;
    int e = xf == 0 ? -100 : xf - 127 - 8 + ((bits & 0x7fffffu) > 0x600000u ? 1 : 0);
    e = max(e, -100);
    const bool zero = amax == 0.f;
    const float scale = zero ? 1.0f : __uint_as_float((uint32_t)(e + 127) << 23);
    const float inv = zero ? 1.0f : __uint_as_float((uint32_t)(127 - e) << 23);
    const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(v0 * inv, v1 * inv), __NV_SATFINITE, __NV_E4M3);
    const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(v2 * inv, v3 * inv), __NV_SATFINITE, __NV_E4M3);
    const int64_t off = (p.row_kvoff ? p.row_kvoff[row] : (int64_t)row * kDh) + (int64_t)kvh * p.ps * kDh;
    if (off < 0 || off + kDh > p.slab_elems) { if (lane == 0) report(p.status, PT_ERR_DEVICE_BOUNDS, LOC_ROPE_PAGE); return; }
    *reinterpret_cast<uint32_t*>(p.codes_l + (size_t)t * p.codes_tstride + off + lane * 4) = lo | (hi << 16);
    if (lane == 0) p.scales_l[(size_t)t * p.scales_tstride + off / kDh] = scale;
    if (p.attn) {
        const float2 d0 = codes_to_float2(lo), d1 = codes_to_float2(hi);
        uint2 o;
        o.x = pack_bf16(d0.x * scale, d0.y * scale);
        o.y = pack_bf16(d1.x * scale, d1.y * scale);
        *reinterpret_cast<uint2*>(p.attn + (size_t)t * p.attn_tstride + p.row_attnoff[row] + (int64_t)kvh * 16 * kDh + lane * 4) = o;
    }
}

struct CtxP {
    const uint8_t* codes_l; int64_t codes_tstride;
    const float* scales_l; int64_t scales_tstride;
    __nv_bfloat16* attn; int64_t attn_tstride;
    const int32_t* bt; int maxp;                          // the cache's block table
    const int32_t* bt_attn; int maxp_attn;                // 16-token pages of the attention copy
    const int32_t* start;                                 // [B] keys cached before the call
    int nkv, ps, num_pages;
    int* status;
};

__global__ void k_kv_dequant_ctx(const CtxP p) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.y, t = blockIdx.z;
    const int nvec = 2 * p.nkv;
    const int pos = warp / nvec, kvh = warp % nvec;
    if (pos >= p.start[b]) return;
    const int page = p.bt[(size_t)b * p.maxp + pos / p.ps];
    if (page < 0 || page >= p.num_pages) { if (lane == 0) report(p.status, PT_ERR_DEVICE_BOUNDS, LOC_FLASH_PAGE); return; }
    const int64_t vi = ((int64_t)page * nvec + kvh) * p.ps + pos % p.ps;
    const uint32_t w = *reinterpret_cast<const uint32_t*>(p.codes_l + (size_t)t * p.codes_tstride + vi * kDh + lane * 4);
    const float scale = p.scales_l[(size_t)t * p.scales_tstride + vi];
    const float2 d0 = codes_to_float2(w & 0xffffu), d1 = codes_to_float2(w >> 16);
    uint2 o;
    o.x = pack_bf16(d0.x * scale, d0.y * scale);
    o.y = pack_bf16(d1.x * scale, d1.y * scale);
    const int64_t dst = (((int64_t)p.bt_attn[(size_t)b * p.maxp_attn + pos / 16] * nvec + kvh) * 16 + pos % 16) * kDh;
    *reinterpret_cast<uint2*>(p.attn + (size_t)t * p.attn_tstride + dst + lane * 4) = o;
}


// ---- decode attention straight from the codes -------------------------------------------------------
// Same work split as the bf16 kernel: a CTA = one (track, sequence, KV head, key range), each of its 4 warps
// streams its own 16-token groups through a private ring, the G query heads of the KV head are the rows of an
// mma.sync m16n8k16 tile.  A group arrives as ONE copy: a 5-D box that takes the K block and, nkv blocks further, the V
// block of the page in one go (element stride nkv in the (K|V, head) dimension); the 32 scales come as 32 four-byte cp.async
// copies, one per lane.  Codes become f16 (exact) on their way into the MMA's B fragments:
//   scores  the contraction indices kappa {2q, 2q+1, 2q+8, 2q+9} (q = lane % 4) of k-steps 2kk and 2kk+1 are mapped
//           to head_dim 32 kk + 8q + {0..3} and + {4..7}, so a thread's four B registers of two k-steps are one
//           64-bit load of eight consecutive codes of its key's row; q is loaded in the same order.  The K scale
//           multiplies the score.
//   P V     a thread needs the codes of keys {2q, 2q+1, 2q+8, 2q+9} at one head_dim column: it loads four
//           consecutive columns 32 m + 4 g + {0..3} (g = lane / 4) of those four rows and takes byte i of each for
//           the n-tile (m, i), whose column g therefore stands for head_dim 32 m + 4 g + i; the accumulators are
//           put back in order when they are merged.  V codes are multiplied by their scale as f16 pairs, so a
//           cached V value must fit f16 (|v| <= 65504; below 2^-24 it flushes to zero).
// With the 128-byte swizzle of the boxes both access patterns are free of bank conflicts.
// Tried and dropped: both products on mma.sync m16n8k32 with E4M3 operands (q and the probabilities split into two
// E4M3 numbers hi + lo / 16 carried by rows g and g + 8 of the 16-row tile, K and V codes fed to the MMA as they
// are, V transposed by byte permutes).  Results matched the oracle, but on this architecture the compiler lowers
// that MMA to conversions plus f16 MMAs (the profiler shows the HMMA pipe and as many instructions as here):
// 2314 GB/s against 2985 on the same case.  The 8-bit tensor path of this chip is tcgen05 only.
constexpr int kDecStages = 3;
constexpr uint32_t kDecSpin = 1u << 24;
constexpr int kSlotBytes = 2 * 16 * kDh;                  // K box + V box
constexpr int kDecThreads = 128;

__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1, int c2, int c3, int c4) {
    asm volatile("cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
                 ::"r"(dst), "l"((uint64_t)map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void mma_f16(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// four codes (a 32-bit word, low byte first) -> two f16 pairs
__device__ __forceinline__ void codes4_to_half(uint32_t w, uint32_t& lo, uint32_t& hi) {
    asm("{\n .reg .b16 a, b;\n mov.b32 {a, b}, %2;\n cvt.rn.f16x2.e4m3x2 %0, a;\n cvt.rn.f16x2.e4m3x2 %1, b;\n}" : "=r"(lo), "=r"(hi) : "r"(w));
}
__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_half2(float a, float b) {
    const __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<const uint32_t*>(&h);
}
// byte offset of byte `c` of row `r` inside a 16 x 128-byte box in the 128-byte swizzle
__device__ __forceinline__ uint32_t box_off(int r, int c) { return (uint32_t)(r * 128 + ((((c >> 4) ^ (r & 7))) << 4) + (c & 15)); }

struct Dec8P {
    AttnP a;                          // q, o, bt, kvlen, items, nsplit, part ... (pool_l unused)
    const float* scales_l; int64_t scales_tstride;
};

__global__ void __launch_bounds__(kDecThreads, 4)
k_decode_attn_e4m3(const __grid_constant__ CUtensorMap kvmap, const Dec8P pp) {
    const AttnP& p = pp.a;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    float* sc_area = (float*)(smem + 4 * kDecStages * kSlotBytes);              // [warp][stage][K|V][16]
    uint64_t* bars = (uint64_t*)(sc_area + 4 * kDecStages * 32);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    grid_dep_wait();                                          // q and this step's codes come from the kernels before it
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

    uint8_t* ring = smem + warp * kDecStages * kSlotBytes;
    float* wsc = sc_area + warp * kDecStages * 32;
    uint64_t* wbar = bars + warp * kDecStages;
    bool bad_page = false;
    // all lanes: lane 0 starts the copy of the codes of local group gidx into its slot, every lane fetches one scale
    // (lanes 0-15 those of K, 16-31 those of V); one cp.async group per call, so groups complete in issue order
    auto issue = [&](int gidx) {
        const int key0 = kstart + gidx * 16;
        int page = p.bt[(size_t)b * p.maxp + key0 / p.ps];
        if (page < 0 || page >= p.num_pages) { bad_page = true; page = 0; }
        const int slot = (gidx >> 2) % kDecStages;
        if (lane == 0) {
            mbar_expect_tx(&wbar[slot], kSlotBytes);
            tma_load_5d(smem_u32(ring + slot * kSlotBytes), &kvmap, &wbar[slot], 0, key0 % p.ps, kvh, page, t);
        }
        const int64_t vec = ((int64_t)(page * 2 + (lane >> 4)) * p.nkv + kvh) * p.ps + key0 % p.ps + (lane & 15);
        cp_async4(smem_u32(wsc + slot * 32 + lane), pp.scales_l + (size_t)t * pp.scales_tstride + vec);
        cp_async_commit();
    };

    const int g = lane >> 2, q4 = lane & 3;
    // q fragments: k-steps 2kk and 2kk+1 take head_dim 32 kk + 8 q + {0..3} and + {4..7}
    // q is a bf16 vector of any magnitude and f16 is narrow: every head is divided by the power of two at its largest
    // element (so that it lies in [1, 2)) before the conversion and the scores are multiplied by it afterwards.
    uint32_t qf[kDh / 16][4];
    float q_unit = 1.0f;
    {
        const __nv_bfloat16* qrow = p.q + ((size_t)t * p.M + b) * (size_t)(p.nq * kDh) + (size_t)(kvh * G + g) * kDh;
        uint4 raw[kDh / 32];
        float amax = 0.f;
#pragma unroll
        for (int kk = 0; kk < kDh / 32; ++kk) {
            raw[kk] = g < G ? *reinterpret_cast<const uint4*>(qrow + kk * 32 + q4 * 8) : make_uint4(0, 0, 0, 0);
            const uint32_t wds[4] = {raw[kk].x, raw[kk].y, raw[kk].z, raw[kk].w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&wds[i]));
                amax = fmaxf(amax, fmaxf(fabsf(f.x), fabsf(f.y)));
            }
        }
        amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
        amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
        float q_inv = 1.0f;
        {
            const int xf = (int)(__float_as_uint(amax) >> 23) & 0xff;
            if (amax > 0.f && amax <= 3.0e38f) {
                const int e = min(max(xf - 127, -100), 100);
                q_unit = __uint_as_float((uint32_t)(e + 127) << 23);
                q_inv = __uint_as_float((uint32_t)(127 - e) << 23);
            }
        }
#pragma unroll
        for (int kk = 0; kk < kDh / 32; ++kk) {
            const uint32_t wds[4] = {raw[kk].x, raw[kk].y, raw[kk].z, raw[kk].w};
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const float2 f0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&wds[2 * h]));
                const float2 f1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&wds[2 * h + 1]));
                qf[2 * kk + h][0] = pack_half2(f0.x * q_inv, f0.y * q_inv);
                qf[2 * kk + h][1] = 0u;
                qf[2 * kk + h][2] = pack_half2(f1.x * q_inv, f1.y * q_inv);
                qf[2 * kk + h][3] = 0u;
            }
        }
        q_unit *= p.scale_log2;
    }
    // byte offsets inside a slot, fixed for the thread (the swizzle's XOR is folded in once):
    //   K: row g (+8 for the second n-tile), the 8 bytes at head_dim 32 kk + 8 q
    //   V: rows 2q + j (+8), the 4 bytes at head_dim 32 m + 4 g
    uint32_t koff[kDh / 32], voff[kDh / 32][2];
#pragma unroll
    for (int kk = 0; kk < kDh / 32; ++kk) koff[kk] = box_off(g, 32 * kk + 8 * q4);
#pragma unroll
    for (int m = 0; m < kDh / 32; ++m)
#pragma unroll
        for (int j = 0; j < 2; ++j) voff[m][j] = 16 * kDh + box_off(2 * q4 + j, 32 * m + 4 * g);
    float o[kDh / 8][4];
#pragma unroll
    for (int i = 0; i < kDh / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    // The V codes enter the MMA as they are (exact in f16); a key's V scale goes into its probability, relative to the
    // largest V scale this warp has met (v_ref, a power of two; the accumulator is rescaled when it grows), so that
    // neither large nor small magnitudes of V leave the f16 range.
    float m_run = -INFINITY, l_run = 0.f, v_ref = 0.f;

#pragma unroll
    for (int s = 0; s < kDecStages; ++s) { int gi = warp + 4 * s; if (gi < npages) issue(gi); else cp_async_commit(); }
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
        cp_async_wait<kDecStages - 1>();                      // this group's scales (the groups after it may still be in flight)
        __syncwarp();
        const uint32_t sb = smem_u32(ring + slot * kSlotBytes);
        const float* scs = wsc + slot * 32;
        const int nvalid = key_end - (kstart + gi * 16);      // >= 1
        if (nvalid < 16) {                                    // tail of the sequence: unused slots may hold anything
            uint8_t* vb = ring + slot * kSlotBytes + 16 * kDh;
            for (int i = lane; i < (16 - nvalid) * 8; i += 32)
                *reinterpret_cast<uint4*>(vb + (nvalid + i / 8) * 128 + (i % 8) * 16) = make_uint4(0, 0, 0, 0);
            __syncwarp();
        }
        // this thread's four keys: 2q, 2q+1, 2q+8, 2q+9 (score columns and P V contraction rows alike)
        float2 sk01 = *reinterpret_cast<const float2*>(scs + 2 * q4), sk89 = *reinterpret_cast<const float2*>(scs + 8 + 2 * q4);
        float2 sv01 = *reinterpret_cast<const float2*>(scs + 16 + 2 * q4), sv89 = *reinterpret_cast<const float2*>(scs + 24 + 2 * q4);
        float s[2][4] = {};
#pragma unroll
        for (int kk = 0; kk < kDh / 32; ++kk) {
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
                uint32_t w0, w1, b0, b1, b2, b3;
                asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(w0), "=r"(w1) : "r"(sb + koff[kk] + nt * 1024));
                codes4_to_half(w0, b0, b1);
                codes4_to_half(w1, b2, b3);
                mma_f16(s[nt], qf[2 * kk], b0, b1);
                mma_f16(s[nt], qf[2 * kk + 1], b2, b3);
            }
        }
        s[0][0] *= sk01.x * q_unit; s[0][1] *= sk01.y * q_unit;
        s[1][0] *= sk89.x * q_unit; s[1][1] *= sk89.y * q_unit;
        if (nvalid < 16) {
            if (2 * q4 >= nvalid) { s[0][0] = -INFINITY; sv01.x = 0.f; }
            if (2 * q4 + 1 >= nvalid) { s[0][1] = -INFINITY; sv01.y = 0.f; }
            if (2 * q4 + 8 >= nvalid) { s[1][0] = -INFINITY; sv89.x = 0.f; }
            if (2 * q4 + 9 >= nvalid) { s[1][1] = -INFINITY; sv89.y = 0.f; }
        }
        float mx = fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float mn = fmaxf(m_run, mx);
        const float corr = ex2f(m_run - mn);
        m_run = mn;
        s[0][0] = ex2f(s[0][0] - mn); s[0][1] = ex2f(s[0][1] - mn);
        s[1][0] = ex2f(s[1][0] - mn); s[1][1] = ex2f(s[1][1] - mn);
        l_run = l_run * corr + ((s[0][0] + s[0][1]) + (s[1][0] + s[1][1]));
        float vmax = fmaxf(fmaxf(sv01.x, sv01.y), fmaxf(sv89.x, sv89.y));     // over the group's 16 keys (the same in every row g)
        vmax = fmaxf(vmax, __shfl_xor_sync(0xffffffffu, vmax, 1));
        vmax = fmaxf(vmax, __shfl_xor_sync(0xffffffffu, vmax, 2));
        float ocorr = corr;
        if (vmax > v_ref) { ocorr *= v_ref / vmax; v_ref = vmax; }           // powers of two: exact (v_ref starts at 0)
        if (__any_sync(0xffffffffu, ocorr != 1.f)) {
#pragma unroll
            for (int i = 0; i < kDh / 8; ++i) { o[i][0] *= ocorr; o[i][1] *= ocorr; }
        }
        const float vinv = v_ref > 0.f ? 1.0f / v_ref : 0.f;
        uint32_t pf[4];
        pf[0] = pack_half2(s[0][0] * (sv01.x * vinv), s[0][1] * (sv01.y * vinv)); pf[1] = 0u;
        pf[2] = pack_half2(s[1][0] * (sv89.x * vinv), s[1][1] * (sv89.y * vinv)); pf[3] = 0u;
#pragma unroll
        for (int m = 0; m < kDh / 32; ++m) {
            uint32_t w0, w1, w2, w3;
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w0) : "r"(sb + voff[m][0]));
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w1) : "r"(sb + voff[m][1]));
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w2) : "r"(sb + voff[m][0] + 1024));
            asm volatile("ld.shared.u32 %0, [%1];" : "=r"(w3) : "r"(sb + voff[m][1] + 1024));
            // bytes (i, i + 1) of two rows side by side: [r0.b_i, r1.b_i, r0.b_i+1, r1.b_i+1]
            const uint32_t a01 = __byte_perm(w0, w1, 0x5140), a23 = __byte_perm(w0, w1, 0x7362);
            const uint32_t c01 = __byte_perm(w2, w3, 0x5140), c23 = __byte_perm(w2, w3, 0x7362);
            uint32_t b0[4], b1[4];
            codes4_to_half(a01, b0[0], b0[1]); codes4_to_half(a23, b0[2], b0[3]);
            codes4_to_half(c01, b1[0], b1[1]); codes4_to_half(c23, b1[2], b1[3]);
#pragma unroll
            for (int i = 0; i < 4; ++i) mma_f16(o[m * 4 + i], pf, b0[i], b1[i]);
        }
        __syncwarp();                                         // every lane is done reading the slot
        {
            const int gn = gi + 4 * kDecStages;
            if (gn < npages) { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); issue(gn); }
            else cp_async_commit();                           // keeps "all but the last kDecStages - 1 groups" meaning this group's successor
        }
    }
    cp_async_wait<0>();
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

    // merge the four warps' partial (max, sum, output) of the G query heads through shared memory; accumulator
    // (n-tile nt, column 2q + j) holds head_dim 32 (nt / 4) + 4 (2q + j) + nt % 4
    float* mg = reinterpret_cast<float*>(smem);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    if (g < G) {
        float* dst = mg + ((size_t)warp * 8 + g) * (kDh + 2);
#pragma unroll
        for (int nt = 0; nt < kDh / 8; ++nt) {
            const int d0 = 32 * (nt >> 2) + 8 * q4 + (nt & 3);
            dst[d0] = o[nt][0] * v_ref; dst[d0 + 4] = o[nt][1] * v_ref;
        }
        if (q4 == 0) { dst[kDh] = m_run; dst[kDh + 1] = l_run; }
    }
    __syncthreads();
    const int ns = p.nsplit[b];
    for (int idx = threadIdx.x; idx < G * kDh; idx += kDecThreads) {
        const int gg = idx / kDh, d = idx % kDh;
        float Mx = -INFINITY;
#pragma unroll
        for (int w = 0; w < 4; ++w) Mx = fmaxf(Mx, mg[((size_t)w * 8 + gg) * (kDh + 2) + kDh]);
        float L = 0.f, acc = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const float* src = mg + ((size_t)w * 8 + gg) * (kDh + 2);
            const float f = src[kDh] == -INFINITY ? 0.f : exp2f(src[kDh] - Mx);
            L += src[kDh + 1] * f;
            acc += src[d] * f;
        }
        const int head = kvh * G + gg;
        if (ns == 1) {
            p.o[((size_t)t * p.M + b) * (size_t)(p.nq * kDh) + (size_t)head * kDh + d] = __float2bfloat16_rn(L > 0.f ? acc / L : 0.f);
        } else {
            float* dst = p.part + ((((size_t)t * p.B + b) * p.nq + head) * p.max_splits + split) * (kDh + 2);
            dst[d] = acc;
            if (d == 0) { dst[kDh] = Mx; dst[kDh + 1] = L; }
        }
    }
}

// (code byte, slot, (K|V, head), page, track): a box is the 16 x 128 code bytes of one 16-token group of a K block and,
// through the element stride nkv of the third dimension, of the V block of the same head
pt_status make_codes_map(CUtensorMap* out, const void* base, int ps, int nkv, int64_t pages, int64_t tracks, int64_t track_stride_bytes) {
    EncodeFn enc = get_encode();
    if (!enc) { set_error("cuTensorMapEncodeTiled is not available from this driver"); return PT_ERR_CUDA; }
    if (nkv > 8) { set_error("an E4M3 cache supports up to 8 KV heads per track"); return PT_ERR_UNSUPPORTED; }
    cuuint64_t dims[5] = {(cuuint64_t)kDh, (cuuint64_t)ps, (cuuint64_t)(2 * nkv), (cuuint64_t)pages, (cuuint64_t)tracks};
    cuuint64_t strides[4] = {(cuuint64_t)kDh, (cuuint64_t)ps * kDh, (cuuint64_t)2 * nkv * ps * kDh, (cuuint64_t)track_stride_bytes};
    cuuint32_t box[5] = {(cuuint32_t)kDh, 16, (cuuint32_t)(nkv + 1), 1, 1};
    cuuint32_t es[5] = {1, 1, (cuuint32_t)nkv, 1, 1};
    CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 5, const_cast<void*>(base), dims, strides, box, es,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled (E4M3 cache) failed with code %d", (int)r); return PT_ERR_CUDA; }
    return PT_OK;
}

}  // namespace

pt_status launch_kv_quant(Call& k, int layer) {
    const pt_model* m = k.m;
    const pt_kv_cache* c = k.c;
    const pt_config& g = m->cfg;
    QuantP p{};
    p.stage = (const __nv_bfloat16*)k.w.kv_stage; p.stage_tstride = (int64_t)2 * m->KVD * k.M;
    p.codes_l = (uint8_t*)c->pool + (size_t)layer * c->slab_elems; p.codes_tstride = (int64_t)g.L * c->slab_elems;
    p.scales_l = c->scales + (size_t)layer * c->slab_vecs(); p.scales_tstride = (int64_t)g.L * c->slab_vecs();
    p.row_kvoff = k.w.meta.row_kvoff;
    p.attn = k.decode ? nullptr : (__nv_bfloat16*)k.w.attn_kv;
    p.attn_tstride = (int64_t)k.w.meta.attn_pages * 2 * m->KVD * 16;
    p.row_attnoff = k.w.meta.row_attnoff;
    p.M = k.M; p.nvec = 2 * g.kv_heads; p.ps = c->ps; p.slab_elems = c->slab_elems; p.status = m->status();
    const unsigned blocks = (unsigned)(((size_t)k.M * 2 * g.kv_heads + 7) / 8);
    cudaError_t e = launch_dependent(k_kv_quant, dim3(blocks, g.T), dim3(256), (size_t)0, k.st, p);
    if (e != cudaSuccess) { set_error("k_kv_quant launch: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return PT_OK;
}

pt_status launch_kv_dequant_ctx(Call& k, int layer) {
    const pt_model* m = k.m;
    const pt_kv_cache* c = k.c;
    const pt_config& g = m->cfg;
    if (k.w.meta.max_start <= 0) return PT_OK;
    CtxP p{};
    p.codes_l = (const uint8_t*)c->pool + (size_t)layer * c->slab_elems; p.codes_tstride = (int64_t)g.L * c->slab_elems;
    p.scales_l = c->scales + (size_t)layer * c->slab_vecs(); p.scales_tstride = (int64_t)g.L * c->slab_vecs();
    p.attn = (__nv_bfloat16*)k.w.attn_kv; p.attn_tstride = (int64_t)k.w.meta.attn_pages * 2 * m->KVD * 16;
    p.bt = k.w.meta.bt; p.maxp = k.w.meta.maxp; p.bt_attn = k.w.meta.bt_attn; p.maxp_attn = k.w.meta.maxp_attn;
    p.start = k.w.meta.ctx_start; p.nkv = g.kv_heads; p.ps = c->ps; p.num_pages = c->num_pages; p.status = m->status();
    const unsigned blocks = (unsigned)(((size_t)k.w.meta.max_start * 2 * g.kv_heads + 7) / 8);
    k_kv_dequant_ctx<<<dim3(blocks, k.B, g.T), 256, 0, k.st>>>(p);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return PT_OK;
}

// Prefill attention of a call on an E4M3 cache: the tensor-memory kernel over the bf16 copy of code * scale.
pt_status launch_flash_prefill_e4m3(Call& k, const __nv_bfloat16* q, __nv_bfloat16* o) {
    const pt_model* m = k.m;
    const pt_config& g = m->cfg;
    AttnP p{};
    p.q = q; p.o = o;
    p.pool_l = (const __nv_bfloat16*)k.w.attn_kv; p.pool_tstride = (int64_t)k.w.meta.attn_pages * 2 * m->KVD * 16;
    p.bt = k.w.meta.bt_attn; p.maxp = k.w.meta.maxp_attn; p.kvlen = k.w.meta.kvlen;
    p.B = k.B; p.S = k.S; p.M = k.M; p.nq = g.heads; p.nkv = g.kv_heads; p.ps = 16; p.num_pages = k.w.meta.attn_pages;
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)m->dh);
    p.status = m->status();
    return launch_flash_prefill_p(p, g.T, m->dh, (g.flags & 2) != 0, k.st);
}

pt_status launch_decode_attn_e4m3_p(const AttnP& p, const Kv8Slab& slab, int T, int n_items, int max_splits, bool mma_sync, cudaStream_t st) {
    if (!mma_sync && n_items <= 65535) return launch_decode_attn_e4m3_tc(p, slab, T, n_items, max_splits, st);   // its key ranges are grid.y
    Dec8P pp{};
    pp.a = p;
    pp.scales_l = slab.scales_l; pp.scales_tstride = slab.scales_tstride;
    CUtensorMap kvmap;
    pt_status s = make_codes_map(&kvmap, slab.codes_l, p.ps, p.nkv, p.num_pages, T, slab.codes_tstride);
    if (s != PT_OK) return s;
    const int smem = 1024 + 4 * kDecStages * kSlotBytes + 4 * kDecStages * 32 * 4 + 4 * kDecStages * 8;
    static bool done_[kMaxDevices] = {};
    bool& done = done_[current_device()];
    if (!done) {
        cudaError_t e = cudaFuncSetAttribute(k_decode_attn_e4m3, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) { set_error("cudaFuncSetAttribute: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
        done = true;
    }
    cudaError_t e = launch_dependent(k_decode_attn_e4m3, dim3(n_items, p.nkv, T), dim3(kDecThreads), (size_t)smem, st, kvmap, pp);
    if (e != cudaSuccess) { set_error("k_decode_attn_e4m3 launch: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (max_splits > 1) return launch_decode_combine(p, T, kDh, st);
    return PT_OK;
}

pt_status launch_decode_attn_e4m3(Call& k, const __nv_bfloat16* q, int layer, __nv_bfloat16* o) {
    const pt_model* m = k.m;
    const pt_kv_cache* c = k.c;
    const pt_config& g = m->cfg;
    AttnP p{};
    p.q = q; p.o = o; p.bt = k.w.meta.bt; p.maxp = k.w.meta.maxp; p.kvlen = k.w.meta.kvlen;
    p.B = k.B; p.S = 1; p.M = k.M; p.nq = g.heads; p.nkv = g.kv_heads; p.ps = c->ps; p.num_pages = c->num_pages;
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)m->dh);
    p.status = m->status();
    p.items = k.items; p.nsplit = k.nsplit; p.part = k.w.part; p.max_splits = kMaxSplits;
    Kv8Slab slab{};
    slab.codes_l = (const uint8_t*)c->pool + (size_t)layer * c->slab_elems; slab.codes_tstride = (int64_t)g.L * c->slab_elems;
    slab.scales_l = c->scales + (size_t)layer * c->slab_vecs(); slab.scales_tstride = (int64_t)g.L * c->slab_vecs();
    return launch_decode_attn_e4m3_p(p, slab, g.T, k.n_items, k.max_splits, (g.flags & 4) != 0, k.st);
}

}  // namespace pt

#include "pt_kernels.h"

extern "C" pt_status pt_kernel_kv_quant_e4m3(const void* src, void* codes, float* scales, int64_t n, void* status, void* stream) {
    using namespace pt;
    if (!src || !codes || !scales || !status) { set_error("null argument"); return PT_ERR_INVALID_ARG; }
    if (n < 1 || n > (1 << 28)) { set_error("n outside [1, 2^28]"); return PT_ERR_INVALID_ARG; }
    if ((uintptr_t)src % 8 || (uintptr_t)codes % 4 || (uintptr_t)scales % 4) { set_error("src must be 8-byte, codes and scales 4-byte aligned"); return PT_ERR_MISALIGNED; }
    QuantP p{};
    p.stage = (const __nv_bfloat16*)src; p.codes_l = (uint8_t*)codes; p.scales_l = scales;
    p.M = (int)n; p.nvec = 1; p.ps = 1; p.slab_elems = n * 128; p.status = (int*)status;
    k_kv_quant<<<dim3((unsigned)((n + 7) / 8), 1), 256, 0, (cudaStream_t)stream>>>(p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("kernel launch failed: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return PT_OK;
}
