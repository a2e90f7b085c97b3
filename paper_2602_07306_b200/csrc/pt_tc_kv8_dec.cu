// Split-KV decode attention over an E4M3 KV cache on the 5th-generation tensor cores (tcgen05, kind::f8f6f4):
// the 8-bit codes go from the cache pages through TMA into shared memory and from there straight into the MMA,
// no thread ever touches them.
//
// The KEYS are the M dimension.  A CTA owns one (track, sequence, KV head, key range) and walks it in tiles of
// 128 keys:
//     S^T = K_tile Q8^T       [128 keys x 16]   A = the K codes as they lie in the cache (K-major), B = q
//     O^T += V_tile^T P8      [128 head_dim x 16]   A = the V codes, read MN-major (head_dim contiguous), B = P
// q and the probabilities are not 8-bit data: each is split into two E4M3 numbers, x ~ hi + lo / 16 (hi = e4m3(x),
// lo = e4m3(16 (x - hi)): relative error 2^-8 where lo is a normal code).  The 16 columns are the G <= 8 query heads
// of the KV head (hi parts) and the same heads again (lo parts), so one MMA gives both partial products and the
// narrowest N of a 128-row MMA is used in full.  q is scaled per head by a power of two so that its largest element
// lands below 448; the probabilities by 64 / (the largest V scale met so far).
// With keys on M every per-key quantity is a per-thread scalar: softmax thread r of 128 owns key r of the tile - its
// K scale multiplies its 8 scores, its V scale its 8 probabilities, its row sums stay in registers until the end.
// Only the tile's maxima (8 heads and the V scale) cross threads: redux.sync per warp, 36 floats of shared memory
// and one named barrier per tile.  The reference maximum is raised only when it grows by more than 2^2 (the
// accumulator is then rescaled in tensor memory), so rescales are rare; the bound keeps 64 p inside the E4M3 range.
// Roles: warp 0 streams K and V tiles page by page with TMA (one 16 x 128-byte box per page and K|V) through
// two-stage rings (so that three CTAs fit an SM: the kernel is bound by the latency of its copies, more CTAs hide it); warp 1 issues the MMAs (the scores of tile j+2 right behind P V of tile j: S^T is double-buffered in
// tensor memory, P in shared memory); warps 2-5 are the softmax threads.  Every mbarrier wait is bounded; the named
// barrier is executed exactly once per tile and twice at the end by every softmax warp whatever happened before.
#include <cuda_fp8.h>

#include "pt_tc.h"
#include "pt_ptx.cuh"

namespace pt {

namespace {

constexpr int kDh = 128;
constexpr int kThreads = 192;
// A CTA's start and drain cost about as much as three or four of its tiles (256 sequences, the same bytes: 18 tiles per
// CTA 0.92 of the copy bandwidth, 9 tiles 0.80, 4.5 tiles 0.56), which is why the split plan avoids short key ranges.  A
// persistent form of this kernel (three CTAs per SM walking the work list in alternating directions, ring stages and
// barrier phases counted across units so that the next unit's copies start under the last tiles of the current one)
// was built and was slower: 0.73 against 0.92 with 18 tiles per unit, 0.66 against 0.88 on the ragged batch.
// Measured alternative, kept as compile-time switches: one K stage and four CTAs per SM (56 KB of shared memory each;
// 80 registers per thread, a few spills): 5 % slower in both E4M3 decode workloads; one K stage at three CTAs: no change.
#ifndef T8_KSTAGES
#define T8_KSTAGES 2
#endif
#ifndef T8_CTAS
#define T8_CTAS 3
#endif
constexpr int kStagesK = T8_KSTAGES;        // K ring (a K tile is free again as soon as its scores are issued)
constexpr int kStages = 2;                  // V ring
constexpr int kTile = 128 * kDh;            // bytes of a K or V tile: 128 keys x 128 code bytes
constexpr int kQBytes = 16 * kDh;           // q (and one P buffer): 16 rows of 128 bytes
constexpr uint32_t kSpin = 1u << 26;
// A head's reference maximum is raised (and the accumulator rescaled) when a tile's maximum exceeds it by more than
// this many powers of two.  Until then a probability can reach 2^kLazyLog2; times the factor 64 of the P codes that
// must stay inside the E4M3 range: 4 * 64 = 256 <= 448.
#ifndef T8_LAZY_LOG2
#define T8_LAZY_LOG2 2.0f
#endif
constexpr float kLazyLog2 = T8_LAZY_LOG2;

enum { B_KFULL = 0, B_KEMPTY = 3, B_VFULL = 6, B_VEMPTY = 9, B_SFULL = 12, B_SEMPTY = 14, B_PFULL = 16, B_PEMPTY = 18,
       B_VRAW = 20, B_COUNT = 21 };

// (A suspend-time hint on mbarrier.try_wait, 1 or 10 us, was measured: no gain.)
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, bool relaxed = false) {
    WaitClock clock;
    for (uint32_t i = 0; i < kSpin; ++i) {
        if (mbar_try(bar, parity)) return true;
        if (relaxed && i >= 2) __nanosleep(64);
        if ((i & 255) == 255 && (*abort_flag || clock.expired())) return false;
    }
    return false;
}
// D[tmem] (+)= A[smem] * B[smem], both operands E4M3
__device__ __forceinline__ void mma_f8(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n .reg .pred p, e;\n elect.sync _|e, 0xffffffff;\n setp.ne.b32 p, %4, 0;\n @e tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n}"
                 ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void tm_ld16(uint32_t taddr, float* v) {
    uint32_t r[16];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr) : "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tm_st16(uint32_t taddr, const float* v) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
                 "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
                 ::"r"(taddr),
                   "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
                   "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
                   "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
                   "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15]))
                 : "memory");
}
__device__ __forceinline__ void tm_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tm_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// float <-> an integer with the same order (so that redux.sync.max can reduce floats, -inf included)
__device__ __forceinline__ int f2ord(float x) { int i = __float_as_int(x); return i ^ ((i >> 31) & 0x7fffffff); }
__device__ __forceinline__ float ord2f(int i) { return __int_as_float(i ^ ((i >> 31) & 0x7fffffff)); }

// two values -> (hi codes, lo codes) of the split x ~ hi + lo / 16, two codes each (first value in the low byte)
__device__ __forceinline__ void split2(float x0, float x1, uint32_t& hi, uint32_t& lo) {
    hi = __nv_cvt_float2_to_fp8x2(make_float2(x0, x1), __NV_SATFINITE, __NV_E4M3);
    const __half2_raw h = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)hi, __NV_E4M3);
    const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&h));
    lo = __nv_cvt_float2_to_fp8x2(make_float2((x0 - b.x) * 16.f, (x1 - b.y) * 16.f), __NV_SATFINITE, __NV_E4M3);
}
// byte offset of byte `c` of row `r` of a tile of 128-byte rows in the 128-byte swizzle
__device__ __forceinline__ uint32_t row_off(int r, int c) { return (uint32_t)(r * 128 + ((((c >> 4) ^ (r & 7))) << 4) + (c & 15)); }

// Shared-memory descriptors (128-byte swizzle, 8-row groups 1024 bytes apart): a K-major operand (rows of 128
// contraction bytes) and an MN-major one (rows are contraction steps, the 128 bytes of a row the M extent).
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFF) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFF) >> 4);
    d |= (uint64_t)(kTile >> 4) << 16;          // distance between 128-byte column blocks: there is only one
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

struct Dec8TcP {
    AttnP a;                          // q, o, bt, kvlen, items, nsplit, part ... (pool_l unused)
    const float* scales_l; int64_t scales_tstride;
};

constexpr int kSmem = 1024 + (kStagesK + kStages) * kTile + kQBytes + 2 * kQBytes + 2 * 4 * 12 * 4 + 8 * 4 + B_COUNT * 8 + 64;

__global__ void __launch_bounds__(kThreads, T8_CTAS)
k_decode_attn_e4m3_tc(const __grid_constant__ CUtensorMap kvmap, const Dec8TcP pp) {
    const AttnP& p = pp.a;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sk = smem;
    uint8_t* sv = sk + kStagesK * kTile;
    uint8_t* sq = sv + kStages * kTile;                      // q: rows 0-7 hi parts of the heads, 8-15 their lo parts
    uint8_t* sp = sq + kQBytes;                               // two P buffers of the same shape
    float* red = (float*)(sp + 2 * kQBytes);                  // [parity][warp][12]: tile maxima of 8 heads and of the V scale
    float* q_unit = red + 2 * 4 * 12;                         // [8] the power of two each head's q was divided by, times log2(e)/sqrt(dh)
    uint64_t* bars = (uint64_t*)(q_unit + 8);
    uint32_t* tmem_slot = (uint32_t*)(bars + B_COUNT);
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // the KV heads of one (track, sequence, key range) are neighbours in the grid: CTAs that run together read
    // neighbouring 2 KB blocks of the same pages
    const int32_t* item = p.items + (size_t)blockIdx.y * 4;
    const int b = item[0], kstart = item[1], kcount = item[2], split = item[3];
    const int kvh = blockIdx.x, t = blockIdx.z;
    const int G = p.nq / p.nkv;

    if (threadIdx.x == 0) {
        for (int i = 0; i < B_COUNT; ++i)
            mbar_init(&bars[i], ((i >= B_SEMPTY && i < B_SEMPTY + 2) || (i >= B_PFULL && i < B_PFULL + 2)) ? 4 : 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(64) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    grid_dep_wait();                                          // q and this step's codes come from the kernels before it
    grid_dep_launch();
    const int key_end = min(kstart + kcount, p.kvlen[b]);
    const int n_tiles = (key_end - kstart + 127) >> 7;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;                    // S^T buffers at columns 0 and 16, O^T at column 32

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer.  K and V advance on their own
        // counters: a K tile is requested the moment its stage is free (two tiles before its scores are issued) and never
        // queues behind the wait for a V stage, which frees a tile later.  One bounded polling loop serves both.
        bool bad_page = false;
        int jk = 0, jv = 0;
        WaitClock clock;
        uint32_t idle = 0;
        auto rows_of = [&](int j, int& ng) {                       // lane < ng: first vector of the lane's 16-key group of tile j
            const int key0 = kstart + j * 128;
            ng = min(8, (key_end - key0 + 15) >> 4);
            int row_k = 0;
            if (lane < ng) {
                const int key = key0 + lane * 16;
                int page = p.bt[(size_t)b * p.maxp + key / p.ps];
                if (page < 0 || page >= p.num_pages) { bad_page = true; page = 0; }
                row_k = (page * 2 * p.nkv + kvh) * p.ps + key % p.ps;
            }
            return row_k;
        };
        while (jk < n_tiles || jv < n_tiles) {
            bool progressed = false;
            if (jk < n_tiles && __any_sync(0xffffffffu, mbar_try(&bars[B_KEMPTY + jk % kStagesK], ((uint32_t)(jk / kStagesK) & 1u) ^ 1u))) {
                const int s = jk % kStagesK;
                int ng;
                const int row_k = rows_of(jk, ng);
                if (lane == 0) mbar_expect_tx(&bars[B_KFULL + s], (uint32_t)ng * 16u * kDh);
                __syncwarp();
                if (lane < ng) tma_load_3d(smem_u32(sk + s * kTile + lane * 2048), &kvmap, &bars[B_KFULL + s], 0, row_k, t);
                ++jk; progressed = true;
            }
            if (jv < n_tiles && __any_sync(0xffffffffu, mbar_try(&bars[B_VEMPTY + jv % kStages], ((uint32_t)(jv / kStages) & 1u) ^ 1u))) {
                const int s = jv % kStages;
                int ng;
                const int row_k = rows_of(jv, ng);
                const int key0 = kstart + jv * 128;
                const bool partial = key0 + 128 > key_end;         // rows past the last key must read as zero
                uint64_t* vbar = partial ? &bars[B_VRAW] : &bars[B_VFULL + s];
                if (lane == 0) mbar_expect_tx(vbar, (uint32_t)ng * 16u * kDh);
                __syncwarp();
                if (lane < ng) tma_load_3d(smem_u32(sv + s * kTile + lane * 2048), &kvmap, vbar, 0, row_k + p.nkv * p.ps, t);
                if (partial) {                                     // at most once per CTA: its last tile
                    if (!mbar_wait(&bars[B_VRAW], 0u, abort_flag)) { if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_FLASH_VRAW); *abort_flag = 1; } break; }
                    const int nvalid = key_end - key0;
                    for (int idx = lane; idx < (128 - nvalid) * 8; idx += 32)
                        *reinterpret_cast<uint4*>(sv + s * kTile + (nvalid + idx / 8) * 128 + (idx % 8) * 16) = make_uint4(0, 0, 0, 0);
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars[B_VFULL + s]);
                }
                ++jv; progressed = true;
            }
            if (progressed) { idle = 0; clock = WaitClock(); continue; }
            __nanosleep(64);
            if ((++idle & 255u) == 255u && (*abort_flag || clock.expired() || idle > kSpin)) {
                if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, jk < n_tiles ? LOC_FLASH_KEMPTY : LOC_FLASH_VEMPTY); *abort_flag = 1; }
                break;
            }
        }
        if (bad_page) report(p.status, PT_ERR_DEVICE_BOUNDS, LOC_DECODE_PAGE);
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (whole warp, one elected lane per instruction)
        constexpr uint32_t idesc_qk = (1u << 4) | ((uint32_t)(16 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        constexpr uint32_t idesc_pv = idesc_qk | (1u << 15);       // A (the V codes) is MN-major
        bool ok = true;
        auto wait = [&](int bar, uint32_t parity, int loc) {
            if (!ok) return;
            if (!__all_sync(0xffffffffu, mbar_wait(&bars[bar], parity, abort_flag))) { ok = false; if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, loc); *abort_flag = 1; } }
            tc_fence_after();
        };
        auto qk = [&](int j) {                                 // S^T[j & 1] = K_j q^T
            const int s = j % kStagesK, bb = j & 1;
            wait(B_KFULL + s, (uint32_t)(j / kStagesK) & 1u, LOC_FLASH_KFULL);
            wait(B_SEMPTY + bb, ((uint32_t)(j >> 1) & 1u) ^ 1u, LOC_FLASH_SFULL);
            if (!ok) return;
            const uint32_t ka = smem_u32(sk + s * kTile), qa = smem_u32(sq);
#pragma unroll
            for (int ks = 0; ks < kDh / 32; ++ks)
                mma_f8(tmem_base + bb * 16, desc_kmajor(ka + ks * 32), desc_kmajor(qa + ks * 32), idesc_qk, ks != 0);
            tc_commit(&bars[B_SFULL + bb]);
            tc_commit(&bars[B_KEMPTY + s]);
        };
        // the softmax warps write q before their first arrival at anything the MMA waits on: B_SEMPTY's first phase
        // is free, so q is guarded by its own arrival on B_PFULL + 1 (see there)
        wait(B_PFULL + 1, 0u, LOC_FLASH_QFULL);
        if (n_tiles > 0) qk(0);
        if (n_tiles > 1) qk(1);
        for (int j = 0; j < n_tiles && ok; ++j) {
            const int s = j % kStages, bb = j & 1;
            // P buffer bb: the q hand-over used one phase of B_PFULL + 1, so that barrier runs one phase ahead
            wait(B_PFULL + bb, ((uint32_t)(j >> 1) + (bb ? 1u : 0u)) & 1u, LOC_FLASH_PFULL);
            wait(B_VFULL + s, (uint32_t)(j / kStages) & 1u, LOC_FLASH_VFULL);
            if (!ok) break;
            const uint32_t va = smem_u32(sv + s * kTile), pa = smem_u32(sp + bb * kQBytes);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
                mma_f8(tmem_base + 32, desc_mnmajor(va + ks * 4096), desc_kmajor(pa + ks * 32), idesc_pv, j > 0 || ks != 0);
            tc_commit(&bars[B_PEMPTY + bb]);
            tc_commit(&bars[B_VEMPTY + s]);
            if (j + 2 < n_tiles) qk(j + 2);                    // scores run two tiles ahead of the softmax threads
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ softmax threads: one key of the tile each
        const int sw = warp - 2;                                   // 0..3
        const int quarter = warp & 3;                              // the tensor-memory lanes this warp reaches
        const int row = quarter * 32 + lane;                       // key of the tile; at the end, head_dim index
        const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const int tid = sw * 32 + lane;
        // q: thread (head h = tid / 16, chunk c = tid % 16) scales, splits and stores 8 values of head h
        {
            const int h = tid >> 4, c = tid & 15;
            float qv[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) qv[i] = 0.f;
            if (h < G) {
                const uint4 raw = *reinterpret_cast<const uint4*>(p.q + ((size_t)t * p.M + b) * (size_t)(p.nq * kDh) + (size_t)(kvh * G + h) * kDh + c * 8);
                const uint32_t wds[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&wds[i]));
                    qv[2 * i] = f.x; qv[2 * i + 1] = f.y;
                }
            }
            float amax = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(qv[i]));
#pragma unroll
            for (int o = 8; o; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
            const uint32_t bits = __float_as_uint(amax);
            const int xf = (int)(bits >> 23) & 0xff;
            int e = xf == 0 ? -100 : xf - 127 - 8 + ((bits & 0x7fffffu) > 0x600000u ? 1 : 0);
            e = max(e, -100);
            const float unit = amax == 0.f ? 1.0f : __uint_as_float((uint32_t)(e + 127) << 23);
            const float inv = amax == 0.f ? 1.0f : __uint_as_float((uint32_t)(127 - e) << 23);
            uint32_t hi[4], lo[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) split2(qv[2 * i] * inv, qv[2 * i + 1] * inv, hi[i], lo[i]);
            *reinterpret_cast<uint2*>(sq + row_off(h, c * 8)) = make_uint2(hi[0] | (hi[1] << 16), hi[2] | (hi[3] << 16));
            *reinterpret_cast<uint2*>(sq + row_off(8 + h, c * 8)) = make_uint2(lo[0] | (lo[1] << 16), lo[2] | (lo[3] << 16));
            if (c == 0) q_unit[h] = unit * p.scale_log2;
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars[B_PFULL + 1]);        // q is in place (one extra phase of this barrier)
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");            // q_unit visible to every softmax thread
        float unit_h[8];
#pragma unroll
        for (int h = 0; h < 8; ++h) unit_h[h] = q_unit[h];

        float m_ref[8], l_sum[8];
#pragma unroll
        for (int h = 0; h < 8; ++h) { m_ref[h] = -INFINITY; l_sum[h] = 0.f; }
        float v_ref = 0.f;
        bool ok = true;
        // scales of this thread's key of the first tile
        const float* scl = pp.scales_l + (size_t)t * pp.scales_tstride;
        auto load_scales = [&](int j, float& ks_, float& vs_) {
            const int key = kstart + j * 128 + row;
            ks_ = 0.f; vs_ = 0.f;
            if (j < n_tiles && key < key_end) {
                int page = p.bt[(size_t)b * p.maxp + key / p.ps];
                if (page < 0 || page >= p.num_pages) page = 0;        // reported by the copy warp
                const int64_t vec = ((int64_t)page * 2 * p.nkv + kvh) * p.ps + key % p.ps;
                ks_ = scl[vec];
                vs_ = scl[vec + (int64_t)p.nkv * p.ps];
            }
        };
        // the scales of a key take two dependent global loads (block table, then the scale): fetched two tiles ahead
        float ks_a, vs_a, ks_b, vs_b;
        load_scales(0, ks_a, vs_a);
        load_scales(1, ks_b, vs_b);
        for (int j = 0; j < n_tiles; ++j) {
            const int bb = j & 1;
            const bool valid = kstart + j * 128 + row < key_end;
            const float ksc = ks_a, vsc = vs_a;
            ks_a = ks_b; vs_a = vs_b;
            load_scales(j + 2, ks_b, vs_b);
            float sc[16];
            if (ok) {
                ok = __all_sync(0xffffffffu, mbar_wait(&bars[B_SFULL + bb], (uint32_t)(j >> 1) & 1u, abort_flag));
                if (!ok && lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_FLASH_SFULL); *abort_flag = 1; }
            }
            float s[8], tmax[9];
            if (ok) {
                tc_fence_after();
                tm_ld16(lane_base + bb * 16, sc);
                tm_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars[B_SEMPTY + bb]);  // the scores of tile j + 2 may overwrite this buffer
#pragma unroll
                for (int h = 0; h < 8; ++h) {
                    s[h] = valid ? (sc[h] + sc[8 + h] * 0.0625f) * (ksc * unit_h[h]) : -INFINITY;
                    tmax[h] = ord2f(__reduce_max_sync(0xffffffffu, f2ord(s[h])));
                }
                tmax[8] = ord2f(__reduce_max_sync(0xffffffffu, f2ord(valid ? vsc : 0.f)));
                float mine = tmax[0];                              // lane h publishes the warp's maximum number h
#pragma unroll
                for (int h = 1; h < 9; ++h) mine = lane == h ? tmax[h] : mine;
                if (lane < 9) red[(bb * 4 + sw) * 12 + lane] = mine;
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");        // the four warps' maxima of this tile
            if (!ok) continue;
            float corr[8], vmax = 0.f;
            bool rescale = false;
#pragma unroll
            for (int h = 0; h < 8; ++h) {
                const float* r = red + bb * 48 + h;
                const float mx = fmaxf(fmaxf(r[0], r[12]), fmaxf(r[24], r[36]));
                corr[h] = 1.0f;
                if ((mx - m_ref[h]) > kLazyLog2) { corr[h] = ex2f(m_ref[h] - mx); m_ref[h] = mx; rescale = true; }
            }
            {
                const float* r = red + bb * 48 + 8;
                vmax = fmaxf(fmaxf(r[0], r[12]), fmaxf(r[24], r[36]));
            }
            float vcorr = 1.0f;
            if (vmax > v_ref) { vcorr = v_ref / vmax; v_ref = vmax; rescale = true; }   // powers of two: exact (v_ref starts at 0)
            if (rescale) {                                         // the same decision in all 128 threads
#pragma unroll
                for (int h = 0; h < 8; ++h) l_sum[h] *= corr[h];
                if (j > 0) {
                    // the previous P V product must have landed before the accumulator is rescaled
                    ok = __all_sync(0xffffffffu, mbar_wait(&bars[B_PEMPTY + (bb ^ 1)], (uint32_t)((j - 1) >> 1) & 1u, abort_flag));
                    if (!ok) { if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_FLASH_OREADY); *abort_flag = 1; } continue; }
                    tc_fence_after();
                    float ov[16];
                    tm_ld16(lane_base + 32, ov);
                    tm_wait_ld();
#pragma unroll
                    for (int h = 0; h < 8; ++h) { ov[h] *= corr[h] * vcorr; ov[8 + h] *= corr[h] * vcorr; }
                    tm_st16(lane_base + 32, ov);
                    tm_wait_st();
                    tc_fence_before();
                }
            }
            // P buffer bb was read by the P V product of tile j - 2
            if (j >= 2) {
                ok = __all_sync(0xffffffffu, mbar_wait(&bars[B_PEMPTY + bb], (uint32_t)((j - 2) >> 1) & 1u, abort_flag));
                if (!ok) { if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_FLASH_OREADY); *abort_flag = 1; } continue; }
            }
            const float p_unit = v_ref > 0.f ? vsc * (64.0f / v_ref) : 0.f;
            uint8_t* pb = sp + bb * kQBytes;
#pragma unroll
            for (int h = 0; h < 8; h += 2) {
                const float p0 = valid ? ex2f(s[h] - m_ref[h]) : 0.f, p1 = valid ? ex2f(s[h + 1] - m_ref[h + 1]) : 0.f;
                l_sum[h] += p0; l_sum[h + 1] += p1;
                uint32_t hi, lo;
                split2(p0 * p_unit, p1 * p_unit, hi, lo);
                pb[row_off(h, row)] = (uint8_t)(hi & 0xff);
                pb[row_off(h + 1, row)] = (uint8_t)(hi >> 8);
                pb[row_off(8 + h, row)] = (uint8_t)(lo & 0xff);
                pb[row_off(9 + h, row)] = (uint8_t)(lo >> 8);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars[B_PFULL + bb]);
        }
        // the last product
        if (ok && n_tiles > 0) {
            ok = __all_sync(0xffffffffu, mbar_wait(&bars[B_PEMPTY + ((n_tiles - 1) & 1)], (uint32_t)((n_tiles - 1) >> 1) & 1u, abort_flag));
            if (!ok && lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_FLASH_OREADY); *abort_flag = 1; }
        }
        // row sums: every thread holds the sums over its own keys; add them up over the 128 threads
#pragma unroll
        for (int h = 0; h < 8; ++h) {
#pragma unroll
            for (int o = 16; o; o >>= 1) l_sum[h] += __shfl_xor_sync(0xffffffffu, l_sum[h], o);
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");            // the last tile's readers of `red` are done
        {
            float mine = l_sum[0];
#pragma unroll
            for (int h = 1; h < 8; ++h) mine = lane == h ? l_sum[h] : mine;
            if (lane < 8) red[sw * 12 + lane] = mine;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (ok && n_tiles > 0) {
            tc_fence_after();
            float ov[16];
            tm_ld16(lane_base + 32, ov);
            tm_wait_ld();
            const float unit = v_ref * (1.0f / 64.0f);
            const int ns = p.nsplit[b];
#pragma unroll
            for (int h = 0; h < 8; ++h) {
                if (h < G) {
                    const float L = (red[h] + red[12 + h]) + (red[24 + h] + red[36 + h]);
                    const float acc = (ov[h] + ov[8 + h] * 0.0625f) * unit;
                    const int head = kvh * G + h;
                    if (ns == 1) {
                        p.o[((size_t)t * p.M + b) * (size_t)(p.nq * kDh) + (size_t)head * kDh + row] = __float2bfloat16_rn(L > 0.f ? acc / L : 0.f);
                    } else {
                        float* dst = p.part + ((((size_t)t * p.B + b) * p.nq + head) * p.max_splits + split) * (kDh + 2);
                        dst[row] = acc;
                        if (row == 0) { dst[kDh] = m_ref[h]; dst[kDh + 1] = L; }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(64) : "memory");
    }
}

// (code byte, vector of a slab, track) with boxes of 16 vectors x 128 bytes in the 128-byte swizzle
pt_status make_codes_map3(CUtensorMap* out, const void* base, int64_t vecs, int64_t tracks, int64_t track_stride_bytes) {
    EncodeFn enc = get_encode();
    if (!enc) { set_error("cuTensorMapEncodeTiled is not available from this driver"); return PT_ERR_CUDA; }
    cuuint64_t dims[3] = {(cuuint64_t)kDh, (cuuint64_t)vecs, (cuuint64_t)tracks};
    cuuint64_t strides[2] = {(cuuint64_t)kDh, (cuuint64_t)track_stride_bytes};
    cuuint32_t box[3] = {(cuuint32_t)kDh, 16, 1};
    cuuint32_t es[3] = {1, 1, 1};
    CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(base), dims, strides, box, es,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled (E4M3 cache) failed with code %d", (int)r); return PT_ERR_CUDA; }
    return PT_OK;
}

}  // namespace

pt_status launch_decode_attn_e4m3_tc(const AttnP& p, const Kv8Slab& slab, int T, int n_items, int max_splits, cudaStream_t st) {
    Dec8TcP pp{};
    pp.a = p;
    pp.scales_l = slab.scales_l; pp.scales_tstride = slab.scales_tstride;
    CUtensorMap kvmap;
    const int64_t slab_vecs = (int64_t)p.num_pages * 2 * p.nkv * p.ps;
    pt_status s = make_codes_map3(&kvmap, slab.codes_l, slab_vecs, T, slab.codes_tstride);
    if (s != PT_OK) return s;
    static bool done_[kMaxDevices] = {};
    bool& done = done_[current_device()];
    if (!done) {
        cudaError_t e = cudaFuncSetAttribute(k_decode_attn_e4m3_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
        if (e != cudaSuccess) { set_error("cudaFuncSetAttribute: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
        done = true;
    }
    cudaError_t e = launch_dependent(k_decode_attn_e4m3_tc, dim3(p.nkv, n_items, T), dim3(kThreads), (size_t)kSmem, st, kvmap, pp);
    if (e != cudaSuccess) { set_error("k_decode_attn_e4m3_tc launch: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (max_splits > 1) return launch_decode_combine(p, T, kDh, st);
    return PT_OK;
}

}  // namespace pt
