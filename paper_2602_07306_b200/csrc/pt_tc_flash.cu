// Causal prefill attention on the 5th-generation tensor cores (tcgen05 + tensor memory), reading
// K and V straight from the paged per-track KV cache.
//
// A CTA owns 256 consecutive query rows of one (track, sequence, head): two 128-row tiles that
// take turns on the tensor pipe.  For every 128-key tile of the sequence
//     S_i = Q_i K^T          (tcgen05.mma, operands in shared memory, S_i in tensor memory)
//     P_i = exp2(c S_i - c m)  written back over S_i as bf16 by the softmax warps
//     O_i += P_i V           (tcgen05.mma with P_i read from tensor memory, V as an MN-major tile)
// Roles: warp 0 streams Q once and K/V page by page with TMA (16-token boxes of the cache's
// [page][K|V][head][slot][dh] blocks, 128-byte swizzle) through two-stage rings; warp 1
// issues every MMA (one elected lane); warps 4-7 and 8-11 are the softmax groups of tile 0 and tile 1, one thread per
// query row (row max and row sum need no shuffles).  While one group works on its scores the
// tensor pipe runs the other tile's products.  The running maximum is only raised when it grows
// by more than 2^8 (the accumulator is then rescaled in tensor memory), so rescales are rare.
// Every mbarrier wait is bounded; on a timeout the CTA records PT_ERR_DEVICE_TIMEOUT, every role
// leaves its loop, and tensor memory is freed before exit.
#include "pt_tc.h"
#include "pt_ptx.cuh"

namespace pt {

namespace {

constexpr int kFlashThreads = 384;
#ifndef FLASH_KSTAGES
#define FLASH_KSTAGES 3
#endif
constexpr int kStagesK = FLASH_KSTAGES;    // K ring depth (head_dim 128: 2 Q tiles + 3 K + 2 V tiles of 32 KB fill the 227 KB of a CTA)
constexpr int kStagesV = 2;                // V ring depth
// Alternatives that were built and measured on the 8 x 4096-token causal shape of 8 tracks (one launch alone,
// 924 TFLOP/s with all of them off and a two-stage K ring), kept as compile-time switches:
//   FLASH_SPLIT_P   P handed to the MMA warp in two parts of 64 keys, so that the first half of P V runs under
//                   the second half of the exponentials: 854 (the extra tcgen05.wait::st and arrive cost more)
//   FLASH_PREFETCH  cp.async.bulk.prefetch.tensor of the K/V pages one ring depth ahead: 780 (the prefetches
//                   take turns with the copies on the SM's one TMA unit)
//   FLASH_POLY      exp2 of 4 / 8 of every 16 scores as a cubic on the FMA pipe instead of the MUFU: 905 / 829
//                   (one softmax warp per scheduler and tile is bound by its own issue rate, not by the MUFU)
//   FLASH_KSTAGES   three K stages instead of two: 938, kept
//   FLASH_SWAIT_NS  softmax warps sleeping between polls of their score barrier: no change
// Two softmax threads per query row (sixteen softmax warps, each thread 64 score columns, half-row maxima
// exchanged through shared memory at a two-warp named barrier) was also built: 814 with the scores kept in
// registers, 697 with a second read of the scores from tensor memory; its per-step overheads (barrier,
// exchange, twice the polls, 104 registers) outweigh the shorter chain.
#ifndef FLASH_SPLIT_P
#define FLASH_SPLIT_P 0
#endif
#ifndef FLASH_PREFETCH
#define FLASH_PREFETCH 0
#endif
#ifndef FLASH_POLY
#define FLASH_POLY 0                       // of every 16 scores, this many (a multiple of 4) take the polynomial exp2
#endif
#ifndef FLASH_SWAIT_NS
#define FLASH_SWAIT_NS 0                   // > 0: the softmax warps sleep this long between polls of their score barrier
#endif
constexpr int kPParts = FLASH_SPLIT_P ? 2 : 1;
constexpr uint32_t kSpin = 1u << 26;
constexpr int kHalfBytes = 128 * 128;      // 128 rows x 64 bf16: one swizzled column block of a tile

enum { B_QFULL = 0, B_KFULL = 2, B_KEMPTY = 5, B_VFULL = 8, B_VEMPTY = 10, B_SFULL = 12, B_PFULL = 14 /* [tile][part] */,
       B_OREADY = 18, B_VRAW = 20, B_COUNT = 21 };
static_assert(kStagesK <= 3 && kStagesV <= 2, "barrier slots");

// `relaxed` waits (the copy warp's, which run stages ahead of their consumers) back off between polls:
// a spinning warp costs issue slots and power; the softmax and MMA hand-offs poll at full rate.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, bool relaxed = false, unsigned sleep_ns = 128) {
    WaitClock clock;
    for (uint32_t i = 0; i < kSpin; ++i) {
        if (mbar_try(bar, parity)) return true;
        if (relaxed && i >= 2) __nanosleep(sleep_ns);
        if ((i & 255) == 255 && (*abort_flag || clock.expired())) return false;
    }
    return false;
}
__device__ __forceinline__ void tma_prefetch_3d(const CUtensorMap* map, int c0, int c1, int c2) {
    asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];"
                 ::"l"((uint64_t)map), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
// The MMA warp runs its issue loop with all 32 lanes (so addresses and descriptors stay
// warp-uniform values) and one elected lane executes each tcgen05 instruction.
// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n .reg .pred p, e;\n elect.sync _|e, 0xffffffff;\n setp.ne.b32 p, %4, 0;\n @e tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                 ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(acc) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d, uint32_t a_tmem, uint64_t b, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n .reg .pred p, e;\n elect.sync _|e, 0xffffffff;\n setp.ne.b32 p, %4, 0;\n @e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}"
                 ::"r"(d), "r"(a_tmem), "l"(b), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void tm_ld32(uint32_t taddr, float* v) {
    uint32_t r[32];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tm_st32(uint32_t taddr, const float* v) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
                 "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
                 "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
                 ::"r"(taddr),
                   "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
                   "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
                   "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
                   "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])),
                   "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
                   "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
                   "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])),
                   "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
                 : "memory");
}
__device__ __forceinline__ void tm_st16(uint32_t taddr, const uint32_t* r) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
                 "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                   "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
                 : "memory");
}
__device__ __forceinline__ void tm_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tm_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// Packed fp32 pairs (one instruction for two lanes of arithmetic) and the three-input maximum.
__device__ __forceinline__ void fma2(float& d0, float& d1, float a0, float a1, float s, float b) {   // a * s + b
    asm("{\n .reg .b64 ra, rs, rb, rd;\n mov.b64 ra, {%2, %3};\n mov.b64 rs, {%4, %4};\n mov.b64 rb, {%5, %5};\n"
        " fma.rn.f32x2 rd, ra, rs, rb;\n mov.b64 {%0, %1}, rd;\n}"
        : "=f"(d0), "=f"(d1) : "f"(a0), "f"(a1), "f"(s), "f"(b));
}
__device__ __forceinline__ void add2(float& d0, float& d1, float a0, float a1) {                    // d += a
    asm("{\n .reg .b64 ra, rd;\n mov.b64 ra, {%2, %3};\n mov.b64 rd, {%0, %1};\n add.rn.f32x2 rd, rd, ra;\n mov.b64 {%0, %1}, rd;\n}"
        : "+f"(d0), "+f"(d1) : "f"(a0), "f"(a1));
}
// 2^x for a pair of arguments on the FMA pipe instead of the MUFU: x = n + f with n = round(x) (adding 1.5 * 2^23
// leaves n in the low mantissa bits), 2^f by a cubic on [-0.5, 0.5] (relative error 7.5e-5, a twenty-fifth of the
// bf16 rounding the result receives), 2^n by adding n to the exponent field.  Arguments below -125 give 2^-125
// (1e-38: a masked score's probability is not exactly zero on this path, but it is far below anything fp32 sums keep).
__device__ __forceinline__ void ex2_poly2(float& x0, float& x1) {
    const float magic = 12582912.0f;
    x0 = fmaxf(x0, -125.0f); x1 = fmaxf(x1, -125.0f);
    float r0, r1, p0, p1;
    asm("{\n .reg .b64 x, m, r, n, f, p, c;\n"
        " mov.b64 x, {%4, %5};\n mov.b64 m, {%6, %6};\n"
        " add.rn.f32x2 r, x, m;\n"                      // r = x + magic: the integer part lands in the mantissa
        " sub.rn.f32x2 n, r, m;\n"                      // n = round(x)
        " sub.rn.f32x2 f, x, n;\n"                      // f in [-0.5, 0.5]
        " mov.b64 p, {%7, %7};\n mov.b64 c, {%8, %8};\n"
        " fma.rn.f32x2 p, p, f, c;\n"
        " mov.b64 c, {%9, %9};\n"
        " fma.rn.f32x2 p, p, f, c;\n"
        " mov.b64 c, {%10, %10};\n"
        " fma.rn.f32x2 p, p, f, c;\n"
        " mov.b64 {%0, %1}, r;\n mov.b64 {%2, %3}, p;\n}"
        : "=f"(r0), "=f"(r1), "=f"(p0), "=f"(p1)
        : "f"(x0), "f"(x1), "f"(magic), "f"(0.05517137795686722f), "f"(0.24261121451854706f), "f"(0.6932610273361206f), "f"(0.9999280571937561f));
    x0 = __uint_as_float(__float_as_uint(p0) + (__float_as_uint(r0) << 23));
    x1 = __uint_as_float(__float_as_uint(p1) + (__float_as_uint(r1) << 23));
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Shared-memory descriptor of a K-major bf16 operand: rows of 128 bytes (64 elements) in the
// 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFF) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Descriptor of an MN-major bf16 operand (V: the contraction index, keys, walks rows; head_dim is
// contiguous): 64-element column blocks kHalfBytes apart, 8-key groups 1024 bytes apart.
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFF) >> 4);
    d |= (uint64_t)(kHalfBytes >> 4) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

template <int DH> struct FlashCfg {
    static constexpr int HALVES = DH / 64;
    static constexpr int TILE_BYTES = HALVES * kHalfBytes;          // one Q, K or V tile of 128 rows
    static constexpr int SMEM = (2 + kStagesK + kStagesV) * TILE_BYTES + 1024 + 256;
    static_assert(SMEM <= 232448, "shared memory of one CTA");
};

template <int DH>
__global__ void __launch_bounds__(kFlashThreads, 1)
k_flash_prefill_tc(const __grid_constant__ CUtensorMap qmap, const __grid_constant__ CUtensorMap kvmap, const AttnP p,
                   const int q_box_rows) {
    using C = FlashCfg<DH>;
    constexpr int HALVES = C::HALVES, TILE = C::TILE_BYTES;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* sq = smem;
    uint8_t* sk = sq + 2 * TILE;
    uint8_t* sv = sk + kStagesK * TILE;
    uint64_t* bars = (uint64_t*)(sv + kStagesV * TILE);
    uint32_t* tmem_slot = (uint32_t*)(bars + B_COUNT);
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // consecutive CTAs are the query blocks of one (track, sequence, head), longest first: they read
    // the same K/V pages at about the same time, so all but the first find them in L2
    const int qb = gridDim.x - 1 - blockIdx.x;
    const int head = blockIdx.y, kvh = head / (p.nq / p.nkv);
    const int t = blockIdx.z / p.B, b = blockIdx.z % p.B;
    const int key_end = p.kvlen[b];
    const int start = key_end - p.S;                               // position of the sequence's first new token
    int n_t[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int q0 = qb * 256 + i * 128;
        n_t[i] = q0 < p.S ? (min(key_end, start + q0 + 128) + 127) >> 7 : 0;
    }
    const int n_max = max(n_t[0], n_t[1]);

    if (threadIdx.x == 0) {
        for (int i = 0; i < B_COUNT; ++i) mbar_init(&bars[i], (i >= B_PFULL && i < B_PFULL + 4) ? 4 : 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // the copy and MMA warps need few registers; hand theirs to the softmax groups, whose threads
    // keep a whole 128-column score row each
    if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const uint32_t qbytes = (uint32_t)q_box_rows * 128u * HALVES;
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                if (n_t[i] == 0) continue;
                mbar_expect_tx(&bars[B_QFULL + i], qbytes);
#pragma unroll
                for (int h = 0; h < HALVES; ++h)
                    tma_load_3d(smem_u32(sq + i * TILE + h * kHalfBytes), &qmap, &bars[B_QFULL + i],
                                head * DH + h * 64, b * p.S + qb * 256 + i * 128, t);
            }
        }
        __syncwarp();
        bool bad_page = false;
        for (int j = 0; j < n_max; ++j) {
            const int sK = j % kStagesK, s = j % kStagesV;
            const uint32_t phK = (uint32_t)(j / kStagesK) & 1u, ph = (uint32_t)(j / kStagesV) & 1u;
            const int key0 = j * 128;
            const int ng = min(8, (key_end - key0 + 15) >> 4);    // 16-key groups of this tile that hold keys
            int row_k = 0;
            if (lane < ng) {
                const int key = key0 + lane * 16;
                int page = p.bt[(size_t)b * p.maxp + key / p.ps];
                if (page < 0 || page >= p.num_pages) { bad_page = true; page = 0; }
                row_k = (page * 2 * p.nkv + kvh) * p.ps + key % p.ps;
            }
            const uint32_t bytes = (uint32_t)ng * 16u * DH * 2u;
            if (!mbar_wait(&bars[B_KEMPTY + sK], phK ^ 1u, abort_flag, true)) { if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_FLASH_KEMPTY); *abort_flag = 1; } break; }
            if (lane == 0) mbar_expect_tx(&bars[B_KFULL + sK], bytes);
            __syncwarp();
            if (lane < ng) {
#pragma unroll
                for (int h = 0; h < HALVES; ++h)
                    tma_load_3d(smem_u32(sk + sK * TILE + h * kHalfBytes + lane * 2048), &kvmap, &bars[B_KFULL + sK], h * 64, row_k, t);
            }
            if (!mbar_wait(&bars[B_VEMPTY + s], ph ^ 1u, abort_flag, true)) { if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_FLASH_VEMPTY); *abort_flag = 1; } break; }
            const bool partial = key0 + 128 > key_end;             // rows past the last key must read as zero
            uint64_t* vbar = partial ? &bars[B_VRAW] : &bars[B_VFULL + s];
            if (lane == 0) mbar_expect_tx(vbar, bytes);
            __syncwarp();
            if (lane < ng) {
#pragma unroll
                for (int h = 0; h < HALVES; ++h)
                    tma_load_3d(smem_u32(sv + s * TILE + h * kHalfBytes + lane * 2048), &kvmap, vbar, h * 64, row_k + p.nkv * p.ps, t);
            }
            if (FLASH_PREFETCH && j + kStagesK < n_max) {          // the tile one ring depth ahead: bring its pages into L2 now
                const int keyp = (j + kStagesK) * 128 + lane * 16;
                if (lane < 8 && keyp < key_end) {
                    const int page = p.bt[(size_t)b * p.maxp + keyp / p.ps];
                    if (page >= 0 && page < p.num_pages) {
                        const int row_p = (page * 2 * p.nkv + kvh) * p.ps + keyp % p.ps;
#pragma unroll
                        for (int h = 0; h < HALVES; ++h) {
                            tma_prefetch_3d(&kvmap, h * 64, row_p, t);
                            tma_prefetch_3d(&kvmap, h * 64, row_p + p.nkv * p.ps, t);
                        }
                    }
                }
            }
            if (partial) {                                         // at most once per CTA: its last tile
                if (!mbar_wait(&bars[B_VRAW], 0u, abort_flag)) { if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_FLASH_VRAW); *abort_flag = 1; } break; }
                const int nvalid = key_end - key0;
                for (int idx = lane; idx < (128 - nvalid) * HALVES * 8; idx += 32) {
                    const int row = nvalid + idx / (HALVES * 8), rem = idx % (HALVES * 8);
                    *reinterpret_cast<uint4*>(sv + s * TILE + (rem >> 3) * kHalfBytes + row * 128 + (rem & 7) * 16) = make_uint4(0, 0, 0, 0);
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars[B_VFULL + s]);
            }
        }
        if (bad_page) report(p.status, PT_ERR_DEVICE_BOUNDS, LOC_FLASH_PAGE);
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (whole warp, see tc_commit)
        {
            constexpr uint32_t idesc_qk = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
            constexpr uint32_t idesc_pv = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(DH >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
            bool ok = true;
            auto wait = [&](int bar, uint32_t parity, int loc) {
                if (!ok) return;
                if (!__all_sync(0xffffffffu, mbar_wait(&bars[bar], parity, abort_flag))) { ok = false; if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, loc); *abort_flag = 1; } }
                tc_fence_after();
            };
            auto qk = [&](int i, int s) {                          // S_i = Q_i K_s^T
                if (!ok) return;
                const uint32_t qa = smem_u32(sq + i * TILE), ka = smem_u32(sk + s * TILE);
#pragma unroll
                for (int ks = 0; ks < DH / 16; ++ks) {
                    const uint32_t off = (uint32_t)(ks >> 2) * kHalfBytes + (uint32_t)(ks & 3) * 32u;
                    mma_ss(tmem_base + i * 128, desc_kmajor(qa + off), desc_kmajor(ka + off), idesc_qk, ks != 0);
                }
                tc_commit(&bars[B_SFULL + i]);
            };
            auto pv = [&](int i, int s, int j) {                   // O_i (+)= P_i V_s, in the parts P arrives in
                const uint32_t va = smem_u32(sv + s * TILE);
                wait(B_PFULL + 2 * i, (uint32_t)j & 1u, LOC_FLASH_PFULL);
                wait(B_VFULL + s, (uint32_t)(j / kStagesV) & 1u, LOC_FLASH_VFULL);
#pragma unroll
                for (int part = 0; part < kPParts; ++part) {
                    if (part) wait(B_PFULL + 2 * i + 1, (uint32_t)j & 1u, LOC_FLASH_PFULL);
                    if (!ok) return;
#pragma unroll
                    for (int u = 0; u < 8 / kPParts; ++u) {
                        const int ks = part * (8 / kPParts) + u;
                        mma_ts(tmem_base + 256 + i * DH, tmem_base + i * 128 + ks * 8, desc_mnmajor(va + ks * 2048), idesc_pv, j > 0 || ks != 0);
                    }
                }
                tc_commit(&bars[B_OREADY + i]);
            };
            wait(B_KFULL + 0, 0, LOC_FLASH_KFULL);
#pragma unroll
            for (int i = 0; i < 2; ++i)
                if (n_t[i] > 0) { wait(B_QFULL + i, 0, LOC_FLASH_QFULL); qk(i, 0); }
            if (ok) tc_commit(&bars[B_KEMPTY + 0]);
            for (int j = 0; j < n_max && ok; ++j) {
                const int s = j % kStagesV, sn = (j + 1) % kStagesK;
                const uint32_t phn = (uint32_t)((j + 1) / kStagesK) & 1u;
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    if (j < n_t[i]) {
                        pv(i, s, j);
                        if (j + 1 < n_t[i]) { wait(B_KFULL + sn, phn, LOC_FLASH_KFULL); qk(i, sn); }
                    }
                }
                if (ok) {
                    tc_commit(&bars[B_VEMPTY + s]);
                    if (j + 1 < n_max) tc_commit(&bars[B_KEMPTY + sn]);
                }
            }
        }
        __syncwarp();
    }
    } else {
        // ------------------------------------------------------------------ softmax groups
        asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
        const int i = (warp - 4) >> 2;                             // query tile of this warp group
        const int w4 = warp & 3;                                   // tensor-memory lane quarter of this warp
        const int n_i = n_t[i];
        const int q0 = qb * 256 + i * 128;
        const int s_row = q0 + w4 * 32 + lane;                     // row inside the sequence
        const int limit = min(start + s_row, key_end - 1);         // last visible key of this row
        const int tile_limit = min(start + q0, key_end - 1);       // last visible key of the tile's first row
        const uint32_t t_s = tmem_base + ((uint32_t)(w4 * 32) << 16) + i * 128;
        const uint32_t t_o = tmem_base + ((uint32_t)(w4 * 32) << 16) + 256 + i * DH;
        const float c = p.scale_log2;
        float m_ref = -INFINITY, l_run = 0.f;
        bool ok = true;
        for (int j = 0; j < n_i; ++j) {
            ok = mbar_wait(&bars[B_SFULL + i], (uint32_t)j & 1u, abort_flag, FLASH_SWAIT_NS > 0, FLASH_SWAIT_NS);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) { if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_FLASH_SFULL); *abort_flag = 1; } break; }
            tc_fence_after();
            const int key0 = j * 128;
            const bool need_mask = key0 + 127 > tile_limit;
            // the whole score row of this thread lives in registers: one round trip to tensor memory
            float v[128];
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) tm_ld32(t_s + cc * 32, v + cc * 32);
            tm_wait_ld();
            if (need_mask) {
#pragma unroll
                for (int e = 0; e < 128; ++e) if (key0 + e > limit) v[e] = -INFINITY;
            }
            float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
            for (int e = 0; e < 128; e += 8) {
                mx0 = max3(mx0, v[e], v[e + 1]); mx1 = max3(mx1, v[e + 2], v[e + 3]);
                mx2 = max3(mx2, v[e + 4], v[e + 5]); mx3 = max3(mx3, v[e + 6], v[e + 7]);
            }
            const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
            if (j == 0) {
                m_ref = mx;                                        // key 0 is visible to every row: finite
            } else {
                const bool grow = (mx - m_ref) * c > 8.0f;
                if (__any_sync(0xffffffffu, grow)) {
                    // the previous P V product must have landed before the accumulator is rescaled
                    ok = mbar_wait(&bars[B_OREADY + i], (uint32_t)(j - 1) & 1u, abort_flag);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) { if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_FLASH_OREADY); *abort_flag = 1; } break; }
                    tc_fence_after();
                    const float corr = grow ? ex2((m_ref - mx) * c) : 1.0f;
                    if (grow) { m_ref = mx; l_run *= corr; }
#pragma unroll 1
                    for (int cc = 0; cc < DH / 32; ++cc) {
                        float v[32];
                        tm_ld32(t_o + cc * 32, v);
                        tm_wait_ld();
#pragma unroll
                        for (int e = 0; e < 32; ++e) v[e] *= corr;
                        tm_st32(t_o + cc * 32, v);
                    }
                }
            }
            const float mc = m_ref * c;
            // P = exp2(c s - c m) as bf16 over the first half of the score columns (masked scores are
            // -inf and give exactly 0)
            float l0 = 0.f, l1 = 0.f, l2 = 0.f, l3 = 0.f;
            const float nmc = -mc;
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                uint32_t pk[16];
#pragma unroll
                for (int e = 0; e < 32; e += 4) {
                    float x0, x1, x2, x3;
                    fma2(x0, x1, v[cc * 32 + e], v[cc * 32 + e + 1], c, nmc);
                    fma2(x2, x3, v[cc * 32 + e + 2], v[cc * 32 + e + 3], c, nmc);
                    if ((e & 15) < FLASH_POLY) { ex2_poly2(x0, x1); ex2_poly2(x2, x3); }
                    else { x0 = ex2(x0); x1 = ex2(x1); x2 = ex2(x2); x3 = ex2(x3); }
                    add2(l0, l1, x0, x1);
                    add2(l2, l3, x2, x3);
                    pk[e >> 1] = pack_bf16(x0, x1);
                    pk[(e >> 1) + 1] = pack_bf16(x2, x3);
                }
                tm_st16(t_s + cc * 16, pk);
                if (FLASH_SPLIT_P && cc == 1) {                    // keys 0-63 are in place: the first half of P V may start
                    tm_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars[B_PFULL + 2 * i]);
                }
            }
            l_run += (l0 + l1) + (l2 + l3);
            tm_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars[B_PFULL + 2 * i + kPParts - 1]);
        }
        if (ok && n_i > 0) {
            ok = mbar_wait(&bars[B_OREADY + i], (uint32_t)(n_i - 1) & 1u, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) { if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_FLASH_OREADY); *abort_flag = 1; } }
        }
        if (ok && n_i > 0) {
            tc_fence_after();
            const float inv = l_run > 0.f ? 1.0f / l_run : 0.f;
            __nv_bfloat16* dst = p.o + ((size_t)t * p.M + (size_t)b * p.S + s_row) * (size_t)(p.nq * DH) + (size_t)head * DH;
#pragma unroll 1
            for (int cc = 0; cc < DH / 32; ++cc) {
                float v[32];
                tm_ld32(t_o + cc * 32, v);
                tm_wait_ld();
                if (s_row < p.S) {
#pragma unroll
                    for (int e = 0; e < 32; e += 8) {
                        uint4 u;
                        u.x = pack_bf16(v[e] * inv, v[e + 1] * inv); u.y = pack_bf16(v[e + 2] * inv, v[e + 3] * inv);
                        u.z = pack_bf16(v[e + 4] * inv, v[e + 5] * inv); u.w = pack_bf16(v[e + 6] * inv, v[e + 7] * inv);
                        *reinterpret_cast<uint4*>(dst + cc * 32 + e) = u;
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 2) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
    }
}

}  // namespace

bool flash_tc_supported(int dh, int ps) { return (dh == 64 || dh == 128) && ps % 16 == 0; }

pt_status launch_flash_prefill_tc(const AttnP& p, int T, int dh, cudaStream_t st) {
    if (!flash_tc_supported(dh, p.ps)) { set_error("tensor-memory prefill attention needs head_dim 64 or 128 and pages of a multiple of 16 tokens"); return PT_ERR_UNSUPPORTED; }
    if ((int64_t)T * p.B > 65535 || p.nq > 65535) { set_error("prefill attention grid too large"); return PT_ERR_INVALID_ARG; }
    CUtensorMap qmap, kvmap;
    pt_status s;
    if ((s = make_map_bf16(&qmap, p.q, (int64_t)p.nq * dh, p.M, T, 128)) != PT_OK) return s;
    if ((s = make_map_bf16_strided(&kvmap, p.pool_l, dh, (int64_t)p.num_pages * 2 * p.nkv * p.ps, T, p.pool_tstride * 2, 16)) != PT_OK) return s;
    const int q_box_rows = std::min(128, p.M);
    dim3 grid((p.S + 255) / 256, p.nq, T * p.B);
#define GO(DH_) { static bool done_[kMaxDevices] = {}; bool& done = done_[current_device()]; \
        if (!done) { cudaError_t e = cudaFuncSetAttribute(k_flash_prefill_tc<DH_>, cudaFuncAttributeMaxDynamicSharedMemorySize, FlashCfg<DH_>::SMEM); \
                     if (e != cudaSuccess) { set_error("cudaFuncSetAttribute: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; } done = true; } \
        k_flash_prefill_tc<DH_><<<grid, kFlashThreads, FlashCfg<DH_>::SMEM, st>>>(qmap, kvmap, p, q_box_rows); }
    if (dh == 64) GO(64) else GO(128)
#undef GO
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return PT_OK;
}

}  // namespace pt
