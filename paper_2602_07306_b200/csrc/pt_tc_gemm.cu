// Track-grouped bf16 GEMM for sm_100a: C[t] = A[t] * W[t]^T with fp32 accumulation in tensor
// memory.  Persistent, warp-specialised: warp 0 feeds a ring of shared-memory stages with TMA
// (3-D tensor maps, coordinates (k, row, track), 128-byte swizzle), warp 1 issues tcgen05.mma
// (128 x BN x 16 per instruction, one elected lane) into one of two TMEM accumulators, warps 2-9
// drain the other accumulator with tcgen05.ld and run the fused epilogue:
//   EPI_QKV     per-row 1/rms scale (RMSNorm), rotary embedding on q and k heads, q to a dense
//               buffer, k and v straight into the paged KV cache
//   EPI_SWIGLU  per-row 1/rms scale, silu(gate) * up on interleaved gate/up columns
//   EPI_RESID   residual add (optionally summed over all tracks = the track-sync of Algorithm 1,
//               with the K loop running over (track, k) so one accumulator collects every track),
//               fp32 stream out, gain-scaled bf16 copy for the next GEMM, partial sums of squares
//               for the next RMSNorm
//   EPI_PLAIN   fp32 C (kernel-level tests)
// Epilogue data path: a warp owns 32 accumulator rows (its tensor-memory lane quarter); the two
// warps of a quarter split the tile's columns.  tcgen05.ld hands every thread one row, and the
// thread reads and writes whole 32-byte sectors of that row (the residual epilogue, which moves
// the most bytes, first turns each 32 x 32 unit through shared memory so that its global accesses
// are 128 contiguous bytes per row).  Global loads that do not depend on the accumulator (row
// statistics, rotary table, residual rows) are issued before the wait for the accumulator and one
// 32-column unit ahead, so their latency hides behind the tensor pipe.
// Three shapes of the same pipeline, chosen by the launch's row count (gemm_bn, gemm_kps,
// gemm_pair_ok): gemm_tc with one k-block per ring stage; gemm_tc with stages of 2 or 4 k-blocks
// and one 4-D copy of W and of A per stage (few rows: a decode step streams W from HBM);
// gemm_tc_pair, two CTAs of a cluster on a 256 x 256 tile with tcgen05.mma.cta_group::2 (many
// rows: halves the W bytes copied into each SM).  All are programmatic dependent launches.
// Every mbarrier wait is bounded; on a timeout the CTA records PT_ERR_DEVICE_TIMEOUT, stops
// issuing work, frees its tensor memory and exits.
#include "pt_tc.h"
#include "pt_ptx.cuh"

namespace pt {

namespace {

constexpr int BM = 128, BK = 64;
constexpr int kEpiWarps = 8;
constexpr int kGemmThreads = 64 + 32 * kEpiWarps;
constexpr uint32_t kSpinLimit = 1u << 26;

// Bounded wait: false when the limit ran out or another warp already gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, unsigned long long limit_ns = kWaitLimitNs) {
    WaitClock clock;
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (mbar_try(bar, parity)) return true;
        if (i >= 4) __nanosleep(64);                       // back off: a spinning warp costs issue slots and power
        if ((i & 255) == 255 && (*abort_flag || clock.expired(limit_ns))) return false;
    }
    return false;
}


__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
                 ::"r"(smem_u32(dst)), "l"((uint64_t)map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(smem_u32(bar)) : "memory");
}


// The MMA warp runs its loop with all 32 lanes, so addresses and descriptors stay warp-uniform
// values, and one elected lane executes each tcgen05 instruction.
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n .reg .pred p, e;\n elect.sync _|e, 0xffffffff;\n setp.ne.b32 p, %4, 0;\n"
                 " @e tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, float* v) {
    uint32_t r[16];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr) : "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major bf16 tile whose rows are 128 bytes (64 elements)
// in the 128-byte swizzle: 8-row groups are 1024 bytes apart; the leading-dimension field is
// unused for this layout.
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFF) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}


// Shared memory of a CTA: a ring of stages, each one k-block of A (the launch's row box: min(M, 128)
// rows, rounded up to the 1024-byte swizzle atom) followed by one of W (BN rows).  The fewer rows a
// launch has, the more stages fit, so a decode step (few rows, weights streamed once) keeps more
// bytes of W in flight per SM.  tcgen05.mma always reads 128 rows of A from a stage: rows past the box
// belong to the stages behind it (or to the slack after the last stage) and only feed accumulator rows
// that nobody stores.  With few rows a stage holds kps k-blocks (A pieces first, then W) and W arrives
// as one copy of kps k-blocks (a 4-D view of W: 64 columns, rows, k-blocks, tracks): a copy occupies the
// SM's TMA unit for about a memory latency whatever its size, so W streams from HBM at full rate only
// with 16 KB or more per copy.
constexpr int kMaxStages = 24;
constexpr int kRingBytes = 192 * 1024;                       // stages + the slack behind the last one
constexpr int kXposeBytes = kEpiWarps * 4096;                // per epilogue warp: 32 rows x 128 bytes to turn row-per-thread data
constexpr int kBarBytes = 512;                               // 2 * kMaxStages + 4 mbarriers, TMEM slot, abort flag
constexpr int kGemmSmem = kRingBytes + kXposeBytes + 1024 /*alignment*/ + kBarBytes;
constexpr int kFullA = BM * BK * 2;

template <int BN> struct Cfg {
    static constexpr int B_BYTES = BN * BK * 2;
};
inline int stage_a_bytes(int M) { return (std::min(M, BM) * BK * 2 + 1023) / 1024 * 1024; }
inline int ring_stages(int a_bytes, int b_bytes, int kps) {
    return std::min(kMaxStages, (kRingBytes - (kFullA - a_bytes)) / (kps * (a_bytes + b_bytes)));
}

// ---- epilogue ------------------------------------------------------------------------------
// tcgen05.ld hands every thread one accumulator row (row0 + lane); a warp works through its share
// of the tile's columns in units of 32.  Each thread reads and writes 64- or 128-byte pieces of
// its own row (whole 32-byte sectors).  Global loads that do not depend on the accumulator (row
// statistics, rotary table, residual rows) are issued before the wait for the accumulator and one
// unit ahead of their use, so their latency hides behind the tensor pipe and the previous unit.

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&v);
}
// 256-bit global accesses (32-byte aligned): every lane moves one whole sector per instruction,
// which halves the load/store-unit work of these row-per-thread access patterns.
__device__ __forceinline__ void ld256(const float* p, float* v) {
    asm volatile("ld.global.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7]) : "l"(p));
}
__device__ __forceinline__ void st256(float* p, const float* v) {
    asm volatile("st.global.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"l"(p), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]) : "memory");
}
// 16 floats -> 16 bf16: one 32-byte store
__device__ __forceinline__ void store16_bf16(__nv_bfloat16* dst, const float* v) {
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"l"(dst), "r"(pack_bf16(v[0], v[1])), "r"(pack_bf16(v[2], v[3])), "r"(pack_bf16(v[4], v[5])), "r"(pack_bf16(v[6], v[7])),
                   "r"(pack_bf16(v[8], v[9])), "r"(pack_bf16(v[10], v[11])), "r"(pack_bf16(v[12], v[13])), "r"(pack_bf16(v[14], v[15]))
                 : "memory");
}

// 1 / rms of this thread's row from the producer's partial sums of squares.
__device__ __forceinline__ float row_rinv(const GemmP& p, int t, int row, bool row_ok) {
    if (!row_ok) return 1.f;
    const float* sp = p.ssq_in + (size_t)t * p.ssq_in_tstride + (size_t)row * p.ssq_tiles;
    float s = 0.f;
    if ((p.ssq_tiles & 7) == 0) {
        for (int i = 0; i < p.ssq_tiles; i += 8) {
            float v[8];
            ld256(sp + i, v);
            s += ((v[0] + v[1]) + (v[2] + v[3])) + ((v[4] + v[5]) + (v[6] + v[7]));
        }
    } else {
        for (int i = 0; i < p.ssq_tiles; ++i) s += sp[i];
    }
    return 1.0f / sqrtf(s / (float)p.K + p.eps);
}

template <int BN, class Wait>
__device__ __forceinline__ bool epi_plain(const GemmP& p, uint32_t taddr, int t, int row, bool row_ok, int n0, int half, Wait wait) {
    constexpr int UNITS = BN / 32;                        // 32-column units of the tile; 64-column groups alternate between the two warps
    if (!wait()) return false;
#pragma unroll 1
    for (int u = 2 * half; u < UNITS; u += (u & 1) ? 3 : 1) {
        const int c = u * 32;
        if (n0 + c >= p.N) break;                          // uniform across the warp
        float v[32];
        tc_ld16(taddr + c, v);
        tc_ld16(taddr + c + 16, v + 16);
        tc_wait_ld();
        if (row_ok) {
            float4* dst = (float4*)(p.c_out + ((size_t)t * p.M + row) * p.N + n0 + c);
#pragma unroll
            for (int i = 0; i < 8; ++i)
                if (n0 + c + 4 * i < p.N) dst[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
        }
    }
    return true;
}

// Accumulator columns come in groups of 32: 16 gate columns followed by their 16 up columns.  A
// unit here is 64 accumulator columns = 32 outputs z = silu(gate / rms) * (up / rms).
template <int BN, class Wait>
__device__ __forceinline__ bool epi_swiglu(const GemmP& p, uint32_t taddr, int t, int row, bool row_ok, int n0, int half, Wait wait) {
    constexpr int UNITS = BN / 64;                        // 64-column units of the tile, alternating between the two warps
    const float rinv = row_rinv(p, t, row, row_ok);
    const int F = p.N >> 1;
    if (!wait()) return false;
#pragma unroll 1
    for (int u = half; u < UNITS; u += 2) {
        const int c = u * 64;
        if (n0 + c >= p.N) break;
        float gu[64];
#pragma unroll
        for (int g4 = 0; g4 < 4; ++g4) tc_ld16(taddr + c + g4 * 16, gu + g4 * 16);
        tc_wait_ld();
        // PT-MoE: the 64 columns of a unit belong to one expert (its block is a multiple of 32 columns wide and starts on one)
        float wgt = 1.0f;
        if (p.gates && row_ok) wgt = p.gates[((size_t)t * p.M + row) * p.n_experts + (n0 + c) / p.expert_cols];
#pragma unroll
        for (int g2 = 0; g2 < 2; ++g2) {
            float z[16];
            if (p.gates && g2 == 1 && row_ok && ((n0 + c + 32) / p.expert_cols) != ((n0 + c) / p.expert_cols) && n0 + c + 32 < p.N)
                wgt = p.gates[((size_t)t * p.M + row) * p.n_experts + (n0 + c + 32) / p.expert_cols];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const float gv = gu[g2 * 32 + i] * rinv, uv = gu[g2 * 32 + 16 + i] * rinv;
                z[i] = __fdividef(gv, 1.0f + __expf(-gv)) * uv * wgt;
            }
            const int zc = ((n0 + c) >> 1) + g2 * 16;      // first output column of this group
            if (row_ok && zc < F) store16_bf16(p.z_out + ((size_t)t * p.M + row) * F + zc, z);
        }
    }
    return true;
}

// A unit is 32 accumulator columns of one head: for q and k heads the 16 columns j0..j0+15 and
// their rotary partners j0+dh/2.., for v heads 32 consecutive columns.  The (cos, sin) pairs of the
// row's position (fp16, 64 bytes per slice) are fetched before the wait for the accumulator.
template <int BN, class Wait>
__device__ __forceinline__ bool epi_qkv(const GemmP& p, uint32_t taddr, int t, int row, bool row_ok, int n0, int half, Wait wait) {
    constexpr int UNITS = BN / 32;                        // units of the tile, alternating between the two warps
    const int dh = p.dh, halfdh = dh >> 1, upd = dh >> 5;  // units per head
    const int heads_total = p.nq + 2 * p.nkv;
    int pos = 0; int64_t kvoff = 0;
    if (row_ok) { pos = p.row_pos[row]; kvoff = p.row_kvoff[row]; }
    const float rinv = row_rinv(p, t, row, row_ok);
    const bool slot_ok = row_ok && kvoff >= 0 && kvoff + (int64_t)(2 * p.nkv - 1) * p.ps * dh + dh <= p.slab_elems;
    if (row_ok && !slot_ok) report(p.status, PT_ERR_DEVICE_BOUNDS, LOC_ROPE_PAGE);
    const float* csr = reinterpret_cast<const float*>(p.cs16 + (size_t)pos * halfdh);   // (cos, sin) fp16 pairs, moved as 32-bit words
    // tab[i] = packed (cos, sin) of column j0 + i for the row's position.  The slice depends on the unit's place inside
    // its head (sub = u % upd), not on the head, and a warp's units u = half, half + 2, ... only ever have the places
    // sub0 = half % upd and sub1 = (half + 2) % upd: both slices are fetched once per tile, before the wait for the
    // accumulator, instead of once per unit.
    auto fetch = [&](int sub, float* tab) {
        if (!row_ok) return;
        const int j0 = sub * 16;
        ld256(csr + j0, tab); ld256(csr + j0 + 8, tab + 8);
    };
    const bool rotates = n0 / dh < p.nq + p.nkv;          // the tile starts in a q or k head (v heads are not rotated)
    const int sub0 = half % upd, sub1 = (half + 2) % upd;
    float tab0[16], tab1[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) { tab0[i] = 0.f; tab1[i] = 0.f; }
    if (rotates) { fetch(sub0, tab0); if (sub1 != sub0) fetch(sub1, tab1); }
    if (!wait()) return false;
    auto unit = [&](int u, const float* tab) -> bool {     // false: past the last head (uniform across the warp)
        const int hc = u / upd, sub = u % upd;
        const int hs = n0 / dh + hc;                       // head slot: q heads, then k heads, then v heads
        if (hs >= heads_total) return false;
        const bool is_v = hs >= p.nq + p.nkv;
        float lo[16], hi[16];
        const int c_lo = hc * dh + (is_v ? sub * 32 : sub * 16);
        const int c_hi = is_v ? c_lo + 16 : c_lo + halfdh;
        tc_ld16(taddr + c_lo, lo);
        tc_ld16(taddr + c_hi, hi);
        __nv_bfloat16* dst;
        bool st_ok;
        if (hs < p.nq) {
            dst = p.q_out + ((size_t)t * p.M + row) * (size_t)(p.nq * dh) + (size_t)hs * dh;
            st_ok = row_ok;
        } else {
            const int kv = is_v ? 1 : 0, head = hs - p.nq - kv * p.nkv;
            dst = p.pool_l + (size_t)t * p.pool_tstride + kvoff + ((int64_t)kv * p.nkv + head) * p.ps * dh;
            st_ok = slot_ok;
        }
        tc_wait_ld();
        if (st_ok) {
            if (!is_v) {
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float l = lo[i] * rinv, h = hi[i] * rinv;
                    const uint32_t w = __float_as_uint(tab[i]);
                    const float2 cs = __half22float2(*reinterpret_cast<const __half2*>(&w));
                    lo[i] = l * cs.x - h * cs.y;
                    hi[i] = h * cs.x + l * cs.y;
                }
                store16_bf16(dst + sub * 16, lo);
                store16_bf16(dst + halfdh + sub * 16, hi);
            } else {
#pragma unroll
                for (int i = 0; i < 16; ++i) { lo[i] *= rinv; hi[i] *= rinv; }
                store16_bf16(dst + sub * 32, lo);
                store16_bf16(dst + sub * 32 + 16, hi);
            }
        }
        return true;
    };
#pragma unroll 1
    for (int u = half; u < UNITS; u += 4) {                // two units per turn: places sub0 and sub1
        if (!unit(u, tab0)) break;
        if (u + 2 < UNITS && !unit(u + 2, sub1 != sub0 ? tab1 : tab0)) break;
    }
    return true;
}

// Residual add (+ track-sync sum), fp32 stream out, gain-scaled bf16 copy, partial sums of squares.
// tcgen05.ld leaves one accumulator row per thread; global accesses in that shape touch 32 different
// 128-byte lines per instruction, and this epilogue moves 10-14 bytes per element, so it was bound by
// load/store-unit wavefronts.  Each 32 x 32 unit is therefore turned through the warp's 4 KB of shared
// memory (16-byte chunks XOR-swizzled by row, conflict-free both ways) into "four lanes per row, eight
// columns per lane": every global instruction then covers 8 rows x 128 contiguous bytes.  Residual rows
// are fetched in the same shape, one unit ahead and before the wait for the accumulator.
template <int BN, class Wait>
__device__ __forceinline__ bool epi_resid(const GemmP& p, uint32_t taddr, int t, int row, int n0, int half, uint8_t* xbuf, Wait wait) {
    constexpr int UNITS = BN / 32;                        // 32-column units of the tile; 64-column groups alternate between the two warps
    const int lane = threadIdx.x & 31;
    const int row0 = row - lane;                          // first row of the warp's 32
    const int rsub = lane >> 2, cc = (lane & 3) * 8;      // this thread: rows row0 + 8r + rsub (r = 0..3), columns cc..cc+7 of the unit
    const float* hbase = p.h_in + (size_t)(p.n_sum > 1 ? 0 : t) * p.h_in_tstride;
    auto fetch = [&](int u, float* h) {                   // h[8r..8r+7]: residual of row r (summed over tracks at a sync)
        const int col = n0 + u * 32 + cc;
#pragma unroll
        for (int i = 0; i < 32; ++i) h[i] = 0.f;
        if (col >= p.N) return;
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int rr = row0 + 8 * r + rsub;
            if (rr < p.M) ld256(hbase + (size_t)rr * p.N + col, h + 8 * r);
        }
        for (int tt = 1; tt < p.n_sum; ++tt) {
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const int rr = row0 + 8 * r + rsub;
                if (rr < p.M) {
                    float x[8];
                    ld256(hbase + (size_t)tt * p.h_in_tstride + (size_t)rr * p.N + col, x);
#pragma unroll
                    for (int k = 0; k < 8; ++k) h[8 * r + k] += x[k];
                }
            }
        }
    };
    const uint32_t xs = smem_u32(xbuf);
    const uint32_t st_base = xs + lane * 128;                         // row-per-thread side: my row
    const uint32_t sw = (uint32_t)(lane & 7);
    float hres[32], hnxt[32];
    fetch(2 * half, hres);
    if (!wait()) return false;
    float ssq[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
    for (int u = 2 * half; u < UNITS; u += (u & 1) ? 3 : 1) {      // units 0,1, 4,5, ... or 2,3, 6,7, ...
        const int c = u * 32;
        if (n0 + c >= p.N) break;                          // uniform across the warp
        const int col = n0 + c + cc;
        const bool col_ok = col < p.N;
        float v[32];
        tc_ld16(taddr + c, v);
        tc_ld16(taddr + c + 16, v + 16);
        const int un = u + ((u & 1) ? 3 : 1);
        if (un < UNITS) fetch(un, hnxt);
        tc_wait_ld();
        __syncwarp();                                      // the previous unit's reads of the buffer are done
#pragma unroll
        for (int j = 0; j < 8; ++j)
            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(st_base + ((j ^ sw) << 4)),
                         "f"(v[4 * j]), "f"(v[4 * j + 1]), "f"(v[4 * j + 2]), "f"(v[4 * j + 3]) : "memory");
        __syncwarp();
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const uint32_t rb = xs + (8 * r + rsub) * 128;            // (8r + rsub) & 7 == rsub
#pragma unroll
            for (int h2 = 0; h2 < 2; ++h2) {
                const uint32_t chunk = (uint32_t)(2 * (lane & 3) + h2) ^ (uint32_t)rsub;
                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                             : "=f"(v[8 * r + 4 * h2]), "=f"(v[8 * r + 4 * h2 + 1]), "=f"(v[8 * r + 4 * h2 + 2]), "=f"(v[8 * r + 4 * h2 + 3])
                             : "r"(rb + (chunk << 4)) : "memory");
            }
        }
        float part[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int rr = row0 + 8 * r + rsub;
            const bool ok = col_ok && rr < p.M;
            float sq = 0.f;
#pragma unroll
            for (int k = 0; k < 8; ++k) { v[8 * r + k] = (v[8 * r + k] + hres[8 * r + k]) * p.scale; sq += v[8 * r + k] * v[8 * r + k]; }
            part[r] = ok ? sq : 0.f;
            if (ok) st256(p.h_out + (size_t)t * p.h_out_tstride + (size_t)rr * p.N + col, v + 8 * r);
        }
        if (p.hb_out && col_ok) {
            for (int to = 0; to < p.n_out; ++to) {
                const int tg = p.n_out > 1 ? to : t;
                const float4 g0 = *(const float4*)(p.gain + (size_t)tg * p.N + col), g1 = *(const float4*)(p.gain + (size_t)tg * p.N + col + 4);
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const int rr = row0 + 8 * r + rsub;
                    if (rr < p.M) {
                        const float* w = v + 8 * r;
                        uint4 o;
                        o.x = pack_bf16(w[0] * g0.x, w[1] * g0.y); o.y = pack_bf16(w[2] * g0.z, w[3] * g0.w);
                        o.z = pack_bf16(w[4] * g1.x, w[5] * g1.y); o.w = pack_bf16(w[6] * g1.z, w[7] * g1.w);
                        *reinterpret_cast<uint4*>(p.hb_out + ((size_t)tg * p.M + rr) * p.N + col) = o;
                    }
                }
            }
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) {                      // row sums over the four lanes of a row
            part[r] += __shfl_xor_sync(0xffffffffu, part[r], 1);
            part[r] += __shfl_xor_sync(0xffffffffu, part[r], 2);
            ssq[r] += part[r];
        }
        if ((u & 1) == 1 || n0 + c + 32 >= p.N) {          // a kSsqTile-column group is complete
            if (p.ssq_out && (lane & 3) == 0) {
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const int rr = row0 + 8 * r + rsub;
                    if (rr < p.M) p.ssq_out[(size_t)t * p.ssq_out_tstride + (size_t)rr * p.ssq_out_tiles + (n0 + c) / kSsqTile] = ssq[r];
                }
            }
#pragma unroll
            for (int r = 0; r < 4; ++r) ssq[r] = 0.f;
        }
#pragma unroll
        for (int i = 0; i < 32; ++i) hres[i] = hnxt[i];     // last: the fetch stays in flight until here
    }
    return true;
}

template <int BN, int EPI, class Wait>
__device__ __forceinline__ bool epilogue(const GemmP& p, uint32_t taddr, int t, int row, bool row_ok, int n0, int half, uint8_t* xbuf, Wait wait) {
    if (EPI == EPI_PLAIN) return epi_plain<BN>(p, taddr, t, row, row_ok, n0, half, wait);
    else if (EPI == EPI_QKV) return epi_qkv<BN>(p, taddr, t, row, row_ok, n0, half, wait);
    else if (EPI == EPI_SWIGLU) return epi_swiglu<BN>(p, taddr, t, row, row_ok, n0, half, wait);
    else return epi_resid<BN>(p, taddr, t, row, n0, half, xbuf, wait);
}

// Tile index -> (column tile, row tile, track).  With one or two row tiles (a decode step) the row
// tile runs fastest, so the CTAs that stream the same W tile are neighbours in time and the second one
// finds it in L2; with many row tiles the column tile runs fastest and neighbours share their A tile.
__device__ __forceinline__ void tile_coords(const GemmP& p, int tile, int& nt, int& mt, int& t) {
    if (p.tiles_m <= 2) { mt = tile % p.tiles_m; nt = (tile / p.tiles_m) % p.tiles_n; }
    else { nt = tile % p.tiles_n; mt = (tile / p.tiles_n) % p.tiles_m; }
    t = tile / (p.tiles_n * p.tiles_m);
}

template <int BN, int EPI>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_tc(const __grid_constant__ CUtensorMap ta, const __grid_constant__ CUtensorMap tb, const GemmP p) {
    using C = Cfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* xpose = smem + kRingBytes;
    uint64_t* full = (uint64_t*)(xpose + kXposeBytes);
    uint64_t* empty = full + kMaxStages;
    uint64_t* acc_full = empty + kMaxStages;
    uint64_t* acc_empty = acc_full + 2;
    uint32_t* tmem_slot = (uint32_t*)(acc_empty + 2);
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
    const int stages = p.stages, kps = p.kps;
    const uint32_t a_bytes = p.a_bytes, w_off = kps * p.a_bytes, stage_bytes = kps * (p.a_bytes + C::B_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], kEpiWarps); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(2 * BN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int num_tiles = p.tiles_m * p.tiles_n * p.T;
    const int kpb = (p.K + BK - 1) / BK;            // k-blocks per track
    const int kblocks = kpb * p.kt;
    const int nsteps = kblocks / kps;                // ring stages one tile consumes (kps divides kblocks)
    const uint32_t stage_tx = p.a_tx + p.w_tx;

    if (warp == 0) {
        if (lane == 0) {
            // Model weights are written by no kernel, so the first ring generation of W tiles is requested
            // before the wait for the previous kernel: their stream is under way when its results arrive.
            int npre = 0;
            auto load_w = [&](int s, int it, int nt, int t) {
                uint8_t* sw = smem + s * stage_bytes + w_off;
                if (kps > 1) tma_load_4d(sw, &tb, &full[s], 0, nt * BN, it * kps, t);        // kps k-blocks in one copy
                else tma_load_3d(sw, &tb, &full[s], (p.kt > 1 ? it % kpb : it) * BK, nt * BN, p.kt > 1 ? it / kpb : t);
            };
            if (p.w_static && (int)blockIdx.x < num_tiles) {
                int nt, mt, t;
                tile_coords(p, blockIdx.x, nt, mt, t);
                npre = min(stages, nsteps);
                for (int it = 0; it < npre; ++it) {
                    mbar_expect_tx(&full[it], stage_tx);
                    load_w(it, it, nt, t);
                }
            }
            grid_dep_wait();
            grid_dep_launch();
            int s = 0; uint32_t ph = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                int nt, mt, t;
                tile_coords(p, tile, nt, mt, t);
                if (kps == 1) {
                    // grouped rows: this row tile's expert shifts the W coordinates (the table is written by a kernel of
                    // the stream, so such launches never prefetch W before the wait: npre is 0)
                    const int ex = p.tile_expert ? p.tile_expert[t * p.tiles_m + mt] : 0;
                    const int w_row = nt * BN + ex * p.w_row_per_expert, w_k = ex * p.w_k_per_expert;
                    for (int kb = 0; kb < kblocks; ++kb) {
                        const int tt = p.kt > 1 ? kb / kpb : t;
                        const int k0 = (p.kt > 1 ? kb % kpb : kb) * BK;
                        uint8_t* sa = smem + s * stage_bytes;
                        if (kb < npre) {                               // the stage is armed and its W copy on the way
                            tma_load_3d(sa, &ta, &full[s], k0, mt * BM, tt);
                        } else {
                            if (!mbar_wait(&empty[s], ph ^ 1, abort_flag)) { ok = false; report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_GEMM_EMPTY_WAIT); *abort_flag = 1; break; }
                            mbar_expect_tx(&full[s], stage_tx);
                            tma_load_3d(sa, &ta, &full[s], k0, mt * BM, tt);
                            tma_load_3d(sa + a_bytes, &tb, &full[s], k0 + w_k, w_row, tt);
                        }
                        if (++s == stages) { s = 0; ph ^= 1; }
                    }
                } else {
                    for (int it = 0; it < nsteps; ++it) {
                        if (it >= npre) {
                            if (!mbar_wait(&empty[s], ph ^ 1, abort_flag)) { ok = false; report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_GEMM_EMPTY_WAIT); *abort_flag = 1; break; }
                            mbar_expect_tx(&full[s], stage_tx);
                        }
                        tma_load_4d(smem + s * stage_bytes, &ta, &full[s], 0, mt * BM, it * kps, t);    // kps k-blocks of A, a_bytes apart
                        if (it >= npre) load_w(s, it, nt, t);
                        if (++s == stages) { s = 0; ph ^= 1; }
                    }
                }
                npre = 0;
            }
        } else {
            grid_dep_wait();
        }
        __syncwarp();
    } else if (warp == 1) {
        // whole warp walks the loop; the tcgen05 instructions run on one elected lane
        grid_dep_wait();
        constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
        const uint64_t desc0 = smem_desc(smem_u32(smem));
        int s = 0; uint32_t ph = 0;
        int a = 0; uint32_t aph = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
            if (!__all_sync(0xffffffffu, mbar_wait(&acc_empty[a], aph ^ 1, abort_flag))) {
                if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_GEMM_ACC_WAIT); *abort_flag = 1; }
                break;
            }
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + a * BN;
            if (kps == 1) {
                // one k-block per stage (every launch with many rows): the loop that bounds the tensor pipe
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!__all_sync(0xffffffffu, mbar_wait(&full[s], ph, abort_flag))) {
                        ok = false;
                        if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_GEMM_TMA_WAIT); *abort_flag = 1; }
                        break;
                    }
                    tc_fence_after();
                    const uint64_t da = desc0 + (uint64_t)((s * stage_bytes) >> 4), db = da + (uint64_t)(a_bytes >> 4);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        tc_mma(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
                    tc_commit(&empty[s]);                     // frees the stage when these MMAs retire
                    if (++s == stages) { s = 0; ph ^= 1; }
                }
            } else {
                for (int it = 0; it < nsteps; ++it) {
                    if (!__all_sync(0xffffffffu, mbar_wait(&full[s], ph, abort_flag))) {
                        ok = false;
                        if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_GEMM_TMA_WAIT); *abort_flag = 1; }
                        break;
                    }
                    tc_fence_after();
                    uint64_t da = desc0 + (uint64_t)((s * stage_bytes) >> 4), db = da + (uint64_t)(w_off >> 4);
                    for (int j = 0; j < kps; ++j) {
#pragma unroll
                        for (int k = 0; k < BK / 16; ++k)
                            tc_mma(d_tmem, da + 2 * k, db + 2 * k, idesc, (it | j | k) != 0);
                        da += a_bytes >> 4;
                        db += p.w_kb_bytes >> 4;
                    }
                    tc_commit(&empty[s]);
                    if (++s == stages) { s = 0; ph ^= 1; }
                }
            }
            if (!ok) break;
            tc_commit(&acc_full[a]);                      // accumulator complete
            if (++a == 2) { a = 0; aph ^= 1; }
        }
        __syncwarp();
    } else {
        const int q = warp & 3;                            // TMEM lane quarter this warp may read
        const int half = (warp - 2) >> 2;                  // which half of the tile's 32-column units it takes
        grid_dep_wait();
        int a = 0; uint32_t aph = 0;
        for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
            int nt, mt, t;
            tile_coords(p, tile, nt, mt, t);
            const int row = mt * BM + q * 32 + lane;       // the row this thread holds after tcgen05.ld
            const bool row_ok = row < p.M;
            const int n0 = nt * BN;
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + a * BN;
            auto wait_acc = [&]() -> bool {
                bool ok = mbar_wait(&acc_full[a], aph, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) { if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_GEMM_EPI_WAIT); *abort_flag = 1; } return false; }
                tc_fence_after();
                return true;
            };
            if (!epilogue<BN, EPI>(p, taddr, t, row, row_ok, n0, half, xpose + (warp - 2) * 4096, wait_acc)) break;
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[a]);
            if (++a == 2) { a = 0; aph ^= 1; }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2 * BN) : "memory");
    }
}

// ---- CTA-pair variant ------------------------------------------------------------------------
// With one CTA per tile the main loop of a 128 x 256 tile pulls 48 KB per k-block into the SM, and that
// copy (about 70 bytes per cycle per SM) takes longer than the 512 cycles of its four MMAs.  Two CTAs of a
// cluster therefore share a 256 x 256 tile: each loads its own 128 rows of A and HALF of the W tile (128
// rows), and one tcgen05.mma.cta_group::2 per 16 columns of K, issued by the even CTA, multiplies both A
// halves with both W halves, leaving each CTA the accumulator of its own 128 rows in its own tensor
// memory.  Per CTA and k-block: 32 KB copied for the same 512 MMA cycles, and six ring stages.
// Barriers live at the same shared-memory offsets in both CTAs.  The even CTA's full[s] collects both
// CTAs' copies (two arrivals with expected bytes); after the MMAs of a stage it commits to both CTAs'
// empty[s], after a tile to both CTAs' acc_full[a]; the epilogue warps of both CTAs arrive at the even
// CTA's acc_empty[a].  Every copy has exactly one destination CTA.  Every wait is bounded as in gemm_tc.
constexpr int kPairStages = 6;
constexpr int kPairStageBytes = 2 * BM * BK * 2;             // 128 rows of A + 128 rows of W per k-block

__device__ __forceinline__ uint32_t cluster_rank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx_cluster(uint32_t bar_cluster_addr, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(bar_cluster_addr), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
// copy whose completion bytes go to a barrier of the even CTA of the pair
__device__ __forceinline__ void tma_load_3d_pair(void* dst, const CUtensorMap* map, uint32_t bar_cluster_addr, int c0, int c1, int c2) {
    asm volatile("cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(smem_u32(dst)), "l"((uint64_t)map), "r"(c0), "r"(c1), "r"(c2), "r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n .reg .pred p, e;\n elect.sync _|e, 0xffffffff;\n setp.ne.b32 p, %4, 0;\n"
                 " @e tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar_cluster_addr) {
    asm volatile("{\n .reg .pred e;\n elect.sync _|e, 0xffffffff;\n"
                 " @e tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];\n}" ::"r"(bar_cluster_addr) : "memory");
}

template <int EPI>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_tc_pair(const __grid_constant__ CUtensorMap ta, const __grid_constant__ CUtensorMap tb, const GemmP p) {
    constexpr int BN = 256;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* xpose = smem + kRingBytes;
    uint64_t* full = (uint64_t*)(xpose + kXposeBytes);
    uint64_t* empty = full + kMaxStages;
    uint64_t* acc_full = empty + kMaxStages;
    uint64_t* acc_empty = acc_full + 2;
    uint32_t* tmem_slot = (uint32_t*)(acc_empty + 2);
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
    const uint32_t rank = cluster_rank();                   // 0: issues the MMAs; 1: its partner
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kPairStages; ++s) { mbar_init(&full[s], 2); mbar_init(&empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], 2 * kEpiWarps); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {                                        // the same warp of both CTAs, the same slot address
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(2 * BN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                     // both CTAs' barriers exist before anything arrives at them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int tiles_m2 = (p.M + 2 * BM - 1) / (2 * BM);     // row tiles of 256
    const int num_tiles = tiles_m2 * p.tiles_n * p.T;
    const int kpb = (p.K + BK - 1) / BK;
    const int kblocks = kpb * p.kt;
    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
    auto coords = [&](int tile, int& nt, int& mt2, int& t) { nt = tile % p.tiles_n; mt2 = (tile / p.tiles_n) % tiles_m2; t = tile / (p.tiles_n * tiles_m2); };
    grid_dep_wait();
    if (threadIdx.x == 0) grid_dep_launch();

    if (warp == 0) {
        if (lane == 0) {
            int s = 0; uint32_t ph = 0;
            bool ok = true;
            for (int tile = pair; tile < num_tiles && ok; tile += npairs) {
                int nt, mt2, t;
                coords(tile, nt, mt2, t);
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(&empty[s], ph ^ 1, abort_flag)) { ok = false; report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_GEMM_EMPTY_WAIT); *abort_flag = 1; break; }
                    const int tt = p.kt > 1 ? kb / kpb : t;
                    const int k0 = (p.kt > 1 ? kb % kpb : kb) * BK;
                    uint8_t* sa = smem + s * kPairStageBytes;
                    const uint32_t fb = map_to_cta(smem_u32(&full[s]), 0);
                    mbar_expect_tx_cluster(fb, p.a_tx + p.w_tx);
                    tma_load_3d_pair(sa, &ta, fb, k0, (mt2 * 2 + (int)rank) * BM, tt);
                    tma_load_3d_pair(sa + BM * BK * 2, &tb, fb, k0, nt * BN + (int)rank * (BN / 2), tt);
                    if (++s == kPairStages) { s = 0; ph ^= 1; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (rank == 0) {
            constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24);
            const uint64_t desc0 = smem_desc(smem_u32(smem));
            int s = 0; uint32_t ph = 0;
            int a = 0; uint32_t aph = 0;
            bool ok = true;
            for (int tile = pair; tile < num_tiles && ok; tile += npairs) {
                if (!__all_sync(0xffffffffu, mbar_wait(&acc_empty[a], aph ^ 1, abort_flag))) {
                    if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_GEMM_ACC_WAIT); *abort_flag = 1; }
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + a * BN;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!__all_sync(0xffffffffu, mbar_wait(&full[s], ph, abort_flag))) {
                        ok = false;
                        if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_GEMM_TMA_WAIT); *abort_flag = 1; }
                        break;
                    }
                    tc_fence_after();
                    const uint64_t da = desc0 + (uint64_t)((s * kPairStageBytes) >> 4), db = da + (uint64_t)((BM * BK * 2) >> 4);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        tc_mma_pair(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
                    tc_commit_pair(smem_u32(&empty[s]));                        // both CTAs may refill the stage
                    tc_commit_pair(map_to_cta(smem_u32(&empty[s]), 1));
                    if (++s == kPairStages) { s = 0; ph ^= 1; }
                }
                if (!ok) break;
                tc_commit_pair(smem_u32(&acc_full[a]));                         // both CTAs' epilogues may drain
                tc_commit_pair(map_to_cta(smem_u32(&acc_full[a]), 1));
                if (++a == 2) { a = 0; aph ^= 1; }
            }
        }
        __syncwarp();
    } else {
        const int q = warp & 3;
        const int half = (warp - 2) >> 2;
        int a = 0; uint32_t aph = 0;
        for (int tile = pair; tile < num_tiles; tile += npairs) {
            int nt, mt2, t;
            coords(tile, nt, mt2, t);
            const int row = (mt2 * 2 + (int)rank) * BM + q * 32 + lane;
            const bool row_ok = row < p.M;
            const int n0 = nt * BN;
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + a * BN;
            auto wait_acc = [&]() -> bool {
                bool ok = mbar_wait(&acc_full[a], aph, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) { if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_GEMM_EPI_WAIT); *abort_flag = 1; } return false; }
                tc_fence_after();
                return true;
            };
            if (!epilogue<BN, EPI>(p, taddr, t, row, row_ok, n0, half, xpose + (warp - 2) * 4096, wait_acc)) break;
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&acc_empty[a]), 0));
            if (++a == 2) { a = 0; aph ^= 1; }
        }
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                     // the partner's shared and tensor memory are in use until both are here
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2 * BN) : "memory");
    }
}

// The same pair kernel for the plain residual epilogue (one residual stream in, one track's operand out), with the
// epilogue's global traffic on the TMA unit instead of the load/store unit: per 32 x 32 unit a warp receives the residual
// rows as one 4 KB box in shared memory, adds them row-per-thread (128-byte swizzled, conflict-free), puts the fp32 result
// and the gain-scaled bf16 copy back into shared memory and stores both as boxes.  The shared memory for it (10 KB per
// epilogue warp) comes from the ring: four stages.
constexpr int kRtStages = 4;
constexpr int kRtStageBytes = 10 * 1024;                     // per epilogue warp: residual in 4 KB, fp32 out 4 KB, bf16 out 2 KB

__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3}], [%4];"
                 ::"l"((uint64_t)map), "r"(c0), "r"(c1), "r"(c2), "r"(src) : "memory");
}

__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_tc_pair_resid(const __grid_constant__ CUtensorMap ta, const __grid_constant__ CUtensorMap tb,
                   const __grid_constant__ CUtensorMap th_in, const __grid_constant__ CUtensorMap th_out,
                   const __grid_constant__ CUtensorMap thb, const GemmP p) {
    constexpr int BN = 256;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* staging = smem + kRtStages * kPairStageBytes;
    uint64_t* full = (uint64_t*)(smem + kRingBytes + kXposeBytes);
    uint64_t* empty = full + kMaxStages;
    uint64_t* acc_full = empty + kMaxStages;
    uint64_t* acc_empty = acc_full + 2;
    uint32_t* tmem_slot = (uint32_t*)(acc_empty + 2);
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
    uint64_t* inbar = (uint64_t*)(tmem_slot + 2);           // one per epilogue warp: its residual box has landed
    const uint32_t rank = cluster_rank();                   // 0: issues the MMAs; 1: its partner
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kRtStages; ++s) { mbar_init(&full[s], 2); mbar_init(&empty[s], 1); }
        for (int w = 0; w < kEpiWarps; ++w) mbar_init(&inbar[w], 1);
        for (int a = 0; a < 2; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], 2 * kEpiWarps); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {                                        // the same warp of both CTAs, the same slot address
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(2 * BN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                     // both CTAs' barriers exist before anything arrives at them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int tiles_m2 = (p.M + 2 * BM - 1) / (2 * BM);     // row tiles of 256
    const int num_tiles = tiles_m2 * p.tiles_n * p.T;
    const int kpb = (p.K + BK - 1) / BK;
    const int kblocks = kpb * p.kt;
    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
    auto coords = [&](int tile, int& nt, int& mt2, int& t) { nt = tile % p.tiles_n; mt2 = (tile / p.tiles_n) % tiles_m2; t = tile / (p.tiles_n * tiles_m2); };
    grid_dep_wait();
    if (threadIdx.x == 0) grid_dep_launch();

    if (warp == 0) {
        if (lane == 0) {
            int s = 0; uint32_t ph = 0;
            bool ok = true;
            for (int tile = pair; tile < num_tiles && ok; tile += npairs) {
                int nt, mt2, t;
                coords(tile, nt, mt2, t);
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(&empty[s], ph ^ 1, abort_flag)) { ok = false; report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_GEMM_EMPTY_WAIT); *abort_flag = 1; break; }
                    const int tt = p.kt > 1 ? kb / kpb : t;
                    const int k0 = (p.kt > 1 ? kb % kpb : kb) * BK;
                    uint8_t* sa = smem + s * kPairStageBytes;
                    const uint32_t fb = map_to_cta(smem_u32(&full[s]), 0);
                    mbar_expect_tx_cluster(fb, p.a_tx + p.w_tx);
                    tma_load_3d_pair(sa, &ta, fb, k0, (mt2 * 2 + (int)rank) * BM, tt);
                    tma_load_3d_pair(sa + BM * BK * 2, &tb, fb, k0, nt * BN + (int)rank * (BN / 2), tt);
                    if (++s == kRtStages) { s = 0; ph ^= 1; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (rank == 0) {
            constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24);
            const uint64_t desc0 = smem_desc(smem_u32(smem));
            int s = 0; uint32_t ph = 0;
            int a = 0; uint32_t aph = 0;
            bool ok = true;
            for (int tile = pair; tile < num_tiles && ok; tile += npairs) {
                if (!__all_sync(0xffffffffu, mbar_wait(&acc_empty[a], aph ^ 1, abort_flag))) {
                    if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_GEMM_ACC_WAIT); *abort_flag = 1; }
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + a * BN;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!__all_sync(0xffffffffu, mbar_wait(&full[s], ph, abort_flag))) {
                        ok = false;
                        if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_GEMM_TMA_WAIT); *abort_flag = 1; }
                        break;
                    }
                    tc_fence_after();
                    const uint64_t da = desc0 + (uint64_t)((s * kPairStageBytes) >> 4), db = da + (uint64_t)((BM * BK * 2) >> 4);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        tc_mma_pair(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
                    tc_commit_pair(smem_u32(&empty[s]));                        // both CTAs may refill the stage
                    tc_commit_pair(map_to_cta(smem_u32(&empty[s]), 1));
                    if (++s == kRtStages) { s = 0; ph ^= 1; }
                }
                if (!ok) break;
                tc_commit_pair(smem_u32(&acc_full[a]));                         // both CTAs' epilogues may drain
                tc_commit_pair(map_to_cta(smem_u32(&acc_full[a]), 1));
                if (++a == 2) { a = 0; aph ^= 1; }
            }
        }
        __syncwarp();
    } else {
        const int q = warp & 3;
        const int half = (warp - 2) >> 2;
        const int ew = warp - 2;
        uint8_t* stg = staging + ew * kRtStageBytes;
        const uint32_t s_in = smem_u32(stg), s_out = s_in + 4096, s_outb = s_in + 8192;
        uint64_t* ib = &inbar[ew];
        uint32_t inph = 0;
        bool in_flight = false;                                            // a residual box has been requested and not yet consumed
        constexpr int UNITS = BN / 32;
        int a = 0; uint32_t aph = 0;
        bool ok = true;
        for (int tile = pair; tile < num_tiles && ok; tile += npairs) {
            int nt, mt2, t;
            coords(tile, nt, mt2, t);
            const int r0 = (mt2 * 2 + (int)rank) * BM + q * 32;          // first of this warp's 32 rows
            const int row = r0 + lane;
            const bool row_ok = row < p.M;
            const int n0 = nt * BN;
            const int t_in = p.h_in_tstride ? t : 0, t_out = p.h_out_tstride ? t : 0;
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + a * BN;
            auto issue_in = [&](int u) {                                   // residual rows of unit u: one box
                if (lane == 0) { mbar_expect_tx(ib, 4096); tma_load_3d(stg, &th_in, ib, n0 + u * 32, r0, t_in); }
                in_flight = true;
            };
            const int u_first = 2 * half;
            if (n0 + u_first * 32 < p.N) issue_in(u_first);
            {
                bool w = mbar_wait(&acc_full[a], aph, abort_flag);
                w = __all_sync(0xffffffffu, w);
                if (!w) { if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_GEMM_EPI_WAIT); *abort_flag = 1; } break; }
                tc_fence_after();
            }
            float ssq = 0.f;
#pragma unroll 1
            for (int u = u_first; u < UNITS; u += (u & 1) ? 3 : 1) {       // units 0,1, 4,5, ... or 2,3, 6,7, ...
                const int c = u * 32, col = n0 + c;
                if (col >= p.N) break;                                      // uniform across the warp
                float v[32], h[32];
                tc_ld16(taddr + c, v);
                tc_ld16(taddr + c + 16, v + 16);
                if (!__all_sync(0xffffffffu, mbar_wait(ib, inph, abort_flag))) {
                    if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_GEMM_EPI_WAIT); *abort_flag = 1; }
                    ok = false; break;
                }
                inph ^= 1;
                in_flight = false;
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(h[4 * j]), "=f"(h[4 * j + 1]), "=f"(h[4 * j + 2]), "=f"(h[4 * j + 3])
                                 : "r"(s_in + lane * 128 + ((j ^ (lane & 7)) << 4)) : "memory");
                __syncwarp();                                               // every lane has its residual row: the box is free
                const int un = u + ((u & 1) ? 3 : 1);
                if (un < UNITS && n0 + un * 32 < p.N) issue_in(un);
                tc_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) { v[i] = (v[i] + h[i]) * p.scale; if (row_ok) ssq += v[i] * v[i]; }
                if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the previous unit's stores have read their boxes
                __syncwarp();
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(s_out + lane * 128 + ((j ^ (lane & 7)) << 4)),
                                 "f"(v[4 * j]), "f"(v[4 * j + 1]), "f"(v[4 * j + 2]), "f"(v[4 * j + 3]) : "memory");
                if (p.hb_out) {
                    const float4* gp = (const float4*)(p.gain + (size_t)t * p.N + col);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {                          // 16-byte chunks of 8 bf16, 64-byte swizzle
                        const float4 g0 = col + 8 * j < p.N ? gp[2 * j] : make_float4(0.f, 0.f, 0.f, 0.f);
                        const float4 g1 = col + 8 * j < p.N ? gp[2 * j + 1] : make_float4(0.f, 0.f, 0.f, 0.f);
                        const float* w = v + 8 * j;
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(s_outb + lane * 64 + ((j ^ ((lane >> 1) & 3)) << 4)),
                                     "r"(pack_bf16(w[0] * g0.x, w[1] * g0.y)), "r"(pack_bf16(w[2] * g0.z, w[3] * g0.w)),
                                     "r"(pack_bf16(w[4] * g1.x, w[5] * g1.y)), "r"(pack_bf16(w[6] * g1.z, w[7] * g1.w)) : "memory");
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0 && r0 < p.M) {                               // rows and columns past the ends are clipped by the copy
                    tma_store_3d(&th_out, s_out, col, r0, t_out);
                    if (p.hb_out) tma_store_3d(&thb, s_outb, col, r0, t);
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
                if ((u & 1) == 1 || col + 32 >= p.N) {                     // a kSsqTile-column group is complete
                    if (row_ok && p.ssq_out) p.ssq_out[(size_t)t * p.ssq_out_tstride + (size_t)row * p.ssq_out_tiles + col / kSsqTile] = ssq;
                    ssq = 0.f;
                }
            }
            if (!ok) break;
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&acc_empty[a]), 0));
            if (++a == 2) { a = 0; aph ^= 1; }
        }
        if (in_flight) mbar_wait(ib, inph, abort_flag);                     // only after a time-out elsewhere: let the copy land before the CTA ends
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // every store of this warp has completed
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                     // the partner's shared and tensor memory are in use until both are here
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(2 * BN) : "memory");
    }
}

// One CTA, one mbarrier that nothing arrives at: the wait must give up after limit_ns, record the timeout and return.
__global__ void k_wait_selftest(int* status, unsigned long long limit_ns) {
    __shared__ uint64_t bar;
    __shared__ int abort_word;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0 && !mbar_wait(&bar, 0, &abort_word, limit_ns)) report(status, PT_ERR_DEVICE_TIMEOUT, LOC_SELFTEST_WAIT);
}

template <int BN, int EPI>
pt_status launch_t(const CUtensorMap& ta, const CUtensorMap& tb, GemmP p, cudaStream_t st, int sms) {
    using C = Cfg<BN>;
    static bool attr_done_[kMaxDevices] = {};
    bool& attr_done = attr_done_[current_device()];
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(gemm_tc<BN, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmem);
        if (e != cudaSuccess) { set_error("cudaFuncSetAttribute: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
        attr_done = true;
    }
    if (p.kps < 1) p.kps = 1;
    p.a_bytes = (uint32_t)stage_a_bytes(p.M);
    p.stages = ring_stages((int)p.a_bytes, C::B_BYTES, p.kps);
    if (p.stages < 2 || ((p.K + BK - 1) / BK * p.kt) % p.kps) { set_error("GEMM ring: kps=%d does not fit M=%d K=%d bn=%d", p.kps, p.M, p.K, BN); return PT_ERR_UNSUPPORTED; }
    p.tiles_m = (p.M + BM - 1) / BM;
    p.tiles_n = (p.N + BN - 1) / BN;
    int tiles = p.tiles_m * p.tiles_n * p.T;
    int grid = std::min(tiles, sms);
    cudaError_t e = launch_dependent(gemm_tc<BN, EPI>, dim3(grid), dim3(kGemmThreads), (size_t)kGemmSmem, st, ta, tb, p);
    if (e != cudaSuccess) { set_error("GEMM launch: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return PT_OK;
}

template <int EPI>
pt_status launch_pair_t(const CUtensorMap& ta, const CUtensorMap& tb, GemmP p, cudaStream_t st, int sms) {
    static int max_pairs_[kMaxDevices] = {};           // 0 = not asked yet on that device
    int& max_pairs = max_pairs_[current_device()];
    if (max_pairs <= 0) {
        cudaError_t e = cudaFuncSetAttribute(gemm_tc_pair<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmem);
        if (e != cudaSuccess) { set_error("cudaFuncSetAttribute: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
        cudaLaunchConfig_t q = {};
        q.gridDim = dim3(sms & ~1); q.blockDim = dim3(kGemmThreads); q.dynamicSmemBytes = kGemmSmem;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension; at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        q.attrs = at; q.numAttrs = 1;
        int n = 0;
        e = cudaOccupancyMaxActiveClusters(&n, gemm_tc_pair<EPI>, &q);
        if (e != cudaSuccess || n < 1) { set_error("cudaOccupancyMaxActiveClusters: %s (%d clusters)", cudaGetErrorString(e), n); cudaGetLastError(); return PT_ERR_CUDA; }
        max_pairs = n;
    }
    p.a_tx = (uint32_t)std::min(BM, p.M) * BK * 2;
    p.w_tx = (uint32_t)std::min(BM, p.N) * BK * 2;
    p.tiles_n = (p.N + 255) / 256;
    const int tiles = ((p.M + 2 * BM - 1) / (2 * BM)) * p.tiles_n * p.T;
    const int pairs = std::min(tiles, max_pairs);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * pairs); cfg.blockDim = dim3(kGemmThreads); cfg.dynamicSmemBytes = kGemmSmem; cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension; at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization; at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 2;
    cudaError_t e = cudaLaunchKernelEx(&cfg, gemm_tc_pair<EPI>, ta, tb, p);
    if (e != cudaSuccess) { set_error("GEMM (CTA pairs) launch: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return PT_OK;
}

// 3-D map (column, row, track) of a row-major [tracks][rows][cols] array with 32 x 32 boxes for the epilogue's copies
pt_status make_box_map(CUtensorMap* out, bool bf16, const void* base, int64_t cols, int64_t rows, int64_t tracks, int64_t tstride_elems) {
    EncodeFn enc = get_encode();
    if (!enc) { set_error("cuTensorMapEncodeTiled is not available from this driver"); return PT_ERR_CUDA; }
    const int es = bf16 ? 2 : 4;
    cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)tracks};
    cuuint64_t strides[2] = {(cuuint64_t)cols * es, (cuuint64_t)(tracks > 1 ? tstride_elems : cols * rows) * es};
    cuuint32_t box[3] = {32, 32, 1};
    cuuint32_t ones[3] = {1, 1, 1};
    CUresult r = enc(out, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base), dims, strides, box, ones,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, bf16 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled (epilogue boxes) failed with code %d (cols=%lld rows=%lld tracks=%lld)", (int)r, (long long)cols, (long long)rows, (long long)tracks); return PT_ERR_CUDA; }
    return PT_OK;
}

// The plain residual epilogue on CTA pairs with its global traffic on the TMA unit; the caller has checked resid_by_tma().
pt_status launch_pair_resid(const CUtensorMap& ta, const CUtensorMap& tb, GemmP p, cudaStream_t st, int sms) {
    static int max_pairs_[kMaxDevices] = {};           // 0 = not asked yet on that device
    int& max_pairs = max_pairs_[current_device()];
    if (max_pairs <= 0) {
        cudaError_t e = cudaFuncSetAttribute(gemm_tc_pair_resid, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmem);
        if (e != cudaSuccess) { set_error("cudaFuncSetAttribute: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
        cudaLaunchConfig_t q = {};
        q.gridDim = dim3(sms & ~1); q.blockDim = dim3(kGemmThreads); q.dynamicSmemBytes = kGemmSmem;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension; at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        q.attrs = at; q.numAttrs = 1;
        int n = 0;
        e = cudaOccupancyMaxActiveClusters(&n, gemm_tc_pair_resid, &q);
        if (e != cudaSuccess || n < 1) { set_error("cudaOccupancyMaxActiveClusters: %s (%d clusters)", cudaGetErrorString(e), n); cudaGetLastError(); return PT_ERR_CUDA; }
        max_pairs = n;
    }
    CUtensorMap th_in, th_out, thb;
    pt_status s;
    if ((s = make_box_map(&th_in, false, p.h_in, p.N, p.M, p.h_in_tstride ? p.T : 1, (int64_t)p.h_in_tstride)) != PT_OK) return s;
    if ((s = make_box_map(&th_out, false, p.h_out, p.N, p.M, p.h_out_tstride ? p.T : 1, (int64_t)p.h_out_tstride)) != PT_OK) return s;
    if (p.hb_out) { if ((s = make_box_map(&thb, true, p.hb_out, p.N, p.M, p.T, (int64_t)p.M * p.N)) != PT_OK) return s; }
    else thb = th_out;
    p.a_tx = (uint32_t)std::min(BM, p.M) * BK * 2;
    p.w_tx = (uint32_t)std::min(BM, p.N) * BK * 2;
    p.tiles_n = (p.N + 255) / 256;
    const int tiles = ((p.M + 2 * BM - 1) / (2 * BM)) * p.tiles_n * p.T;
    const int pairs = std::min(tiles, max_pairs);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * pairs); cfg.blockDim = dim3(kGemmThreads); cfg.dynamicSmemBytes = kGemmSmem; cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension; at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization; at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 2;
    cudaError_t e = cudaLaunchKernelEx(&cfg, gemm_tc_pair_resid, ta, tb, th_in, th_out, thb, p);
    if (e != cudaSuccess) { set_error("GEMM (CTA pairs, residual by TMA) launch: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return PT_OK;
}

static bool resid_by_tma(const GemmP& p) {
    // One residual stream, this track's operand only, whole 32-column units, many rows - and a short K: the four-stage
    // ring costs a main-loop-bound GEMM more than the epilogue gains (measured at the cfg3 width: out-projection, K = 1024,
    // 730 -> 888 TFLOP/s; down, K = 2816, 9 % slower)
    return p.n_sum == 1 && p.n_out == 1 && p.kt == 1 && p.K <= 2048 && p.N % 32 == 0 && p.M >= 1024 && p.h_in && p.h_out
        && ((uintptr_t)p.h_in % 16) == 0 && ((uintptr_t)p.h_out % 16) == 0 && (p.h_in_tstride % 4) == 0 && (p.h_out_tstride % 4) == 0;
}

}  // namespace

EncodeFn get_encode() {
    static EncodeFn fn = nullptr;
    if (!fn) {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = (EncodeFn)f;
    }
    return fn;
}

pt_status make_map_bf16(CUtensorMap* out, const void* base, int64_t k, int64_t rows, int64_t tracks, int box_rows) {
    return make_map_bf16_strided(out, base, k, rows, tracks, k * 2 * rows, box_rows);
}

pt_status make_map_bf16_strided(CUtensorMap* out, const void* base, int64_t k, int64_t rows, int64_t tracks,
                                int64_t track_stride_bytes, int box_rows) {
    EncodeFn enc = get_encode();
    if (!enc) { set_error("cuTensorMapEncodeTiled is not available from this driver"); return PT_ERR_CUDA; }
    cuuint64_t dims[3] = {(cuuint64_t)k, (cuuint64_t)rows, (cuuint64_t)tracks};
    cuuint64_t strides[2] = {(cuuint64_t)k * 2, (cuuint64_t)track_stride_bytes};
    cuuint32_t box[3] = {(cuuint32_t)BK, (cuuint32_t)std::min<int64_t>(box_rows, rows), 1};
    cuuint32_t es[3] = {1, 1, 1};
    CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled failed with code %d (k=%lld rows=%lld tracks=%lld)", (int)r, (long long)k, (long long)rows, (long long)tracks); return PT_ERR_CUDA; }
    return PT_OK;
}

// Clusters of two CTAs with this kernel's shared memory must be launchable on the current device; asked once.
static bool pair_launchable() {
    static int state_[kMaxDevices] = {};               // 0 = not asked yet on that device, 1 = yes, 2 = no
    const int dev = current_device();
    int& state = state_[dev];
    if (state == 0) {
        state = 2;
        int sms = 0;
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (cudaFuncSetAttribute(gemm_tc_pair<EPI_PLAIN>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmem) == cudaSuccess && sms >= 2) {
            cudaLaunchConfig_t q = {};
            q.gridDim = dim3(sms & ~1); q.blockDim = dim3(kGemmThreads); q.dynamicSmemBytes = kGemmSmem;
            cudaLaunchAttribute at[1];
            at[0].id = cudaLaunchAttributeClusterDimension; at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
            q.attrs = at; q.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, gemm_tc_pair<EPI_PLAIN>, &q) == cudaSuccess && n >= 1) state = 1;
        }
        cudaGetLastError();
    }
    return state == 1;
}

// 129-1023 rows: pairs pay when there are enough 256 x 256 tiles to occupy most pairs (measured at 176 rows: gate/up with
// 176 tiles 11 % faster, QKV with 48 tiles 3 %, the projections back to the hidden size with 32 tiles 20 % slower).
static bool enough_pair_tiles(int N, int M, int T) {
    return M > 128 && N >= 256 && (int64_t)((M + 255) / 256) * ((N + 255) / 256) * T >= 40;
}

pt_status launch_wait_selftest(int* status, unsigned long long limit_ns, cudaStream_t st) {
    k_wait_selftest<<<1, 32, 0, st>>>(status, limit_ns);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("kernel launch failed: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return PT_OK;
}

bool gemm_pair_ok(int bn, int M, int N, int T) {
    // Two CTAs per 256 x 256 tile, so that a W tile enters each SM only by half: every launch of many rows, and
    // launches of more than one 128-row tile (a large decode batch) when they have enough tiles
    if (bn != 256 || N < 256 || !pair_launchable()) return false;
    return M >= 1024 || enough_pair_tiles(N, M, T);
}

int gemm_kps(int bn, int M, int K, int kt) {
    if (kt > 1 || K % BK || M > 256) return 1;
    int kps = std::max(1, 256 / bn);
    while (kps > 1 && ((K / BK) % kps || ring_stages(stage_a_bytes(M), bn * BK * 2, kps) < 3)) kps >>= 1;
    return kps;
}

pt_status make_w_map(CUtensorMap* out, const void* base, int64_t k, int64_t rows, int64_t tracks, int bn, int kps) {
    if (kps <= 1) return make_map_bf16(out, base, k, rows, tracks, bn);
    EncodeFn enc = get_encode();
    if (!enc) { set_error("cuTensorMapEncodeTiled is not available from this driver"); return PT_ERR_CUDA; }
    if (k % BK) { set_error("a W map of several k-blocks needs k %% 64 == 0"); return PT_ERR_INVALID_ARG; }
    cuuint64_t dims[4] = {(cuuint64_t)BK, (cuuint64_t)rows, (cuuint64_t)(k / BK), (cuuint64_t)tracks};
    cuuint64_t strides[3] = {(cuuint64_t)k * 2, (cuuint64_t)BK * 2, (cuuint64_t)k * 2 * (cuuint64_t)rows};
    cuuint32_t box[4] = {(cuuint32_t)BK, (cuuint32_t)std::min<int64_t>(bn, rows), (cuuint32_t)kps, 1};
    cuuint32_t es[4] = {1, 1, 1, 1};
    CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, es,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled (4-D W view) failed with code %d (k=%lld rows=%lld tracks=%lld kps=%d)", (int)r, (long long)k, (long long)rows, (long long)tracks, kps); return PT_ERR_CUDA; }
    return PT_OK;
}

pt_status make_a_map(CUtensorMap* out, const void* base, int64_t k, int64_t rows, int64_t tracks, int kps) {
    if (kps <= 1) return make_map_bf16(out, base, k, rows, tracks, BM);
    EncodeFn enc = get_encode();
    if (!enc) { set_error("cuTensorMapEncodeTiled is not available from this driver"); return PT_ERR_CUDA; }
    if (k % BK) { set_error("an A map of several k-blocks needs k %% 64 == 0"); return PT_ERR_INVALID_ARG; }
    // the box is a whole number of 8-row swizzle atoms, so that every k-block of the copy starts one; rows past
    // the tensor's end are filled with zeros by the copy
    const int box_rows = stage_a_bytes((int)std::min<int64_t>(rows, BM)) / (BK * 2);
    cuuint64_t dims[4] = {(cuuint64_t)BK, (cuuint64_t)rows, (cuuint64_t)(k / BK), (cuuint64_t)tracks};
    cuuint64_t strides[3] = {(cuuint64_t)k * 2, (cuuint64_t)BK * 2, (cuuint64_t)k * 2 * (cuuint64_t)rows};
    cuuint32_t box[4] = {(cuuint32_t)BK, (cuuint32_t)box_rows, (cuuint32_t)kps, 1};
    cuuint32_t es[4] = {1, 1, 1, 1};
    CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, es,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled (4-D A view) failed with code %d (k=%lld rows=%lld tracks=%lld kps=%d)", (int)r, (long long)k, (long long)rows, (long long)tracks, kps); return PT_ERR_CUDA; }
    return PT_OK;
}

int gemm_bn(int N, int M, int T, int epi) {
    // Tile width by a round model: a launch runs ceil(tiles / SMs) rounds and a round costs about
    // bn + min(M, 128) (bytes of B and A streamed per k-block when M is small, and near enough the MMA
    // and A-reload cost when it is large).  Ties go to the wider tile.  The QKV epilogue needs whole
    // heads (rotary partners) in a tile, so it never goes below 128.
    if (M <= 512 && enough_pair_tiles(N, M, T) && pair_launchable()) return 256;      // CTA pairs: see gemm_pair_ok
    const int widths[3] = {256, 128, 64};
    const int tiles_m = (M + BM - 1) / BM;
    int best_bn = 128;
    int64_t best = -1;
    for (int i = 0; i < 3; ++i) {
        const int bn = widths[i];
        if (bn == 64 && epi == EPI_QKV) continue;
        const int64_t tiles = (int64_t)tiles_m * ((N + bn - 1) / bn) * T;
        const int64_t cost = ((tiles + 147) / 148) * (bn + std::min(M, BM));
        if (best < 0 || cost < best) { best = cost; best_bn = bn; }
    }
    return best_bn;
}

pt_status launch_gemm(int epi, int bn, const CUtensorMap& ta, const CUtensorMap& tb, GemmP p, cudaStream_t st) {
    static int sms_[kMaxDevices] = {};
    const int dev = current_device();
    int& sms = sms_[dev];
    if (!sms) {
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (sms <= 0) sms = 148;
    }
    const int box_b = std::min(bn, p.N);
    p.a_tx = p.kps > 1 ? (uint32_t)p.kps * (uint32_t)stage_a_bytes(p.M) : (uint32_t)std::min(BM, p.M) * BK * 2;
    p.w_kb_bytes = (uint32_t)box_b * BK * 2;
    p.w_tx = (uint32_t)std::max(p.kps, 1) * p.w_kb_bytes;
    if (p.pair) {          // tb holds 128-row boxes of W; see gemm_pair_ok
        if (bn != 256) { set_error("the CTA-pair GEMM has 256-column tiles"); return PT_ERR_INVALID_ARG; }
        switch (epi) {
        case EPI_PLAIN: return launch_pair_t<EPI_PLAIN>(ta, tb, p, st, sms);
        case EPI_QKV: return launch_pair_t<EPI_QKV>(ta, tb, p, st, sms);
        case EPI_SWIGLU: return launch_pair_t<EPI_SWIGLU>(ta, tb, p, st, sms);
        default: return resid_by_tma(p) ? launch_pair_resid(ta, tb, p, st, sms) : launch_pair_t<EPI_RESID>(ta, tb, p, st, sms);
        }
    }
#define CASE(BN_, E_) if (bn == BN_ && epi == E_) return launch_t<BN_, E_>(ta, tb, p, st, sms)
    CASE(64, EPI_PLAIN); CASE(64, EPI_SWIGLU); CASE(64, EPI_RESID);
    CASE(128, EPI_PLAIN); CASE(128, EPI_QKV); CASE(128, EPI_SWIGLU); CASE(128, EPI_RESID);
    CASE(256, EPI_PLAIN); CASE(256, EPI_QKV); CASE(256, EPI_SWIGLU); CASE(256, EPI_RESID);
#undef CASE
    set_error("no GEMM variant for bn=%d epi=%d", bn, epi);
    return PT_ERR_UNSUPPORTED;
}

}  // namespace pt
