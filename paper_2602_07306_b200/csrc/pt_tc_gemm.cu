// Track-grouped bf16 GEMM for sm_100a: C[t] = A[t] * W[t]^T with fp32 accumulation in tensor
// memory.  Persistent, warp-specialised: warp 0 feeds a ring of shared-memory stages with TMA
// (3-D tensor maps, coordinates (k, row, track), 128-byte swizzle), warp 1 issues tcgen05.mma
// (128 x BN x 16 per instruction) into one of two TMEM accumulators, warps 2-5 drain the other
// accumulator with tcgen05.ld and run the fused epilogue:
//   EPI_QKV     per-row 1/rms scale (RMSNorm), rotary embedding on q and k heads, q to a dense
//               buffer, k and v straight into the paged KV cache
//   EPI_SWIGLU  per-row 1/rms scale, silu(gate) * up on interleaved gate/up columns
//   EPI_RESID   residual add (optionally summed over all tracks = the track-sync of Algorithm 1,
//               with the K loop running over (track, k) so one accumulator collects every track),
//               fp32 stream out, gain-scaled bf16 copy for the next GEMM, partial sums of squares
//               for the next RMSNorm
//   EPI_PLAIN   fp32 C (kernel-level tests)
// Every mbarrier wait is bounded; on a timeout the CTA records PT_ERR_DEVICE_TIMEOUT, stops
// issuing work, frees its tensor memory and exits.
#include "pt_tc.h"

namespace pt {

namespace {

constexpr int BM = 128, BK = 64;
constexpr uint32_t kSpinLimit = 1u << 26;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false when the limit ran out or another warp already gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (mbar_try(bar, parity)) return true;
        if ((i & 1023) == 1023 && *abort_flag) return false;
    }
    return false;
}

__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1, int c2) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(smem_u32(dst)), "l"((uint64_t)map), "r"(c0), "r"(c1), "r"(c2), "r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
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

__device__ __forceinline__ void report(int* status, int code, int loc) {
    if (atomicCAS(status, 0, code) == 0) status[1] = loc;
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&v);
}
// 16 floats -> 16 bf16 (32 bytes, two 16-byte stores)
__device__ __forceinline__ void store16_bf16(__nv_bfloat16* dst, const float* v) {
    uint4 a, b;
    a.x = pack_bf16(v[0], v[1]); a.y = pack_bf16(v[2], v[3]); a.z = pack_bf16(v[4], v[5]); a.w = pack_bf16(v[6], v[7]);
    b.x = pack_bf16(v[8], v[9]); b.y = pack_bf16(v[10], v[11]); b.z = pack_bf16(v[12], v[13]); b.w = pack_bf16(v[14], v[15]);
    reinterpret_cast<uint4*>(dst)[0] = a;
    reinterpret_cast<uint4*>(dst)[1] = b;
}

template <int BN> struct Cfg {
    static constexpr int STAGES = BN == 256 ? 4 : 6;
    static constexpr int A_BYTES = BM * BK * 2;
    static constexpr int B_BYTES = BN * BK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int SMEM = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

template <int BN, int EPI>
__global__ void __launch_bounds__(192, 1)
gemm_tc(const __grid_constant__ CUtensorMap ta, const __grid_constant__ CUtensorMap tb, const GemmP p) {
    using C = Cfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t* full = (uint64_t*)(smem + C::STAGES * C::STAGE_BYTES);
    uint64_t* empty = full + C::STAGES;
    uint64_t* acc_full = empty + C::STAGES;
    uint64_t* acc_empty = acc_full + 2;
    uint32_t* tmem_slot = (uint32_t*)(acc_empty + 2);
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < C::STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], 4); }
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

    if (warp == 0) {
        if (lane == 0) {
            int s = 0; uint32_t ph = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                int nt = tile % p.tiles_n, mt = (tile / p.tiles_n) % p.tiles_m, t = tile / (p.tiles_n * p.tiles_m);
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(&empty[s], ph ^ 1, abort_flag)) { ok = false; report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_GEMM_EMPTY_WAIT); *abort_flag = 1; break; }
                    int tt = p.kt > 1 ? kb / kpb : t;
                    int k0 = (p.kt > 1 ? kb % kpb : kb) * BK;
                    uint8_t* sa = smem + s * C::STAGE_BYTES;
                    mbar_expect_tx(&full[s], p.tx_bytes);
                    tma_load_3d(sa, &ta, &full[s], k0, mt * BM, tt);
                    tma_load_3d(sa + C::A_BYTES, &tb, &full[s], k0, nt * BN, tt);
                    if (++s == C::STAGES) { s = 0; ph ^= 1; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
            int s = 0; uint32_t ph = 0;
            int a = 0; uint32_t aph = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                if (!mbar_wait(&acc_empty[a], aph ^ 1, abort_flag)) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_GEMM_ACC_WAIT); *abort_flag = 1; break; }
                tc_fence_after();
                uint32_t d_tmem = tmem_base + a * BN;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!mbar_wait(&full[s], ph, abort_flag)) { ok = false; report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_GEMM_TMA_WAIT); *abort_flag = 1; break; }
                    tc_fence_after();
                    uint32_t sa = smem_u32(smem + s * C::STAGE_BYTES);
                    uint64_t da = smem_desc(sa), db = smem_desc(sa + C::A_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        tc_mma(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
                    tc_commit(&empty[s]);                 // frees the stage when these MMAs retire
                    if (++s == C::STAGES) { s = 0; ph ^= 1; }
                }
                if (!ok) break;
                tc_commit(&acc_full[a]);                  // accumulator complete
                if (++a == 2) { a = 0; aph ^= 1; }
            }
        }
        __syncwarp();
    } else {
        const int ew = warp & 3;                           // TMEM lane quarter this warp may read
        int a = 0; uint32_t aph = 0;
        for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
            int nt = tile % p.tiles_n, mt = (tile / p.tiles_n) % p.tiles_m, t = tile / (p.tiles_n * p.tiles_m);
            bool ok = mbar_wait(&acc_full[a], aph, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) { if (lane == 0) { report(p.status, PT_ERR_DEVICE_TIMEOUT, LOC_GEMM_EPI_WAIT); *abort_flag = 1; } break; }
            tc_fence_after();
            const int row = mt * BM + ew * 32 + lane;
            const bool row_ok = row < p.M;
            const int n0 = nt * BN;
            const uint32_t taddr = tmem_base + ((uint32_t)(ew * 32) << 16) + a * BN;
            const size_t trow = (size_t)t * p.M + row;

            float rinv = 1.f;
            if ((EPI == EPI_QKV || EPI == EPI_SWIGLU) && row_ok) {
                const float* sp = p.ssq_in + (size_t)t * p.ssq_in_tstride + (size_t)row * p.ssq_tiles;
                float s = 0.f;
                for (int i = 0; i < p.ssq_tiles; ++i) s += sp[i];
                rinv = 1.0f / sqrtf(s / (float)p.K + p.eps);
            }

            if (EPI == EPI_PLAIN) {
                for (int c = 0; c < BN; c += 16) {
                    float v[16];
                    tc_ld16(taddr + c, v);
                    tc_wait_ld();
                    if (row_ok && n0 + c < p.N) {
                        float4* dst = (float4*)(p.c_out + trow * p.N + n0 + c);
#pragma unroll
                        for (int i = 0; i < 4; ++i) dst[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
                    }
                }
            } else if (EPI == EPI_QKV) {
                const int dh = p.dh, half = dh >> 1;
                int pos = 0; int64_t kvoff = 0;
                if (row_ok) { pos = p.row_pos[row]; kvoff = p.row_kvoff[row]; }
                bool slot_ok = row_ok && kvoff >= 0 && kvoff + (int64_t)(2 * p.nkv - 1) * p.ps * dh + dh <= p.slab_elems;
                if (row_ok && !slot_ok) report(p.status, PT_ERR_DEVICE_BOUNDS, LOC_ROPE_PAGE);
                const float* cs = p.cs + (size_t)pos * half;
                const float* sn = p.sn + (size_t)pos * half;
                for (int hc = 0; hc < BN; hc += dh) {
                    const int col = n0 + hc;
                    if (col >= p.N) break;                              // uniform across the CTA
                    const int hs = col / dh;                            // head slot: q heads, k heads, v heads
                    __nv_bfloat16* dst;
                    bool st_ok;
                    if (hs < p.nq) { dst = p.q_out + trow * (size_t)(p.nq * dh) + (size_t)hs * dh; st_ok = row_ok; }
                    else {
                        int kv = hs >= p.nq + p.nkv, head = hs - p.nq - kv * p.nkv;
                        dst = p.pool_l + (size_t)t * p.pool_tstride + kvoff + ((int64_t)kv * p.nkv + head) * p.ps * dh;
                        st_ok = slot_ok;
                    }
                    if (hs < p.nq + p.nkv) {
                        for (int j0 = 0; j0 < half; j0 += 16) {
                            float lo[16], hi[16];
                            tc_ld16(taddr + hc + j0, lo);
                            tc_ld16(taddr + hc + half + j0, hi);
                            tc_wait_ld();
                            if (st_ok) {
                                float c[16], s[16];
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    float4 cv = ((const float4*)(cs + j0))[i], sv = ((const float4*)(sn + j0))[i];
                                    c[4 * i] = cv.x; c[4 * i + 1] = cv.y; c[4 * i + 2] = cv.z; c[4 * i + 3] = cv.w;
                                    s[4 * i] = sv.x; s[4 * i + 1] = sv.y; s[4 * i + 2] = sv.z; s[4 * i + 3] = sv.w;
                                }
#pragma unroll
                                for (int i = 0; i < 16; ++i) {
                                    float l = lo[i] * rinv, h = hi[i] * rinv;
                                    lo[i] = l * c[i] - h * s[i];
                                    hi[i] = h * c[i] + l * s[i];
                                }
                                store16_bf16(dst + j0, lo);
                                store16_bf16(dst + half + j0, hi);
                            }
                        }
                    } else {
                        for (int j0 = 0; j0 < dh; j0 += 16) {
                            float v[16];
                            tc_ld16(taddr + hc + j0, v);
                            tc_wait_ld();
                            if (st_ok) {
#pragma unroll
                                for (int i = 0; i < 16; ++i) v[i] *= rinv;
                                store16_bf16(dst + j0, v);
                            }
                        }
                    }
                }
            } else if (EPI == EPI_SWIGLU) {
                for (int c = 0; c < BN; c += 32) {
                    if (n0 + c >= p.N) break;
                    float g[16], u[16];
                    tc_ld16(taddr + c, g);
                    tc_ld16(taddr + c + 16, u);
                    tc_wait_ld();
                    if (row_ok) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            float gv = g[i] * rinv, uv = u[i] * rinv;
                            g[i] = gv / (1.0f + __expf(-gv)) * uv;
                        }
                        store16_bf16(p.z_out + trow * (size_t)(p.N >> 1) + ((n0 + c) >> 1), g);
                    }
                }
            } else {  // EPI_RESID
                float ssq = 0.f;
                for (int c = 0; c < BN; c += 16) {
                    if (n0 + c >= p.N) break;
                    float v[16];
                    tc_ld16(taddr + c, v);
                    tc_wait_ld();
                    if (row_ok) {
                        const size_t eo = (size_t)row * p.N + n0 + c;
                        for (int tt = 0; tt < p.n_sum; ++tt) {
                            const float4* hp = (const float4*)(p.h_in + (size_t)(p.n_sum > 1 ? tt : t) * p.h_in_tstride + eo);
#pragma unroll
                            for (int i = 0; i < 4; ++i) { float4 h = hp[i]; v[4 * i] += h.x; v[4 * i + 1] += h.y; v[4 * i + 2] += h.z; v[4 * i + 3] += h.w; }
                        }
                        if (p.scale != 1.0f) {
#pragma unroll
                            for (int i = 0; i < 16; ++i) v[i] *= p.scale;
                        }
                        float4* ho = (float4*)(p.h_out + (size_t)t * p.h_out_tstride + eo);
#pragma unroll
                        for (int i = 0; i < 4; ++i) ho[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
#pragma unroll
                        for (int i = 0; i < 16; ++i) ssq += v[i] * v[i];
                        if (p.hb_out) {
                            for (int to = 0; to < p.n_out; ++to) {
                                const int tg = p.n_out > 1 ? to : t;
                                const float* gp = p.gain + (size_t)tg * p.N + n0 + c;
                                float w[16];
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    float4 g = ((const float4*)gp)[i];
                                    w[4 * i] = v[4 * i] * g.x; w[4 * i + 1] = v[4 * i + 1] * g.y; w[4 * i + 2] = v[4 * i + 2] * g.z; w[4 * i + 3] = v[4 * i + 3] * g.w;
                                }
                                store16_bf16(p.hb_out + ((size_t)tg * p.M + row) * p.N + n0 + c, w);
                            }
                        }
                    }
                    if (((c + 16) % kSsqTile) == 0 || n0 + c + 16 >= p.N) {
                        if (row_ok && p.ssq_out)
                            p.ssq_out[(size_t)t * p.ssq_out_tstride + (size_t)row * p.ssq_out_tiles + (n0 + c) / kSsqTile] = ssq;
                        ssq = 0.f;
                    }
                }
            }
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

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

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

template <int BN, int EPI>
pt_status launch_t(const CUtensorMap& ta, const CUtensorMap& tb, GemmP p, cudaStream_t st, int sms) {
    using C = Cfg<BN>;
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(gemm_tc<BN, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
        if (e != cudaSuccess) { set_error("cudaFuncSetAttribute: %s", cudaGetErrorString(e)); return PT_ERR_CUDA; }
        attr_done = true;
    }
    p.tiles_m = (p.M + BM - 1) / BM;
    p.tiles_n = (p.N + BN - 1) / BN;
    int tiles = p.tiles_m * p.tiles_n * p.T;
    int grid = std::min(tiles, sms);
    gemm_tc<BN, EPI><<<grid, 192, C::SMEM, st>>>(ta, tb, p);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return PT_OK;
}

}  // namespace

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

int gemm_bn(int N, int M, int T) {
    // wide tiles when there are enough of them to fill the machine
    if (N % 256 == 0 && (int64_t)((M + BM - 1) / BM) * (N / 256) * T >= 148) return 256;
    return 128;
}

pt_status launch_gemm(int epi, int bn, const CUtensorMap& ta, const CUtensorMap& tb, GemmP p, cudaStream_t st) {
    static int sms = 0;
    if (!sms) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (sms <= 0) sms = 148;
    }
    int box_a = std::min(BM, p.M), box_b = std::min(bn, p.kt > 1 ? p.N : p.N);
    p.tx_bytes = (uint32_t)(box_a + box_b) * BK * 2;
#define CASE(BN_, E_) if (bn == BN_ && epi == E_) return launch_t<BN_, E_>(ta, tb, p, st, sms)
    CASE(128, EPI_PLAIN); CASE(128, EPI_QKV); CASE(128, EPI_SWIGLU); CASE(128, EPI_RESID);
    CASE(256, EPI_PLAIN); CASE(256, EPI_QKV); CASE(256, EPI_SWIGLU); CASE(256, EPI_RESID);
#undef CASE
    set_error("no GEMM variant for bn=%d epi=%d", bn, epi);
    return PT_ERR_UNSUPPORTED;
}

}  // namespace pt
