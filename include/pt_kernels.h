/*
 * pt_kernels.h - kernel-level entry points of libpt.so, for unit parity tests and for timing a
 * single kernel of the PT forward pass in isolation.  Same conventions as pt.h: pt_status
 * returns, caller-owned device buffers, asynchronous on `stream`.
 */
#ifndef PT_KERNELS_H_
#define PT_KERNELS_H_

#include "pt.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Track-grouped GEMM, the contraction behind every projection of a track layer (the
 * "standard transformer layers" of Section 2.2, one set of weights per track):
 *   c[t][m][n] = sum_k a[t][m][k] * w[t][n][k]      t < T, m < M, n < N
 *   a  device bf16 [T][M][K] row-major        w  device bf16 [T][N][K] row-major
 *   c  device fp32 [T][M][N]                  status  device int32[16], zeroed by the caller
 * K must be a multiple of 8 and >= 64, N a multiple of 16; bn (N-tile width) is 128 or 256, 0 lets
 * the library choose.  With fold_tracks != 0 the K loop runs over (track, k) and a single
 * c[0][m][n] = sum_t sum_k ... is produced: the contraction of the track-sync (Algorithm 1,
 * h = all-reduce(h_1..h_n)) fused into the last GEMM of a track block. */
pt_status pt_kernel_gemm_bf16(const void* a, const void* w, void* c, int32_t T, int32_t M, int32_t N,
                              int32_t K, int32_t bn, int32_t fold_tracks, void* status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* PT_KERNELS_H_ */
