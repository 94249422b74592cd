/* SmoothGEMM for sm_100a (Section 5): a fixed-tile tensor-core GEMM for the Linear operators
 * (QKV, OProj, GateUp, Down) whose token dimension M takes any value.
 *
 *     C[M, N] = A[M, K] * W[N, K]^T      bf16 inputs, fp32 accumulation, bf16 output
 *
 * The kernel always computes whole 128 x tile_n tiles (Section 5.1: computation on fixed shapes).
 * M is padded virtually: the tile loads read rows past M as zeros on chip (selective read; no
 * padded copy of A exists in global memory) and the epilogue stores only rows below M (selective
 * write).  N and K come from the model (Section 5.2) and need no padding beyond 8-element
 * alignment; a last partial tile in N or K is handled the same way (zeros in, clipped store).
 * Tiles are handed to the SMs with the M tiles of one N tile next to each other, so the SMs that
 * run at the same time share the weight tile through L2 (Section 5.3's task order).
 */
#ifndef XY_GEMM_H_
#define XY_GEMM_H_

#include <stdint.h>

#include "xy_attn.h"

#ifdef __cplusplus
extern "C" {
#endif

/* tile_n flag: compute 256 x tile_n tiles on pairs of CTAs (tcgen05 cta_group::2; tile_n 128 or 256). */
#define XY_GEMM_PAIR 0x1000

/* Asynchronous on `stream` (a cudaStream_t, may be 0); allocates nothing; no host sync.
 *   a  DEVICE bf16, row m at a + m*lda (elements), K contiguous; lda >= K
 *   w  DEVICE bf16, row n at w + n*ldw, K contiguous (the layout of a Linear weight); ldw >= K
 *   c  DEVICE bf16, row m at c + m*ldc, N contiguous; ldc >= N; written for m < M, n < N only
 *   M >= 0 (0: nothing to do), N >= 8, K >= 8; N, K, lda, ldw, ldc multiples of 8; the three base
 *   pointers 16-byte aligned
 *   tile_n  columns per tile: 32, 64, 128, 256 (128-row tiles on single CTAs), XY_GEMM_PAIR | 128
 *           or XY_GEMM_PAIR | 256 (256-row tiles on CTA pairs), or 0 to let the library choose:
 *           256 x 256 pair tiles when M > 128 pads to a multiple of 256 with at most 15 % waste
 *           and those tiles number at least a quarter of the SMs; else, for M <= 512 with few
 *           tiles, a split of K over a thread-block cluster (2..8 CTAs per 128 x 128 tile, partial
 *           sums added through distributed shared memory), which puts the idle SMs to work; else
 *           128 x 256 tiles when they give half of the SMs a tile, else 128 x 128
 * Returns XY_OK, XY_ERR_INVALID_ARG (null pointer, bad size or alignment), XY_ERR_UNSUPPORTED
 * (tile_n not one of the values above) or XY_ERR_CUDA.  Calls on one stream are ordered; the caller
 * owns all buffers. */
int xy_gemm_run(const void* a, int64_t lda, const void* w, int64_t ldw, void* c, int64_t ldc, int32_t M,
                int32_t N, int32_t K, int32_t tile_n, void* stream);

/* The same with DEVICE scratch memory, which lets the last, partial wave of tiles be split along K
 * over every SM when K is long (K >= 8192 and a last wave of at most 0.6 of the SMs; measured
 * rule): each SM multiplies a run of K chunks of one or two of those tiles and leaves fp32 partial
 * sums in the scratch; a second, small kernel on the same stream adds a tile's partial sums in a
 * fixed order (bit-reproducible) and stores the tile.  No thread waits for another CTA.
 *   workspace        DEVICE, 16-byte aligned, at least xy_gemm_workspace_bytes() bytes (a smaller
 *                    one, or NULL, gives xy_gemm_run's behaviour); contents do not matter.  Calls
 *                    that may run at the same time need scratch of their own.
 * Errors as xy_gemm_run. */
int xy_gemm_run_ws(const void* a, int64_t lda, const void* w, int64_t ldw, void* c, int64_t ldc, int32_t M,
                   int32_t N, int32_t K, int32_t tile_n, void* workspace, int64_t workspace_bytes, void* stream);

/* Bytes of scratch xy_gemm_run_ws can use on the current device (2 slots of a 128 x 256 fp32 tile
 * per SM: 38.8 MB with 148 SMs), or -1 if the device cannot be queried. */
int64_t xy_gemm_workspace_bytes(void);

/* Status of the device-side waits of the GEMM kernels on the current device since the last call of
 * this function: 0, or XY_ERR_DEVICE_TIMEOUT if a bounded wait inside a kernel gave up (the
 * kernel then returns early and its output is invalid).  Synchronises the device. */
int xy_gemm_device_status(int32_t* status /*HOST*/);

#ifdef __cplusplus
}
#endif
#endif /* XY_GEMM_H_ */
