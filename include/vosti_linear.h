/* vosti_linear.h -- batch-invariant linear layer and RMS normalisation for
 * B200 (sm_100a), the two operators that surround attention in a decoder layer.
 *
 * Contract (Sec. "Relational Kernel Contracts", matmul): for activations x
 * [M, K] (one token per row), fixed weights and an output row x_i W^T, the
 * bits of that row are the same whether x_i runs alone (M = 1) or anywhere in
 * a batch of any size; the other rows are unconstrained.  It holds because
 * (Sec. "Relational Structural Analysis") the tile shape is a function of
 * (N, K) only, never of M; the K range is cut into segments that depend on
 * (N, K) only, every segment sum starts from a zero fp32 accumulator and takes
 * its products in ascending order (chunks of 16, tcgen05.mma), and the segment
 * sums are added left to right in fp32; and a row of an MMA tile depends on its
 * own operand row only.  Whether a pair of CTAs computes 256 x 256 tiles with
 * two-SM MMA instructions (large batches), one CTA walks all segments of a
 * 128-row tile, or the segments of a tile are spread over CTAs and added by a
 * second kernel (one row tile, so that every SM streams a slice of the weight)
 * is a scheduling decision that may depend on M: all compute the same sums in
 * the same order.  The tile shape reported by vosti_linear_tile_shape is the
 * unit of that arithmetic (one CTA's rows, one instruction's columns and K
 * block); a pair kernel works on two such row tiles at a time.
 *
 * All tensors are bf16, row-major, in device memory, 16-byte aligned; fp32
 * accumulation; round-to-nearest-even to bf16 at the end.  Kernels are
 * enqueued on `cuda_stream`; nothing is allocated.  Every device-side wait is
 * bounded: a kernel that gives up sets a status word read by
 * vosti_linear_poll_status.
 */
#ifndef VOSTI_LINEAR_H_
#define VOSTI_LINEAR_H_

#include <stdint.h>

#include "vosti.h"

#ifdef __cplusplus
extern "C" {
#endif

/* The tile shape used for an (N, K) weight: a pure host-side function of N and
 * K (B_M = 128, B_K = 64, B_N = 256 when N is a multiple of 256, else 128).
 * UNSUPPORTED_CONFIG unless N is a positive multiple of 128 and K of 64. */
vosti_status vosti_linear_tile_shape(int64_t N, int64_t K, int32_t* b_m, int32_t* b_n, int32_t* b_k);

/* The number of K segments of an (N, K) weight, a pure host-side function of N
 * and K: floor(148 / column tiles), at most K / 1024 and at least 1; segment j
 * covers the 64-wide blocks [j B / n, (j + 1) B / n) of the B = K / 64 blocks. */
vosti_status vosti_linear_segments(int64_t N, int64_t K, int32_t* n_segments);

/* Bytes of device workspace that let vosti_linear spread the K segments of a
 * tile over CTAs when M is small (one fp32 [M, N] slab per segment); 0 for an
 * unsupported shape. */
size_t vosti_linear_workspace_bytes(int64_t M, int64_t N, int64_t K);

/* y [M, N] = x [M, K] * w [N, K]^T (one weight row per output feature, as a
 * linear layer stores it).  M >= 0 is free; M = 0 does nothing.
 * workspace: device memory, 16-byte aligned, or NULL.  With at least
 * vosti_linear_workspace_bytes(M, N, K) bytes the call may spread the K
 * segments of a tile over CTAs also where a tile has more than eight segments
 * (see vosti_linear_ex).  The output bits are the same whichever schedule runs.
 * Errors: INVALID_ARG (null or misaligned pointers, negative M),
 * UNSUPPORTED_CONFIG (see vosti_linear_tile_shape), CUDA. */
vosti_status vosti_linear(const void* x, const void* w, void* y, int64_t M, int64_t N, int64_t K,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The same with the schedule named by the caller (tests compare them bit for
 * bit; measurements).  vosti_linear picks one by itself, VOSTI_LINEAR_AUTO:
 * with few row tiles the K segments of a tile are spread over CTAs -- in
 * clusters that add the segment sums out of each other's shared memory when a
 * tile has two to eight segments (by name: up to sixteen, clusters beyond the
 * portable size), else through the workspace if one is given;
 * with many row tiles CTA pairs (B_N = 256, large M) or single CTAs walk whole
 * tiles.  A schedule that does not apply to the shape (SPLIT_CLUSTER with one
 * or more than sixteen segments, SPLIT_WORKSPACE with one segment or without the
 * workspace, PAIRS with B_N = 128) returns UNSUPPORTED_CONFIG. */
enum {
  VOSTI_LINEAR_AUTO = 0,
  VOSTI_LINEAR_WHOLE_TILES = 1,
  VOSTI_LINEAR_SPLIT_WORKSPACE = 2,
  VOSTI_LINEAR_SPLIT_CLUSTER = 3,
  VOSTI_LINEAR_PAIRS = 4
};
vosti_status vosti_linear_ex(const void* x, const void* w, void* y, int64_t M, int64_t N, int64_t K,
                             void* workspace, size_t workspace_bytes, int32_t schedule, void* cuda_stream);

/* y [M, K] = x * rsqrt(mean_k(x^2) + eps) * weight [K], per row: the sum of
 * squares is taken in a fixed order that depends on K only (each lane of the
 * row's warp adds its 16-byte vectors in ascending order, lanes are combined by
 * a butterfly), so a row's bits do not depend on M or on the row's place.
 * K must be a multiple of 8.  y may alias x. */
vosti_status vosti_rmsnorm(const void* x, const void* weight, void* y, int64_t M, int64_t K, float eps,
                           void* cuda_stream);

/* Hash of everything that decides the bits of vosti_linear and vosti_rmsnorm
 * (Sec. "A System-Level Formulation": the deployment configuration): the
 * version, the tile sizes, the segment rule's two constants -- the wave of 148
 * units is a frozen number, not the SM count of the device in use -- and one
 * id per reduction rule.  vosti_linear_contract returns those words (their
 * number; writes min(number, cap)).  Host-only. */
uint64_t vosti_linear_fingerprint(void);
int32_t vosti_linear_contract(uint32_t* words, int32_t cap);

/* Waits for `cuda_stream` and reports whether a linear kernel gave up on a
 * bounded wait since the last poll (VOSTI_ERR_TIMEOUT), clearing the word. */
vosti_status vosti_linear_poll_status(void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* VOSTI_LINEAR_H_ */
