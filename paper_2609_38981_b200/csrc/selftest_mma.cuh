// Self-test of the hardware premises the numerical contract rests on (the paper trusts the
// analogous facts about its tile operations, Sec. "Value-Aware Regional Analysis" and App. A,
// the dot rule): one CTA computes the same small product twice, with tcgen05.mma (operands
// from shared-memory descriptors, or weights from tensor memory) and with mma.sync.m16n8k16
// (ldmatrix fragments), both in chunks of 16 ascending from a zero accumulator, from the very
// same swizzled shared-memory tiles, and writes both results.  The caller compares bits.
//   mode 0 (the score form):  D[128][64] = A[128][64] . B[64][64]^T, both K-major
//   mode 1 (the value form):  D[128][64] = W[128][64] . V[64][64], W = bf16 weights held in
//                             tensor memory (tcgen05) / as A fragments (mma.sync), V MN-major
#pragma once
#include "ptx.cuh"
#include "tcgen05.cuh"
#include "tile_math.cuh"

namespace vosti {

__global__ void __launch_bounds__(128, 1)
mma_selftest_kernel(const __nv_bfloat16* __restrict__ a, const __nv_bfloat16* __restrict__ b, int mode,
                    float* __restrict__ d_tc, float* __restrict__ d_warp, uint32_t* status) {
  constexpr int M = 128, N = 64, K = 64;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* sp = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sa = base, sb = base + M * 128, bar = base + M * 128 + N * 128, slot = bar + 8;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // both operands as [row][128 B] tiles with the 128-byte swizzle (chunk c of row r at c ^ (r % 8))
  for (int i = tid; i < M * 8; i += 128) {
    const int r = i >> 3, c = i & 7;
    *reinterpret_cast<uint4*>(sp + r * 128 + ((c ^ (r & 7)) << 4)) = *reinterpret_cast<const uint4*>(a + r * K + c * 8);
  }
  for (int i = tid; i < N * 8; i += 128) {
    const int r = i >> 3, c = i & 7;
    *reinterpret_cast<uint4*>(sp + M * 128 + r * 128 + ((c ^ (r & 7)) << 4)) =
        *reinterpret_cast<const uint4*>(b + r * K + c * 8);
  }
  if (tid == 0) {
    mbar_init(bar, 1);
    mbar_fence_init();
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot), "r"(128));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(sp + M * 128 + N * 128 + 8);
  const uint32_t lane_sel = static_cast<uint32_t>(warp * 32) << 16;

  // ---- warp MMA: rows 32 warp .. 32 warp + 31 as two 16-row groups ----------------------------
  const int quad = lane & 3, lm_mat = lane >> 3, lm_row = lane & 7;
  for (int g = 0; g < 2; ++g) {
    const int r0 = warp * 32 + g * 16;
    uint32_t fa[4][4];  // A fragments of the group: K chunks of 16
    const __nv_bfloat16* ra = a + (r0 + (lane >> 2)) * K;
    const __nv_bfloat16* rb = ra + 8 * K;
#pragma unroll
    for (int kc = 0; kc < 4; ++kc) {
      fa[kc][0] = *reinterpret_cast<const uint32_t*>(ra + 16 * kc + 2 * quad);
      fa[kc][1] = *reinterpret_cast<const uint32_t*>(rb + 16 * kc + 2 * quad);
      fa[kc][2] = *reinterpret_cast<const uint32_t*>(ra + 16 * kc + 8 + 2 * quad);
      fa[kc][3] = *reinterpret_cast<const uint32_t*>(rb + 16 * kc + 8 + 2 * quad);
    }
    float acc[8][4];
#pragma unroll
    for (int n = 0; n < 8; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
    if (mode == 0) {
#pragma unroll
      for (int cp = 0; cp < 2; ++cp)
#pragma unroll
        for (int n = 0; n < 8; ++n) {
          uint32_t b0, b1, b2, b3;
          ldsm_x4(stage_addr<64, 64, false>(sb, n * 8 + lm_row, 4 * cp + lm_mat), b0, b1, b2, b3);
          mma_bf16_16816(acc[n], fa[2 * cp], b0, b1);
          mma_bf16_16816(acc[n], fa[2 * cp + 1], b2, b3);
        }
    } else {
#pragma unroll
      for (int kk = 0; kk < 4; ++kk)
#pragma unroll
        for (int e = 0; e < 8; e += 2) {
          uint32_t b0, b1, b2, b3;
          ldsm_x4_trans(stage_addr<64, 64, false>(sb, kk * 16 + (lm_mat & 1) * 8 + lm_row, e + (lm_mat >> 1)), b0, b1, b2, b3);
          mma_bf16_16816(acc[e], fa[kk], b0, b1);
          mma_bf16_16816(acc[e + 1], fa[kk], b2, b3);
        }
    }
#pragma unroll
    for (int n = 0; n < 8; ++n) {
      float* o = d_warp + (r0 + (lane >> 2)) * N + n * 8 + 2 * quad;
      o[0] = acc[n][0];
      o[1] = acc[n][1];
      o[8 * N] = acc[n][2];
      o[8 * N + 1] = acc[n][3];
    }
  }

  // ---- tcgen05: the same product, accumulator in tensor-memory columns 0..63 -------------------
  if (mode == 1) {  // weights to tensor memory columns 64..95 (32 columns of packed bf16 pairs per row)
    uint32_t pk[32];
    const uint32_t* row = reinterpret_cast<const uint32_t*>(a + tid * K);
#pragma unroll
    for (int i = 0; i < 32; ++i) pk[i] = row[i];
    tmem_st32(tmem + lane_sel + 64, pk);
    tmem_wait_st();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (tid == 0) {
    if (mode == 0) {
      constexpr uint32_t idesc = umma_idesc(128, 64, false);
      for (int kc = 0; kc < 4; ++kc)
        tc_mma_ss(tmem, smem_desc_sw128(sa + kc * 32, 16, 1024), smem_desc_sw128(sb + kc * 32, 16, 1024), idesc,
                  kc > 0 ? 1u : 0u);
    } else {
      constexpr uint32_t idesc = umma_idesc(128, 64, true);
      for (int kc = 0; kc < 4; ++kc)
        tc_mma_ts(tmem, tmem + 64 + kc * 8, smem_desc_sw128(sb + kc * 2048, 64 * 128, 1024), idesc, kc > 0 ? 1u : 0u);
    }
    tc_commit(bar);
  }
  const bool ok = __all_sync(kFullMask, mbar_wait_bounded(bar, 0, 100000000ull));
  if (ok) {
    tc_fence_after();
    uint32_t lo32[32], hi32[32];
    tmem_ld32(tmem + lane_sel, lo32);
    tmem_ld32(tmem + lane_sel + 32, hi32);
    tmem_wait_ld();
    float* o = d_tc + tid * N;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      o[i] = __uint_as_float(lo32[i]);
      o[32 + i] = __uint_as_float(hi32[i]);
    }
  } else if (lane == 0) {
    atomicOr(status, 1u);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(128));
}

}  // namespace vosti
