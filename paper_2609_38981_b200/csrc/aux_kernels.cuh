// Cross-split combine and KV append kernels.
#pragma once
#include "meta.cuh"
#include "nc_math.cuh"
#include "ptx.cuh"

namespace vosti {

// Cross-split combine for split-parallel rows: one warp per (token, query
// head) folds the partials of splits 0..floor(p / L_S) left to right, then
// normalises.  Order depends on the split index only.
template <int D>
__global__ void __launch_bounds__(128) combine_kernel(const AttnParams P) {
  constexpr int V = D / 32;   // floats per lane
  constexpr int BATCH = 8;    // partial rows of a batch; two batches of loads are in flight
  const int lane = threadIdx.x & 31;
  const int widx = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (P.counts != nullptr) griddep_wait();  // device-planned: the metadata too comes from the stream
  if (widx >= (P.counts != nullptr ? P.counts[1] : P.n_split_tokens) * P.Hq) return;
  // Metadata does not depend on the kernel before this one: read it first, so that
  // only the partial rows themselves wait for the attention kernel to finish.
  const int2 rt = P.split_tokens[widx / P.Hq];
  const int head = widx % P.Hq;
  const ReqMeta rq = P.reqs[rt.x];
  const int kvh = head / P.G;
  const int row = rt.y * P.G + head % P.G;
  const int rows = rq.q_len * P.G;
  const int p = rq.start + rt.y;
  // the row's splits: from the one holding its first visible key to the one holding p;
  // partial slabs of the request are indexed from the request's first split
  const int k_lo = nc::first_key(p, P.window) / nc::kSplitLen;
  const int n_splits = p / nc::kSplitLen - k_lo + 1;
  const int64_t slab0 =
      rq.part_base + (static_cast<int64_t>(kvh) * rq.n_splits + (k_lo - rq.first_split)) * rows + row;
  griddep_wait();  // partials come from the kernel before this one in the stream

  auto load_u = [&](int64_t slab, float (&u)[V]) {
    const float* src = P.ws_u + slab * D + lane * V;
    if constexpr (V == 4) {
      const float4 x = *reinterpret_cast<const float4*>(src);
      u[0] = x.x; u[1] = x.y; u[2] = x.z; u[3] = x.w;
    } else {
      const float2 x = *reinterpret_cast<const float2*>(src);
      u[0] = x.x; u[1] = x.y;
    }
  };
  float uc[V];
  float mc = 0.f, zc = 0.f;
  // Two batches of partial rows: the loads of the next one are in flight while this one is folded.
  float uk[BATCH][V], un[BATCH][V];
  float2 mz[BATCH], mzn[BATCH];
  auto load_batch = [&](int k0, float (&u)[BATCH][V], float2 (&m2)[BATCH]) {
#pragma unroll
    for (int j = 0; j < BATCH; ++j)
      if (k0 + j < n_splits) {
        const int64_t slab = slab0 + static_cast<int64_t>(k0 + j) * rows;
        m2[j] = P.ws_mz[slab];
        load_u(slab, u[j]);
      }
  };
  load_batch(0, un, mzn);
  for (int k0 = 0; k0 < n_splits; k0 += BATCH) {
#pragma unroll
    for (int j = 0; j < BATCH; ++j) {
      mz[j] = mzn[j];
#pragma unroll
      for (int i = 0; i < V; ++i) uk[j][i] = un[j][i];
    }
    if (k0 + BATCH < n_splits) load_batch(k0 + BATCH, un, mzn);
#pragma unroll
    for (int j = 0; j < BATCH; ++j)
      if (k0 + j < n_splits) {
        if (k0 + j == 0) {  // folding starts from the first partial as it is
          mc = mz[0].x;
          zc = mz[0].y;
#pragma unroll
          for (int i = 0; i < V; ++i) uc[i] = uk[0][i];
        } else {
          const nc::FoldFactors f = nc::fold_scalars(mc, zc, mz[j].x, mz[j].y);
#pragma unroll
          for (int i = 0; i < V; ++i) uc[i] = nc::fold_u(uc[i], uk[j][i], f);
        }
      }
  }
  const float inv = nc::out_scale(zc);
  if (P.lse != nullptr && lane == 0) P.lse[static_cast<size_t>(rq.q_row0 + rt.y) * P.Hq + head] = nc::lse_value(mc, zc);
  __nv_bfloat16* dst = P.out + (static_cast<size_t>(rq.q_row0 + rt.y) * P.Hq + head) * D + lane * V;
#pragma unroll
  for (int i = 0; i < V; i += 2)
    *reinterpret_cast<__nv_bfloat162*>(dst + i) =
        __floats2bfloat162_rn(nc::out_value(uc[i], inv), nc::out_value(uc[i + 1], inv));
}

// KV append: one warp per (token, KV head); lanes 0-15 copy the K row, lanes
// 16-31 the V row, 16 bytes (D = 128) or 8 bytes (D = 64) each.
template <int D>
__global__ void __launch_bounds__(128) kv_append_kernel(const AppendParams P) {
  const int lane = threadIdx.x & 31;
  const int widx = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (widx >= P.n_tokens * P.Hkv) return;
  const int tok = widx / P.Hkv, kvh = widx % P.Hkv;
  const int slot = P.slot ? P.slot[tok] : P.inline_slot[tok];
  griddep_wait();  // earlier kernels in the stream may still be reading the pool
  const int page = slot / nc::kPageSize, within = slot % nc::kPageSize;
  const int is_v = lane >> 4, part = lane & 15;
  const __nv_bfloat16* src = (is_v ? P.v_new : P.k_new) + (static_cast<size_t>(tok) * P.Hkv + kvh) * D;
  __nv_bfloat16* dst = P.pool +
      ((static_cast<size_t>(page) * P.Hkv + kvh) * 2 + is_v) * (nc::kPageSize * D) +
      static_cast<size_t>(within) * D;
  if constexpr (D == 128) {
    reinterpret_cast<uint4*>(dst)[part] = reinterpret_cast<const uint4*>(src)[part];
  } else {
    reinterpret_cast<uint2*>(dst)[part] = reinterpret_cast<const uint2*>(src)[part];
  }
}

// Failure-detection self-test: one warp waits on a barrier that nothing will ever
// complete, with the same bounded wait the attention kernels use, gives up after
// `limit_ns`, records the failure in the status word and returns normally.
static __global__ void bounded_wait_selftest_kernel(uint32_t* status, uint64_t limit_ns) {
  __shared__ uint64_t bar;
  const uint32_t b = smem_u32(&bar);
  if (threadIdx.x == 0) {
    mbar_init(b, 1);
    mbar_fence_init();
  }
  __syncwarp();
  const bool ok = __all_sync(0xffffffffu, mbar_wait_bounded(b, 0, limit_ns));
  if (!ok && threadIdx.x == 0) atomicOr(status, 1u);
}

}  // namespace vosti
