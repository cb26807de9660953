// Sequential attention (long queries: prefill chunks): one warp per (16-row
// group, KV head) walks ALL key tiles of its rows in ascending order and, at
// every split boundary, folds the finished split into a running result with
// the same fold the combine kernel applies to stored partials -- so a row
// computed here has the bits it would have on the split-parallel path.
// Warps are independent workers with private TMA-fed stage rings.
#pragma once
#include "attn_split.cuh"

namespace vosti {

template <int D>
struct SeqKernelCfg {
  static constexpr int kWarps = 4;
  static constexpr int kStages = (D == 128) ? 3 : 6;  // per warp, one whole K or V tile each
  static constexpr int kSmemBytes =
      kWarps * kStages * TileCfg<D, nc::kKeyTile>::kStageBytes + kWarps * kStages * 8 + 1024;
};

template <int D>
__global__ void __launch_bounds__(SeqKernelCfg<D>::kWarps * 32, 1)
attn_seq_kernel(const __grid_constant__ CUtensorMap kv_map, const AttnParams P) {
  constexpr int SK = nc::kKeyTile;
  using C = TileCfg<D, SK>;
  constexpr int kWarpsPerCta = SeqKernelCfg<D>::kWarps;
  constexpr int R = SeqKernelCfg<D>::kStages;
  constexpr int TPS = nc::kTilesPerSplit;

  extern __shared__ uint8_t smem_raw[];
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int quad = lane & 3;
  const int worker = blockIdx.x * kWarpsPerCta + warp;
  if (worker >= P.n_workers) return;  // warps never synchronise with one another

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t stage0 = base + warp * R * C::kStageBytes;
  const uint32_t bar0 = base + kWarpsPerCta * R * C::kStageBytes + warp * R * 8;
  if (lane == 0) {
    tma_prefetch_desc(&kv_map);
#pragma unroll
    for (int s = 0; s < R; ++s) mbar_init(bar0 + s * 8, 1);
    mbar_fence_init();
    fence_proxy_async();
  }
  __syncwarp();

  const vosti_work_item item = P.items[worker / P.Hkv];
  const int kvh = worker % P.Hkv;
  const ReqMeta rq = P.reqs[item.req];
  const int G = P.G;
  const float c = P.c;

  const int row_a = item.row_group * nc::kRowsPerGroup + (lane >> 2);
  const int row_b = row_a + 8;
  const int tok_a = row_a / G, tok_b = row_b / G;
  const bool valid_a = tok_a < rq.q_len, valid_b = tok_b < rq.q_len;
  RowPair r;
  r.p_a = valid_a ? rq.start + tok_a : -1;  // padding rows see nothing
  r.p_b = valid_b ? rq.start + tok_b : -1;
  r.reset();
  const int head_a = kvh * G + row_a % G, head_b = kvh * G + row_b % G;
  const int last_tok = min(rq.q_len - 1, (item.row_group * nc::kRowsPerGroup + 15) / G);
  const int p_max = rq.start + last_tok;
  const int n_eff = rq.start + rq.q_len;  // slots at or beyond this hold nothing we may read
  const int p_min = rq.start + (item.row_group * nc::kRowsPerGroup) / G;
  const bool upper_rows = (item.row_group * nc::kRowsPerGroup + 8) / G < rq.q_len;

  const int t_begin = item.split_begin * TPS;
  const int t_end = min(item.split_end * TPS, p_max / nc::kKeyTile + 1);
  const int n_loads = 2 * (t_end - t_begin);

  uint32_t qa[C::KC][4];
  load_q_frags<D>(qa, P.q + (static_cast<size_t>(rq.q_row0 + tok_a) * P.Hq + head_a) * D,
                  P.q + (static_cast<size_t>(rq.q_row0 + tok_b) * P.Hq + head_b) * D, valid_a, valid_b,
                  quad);

  // Page ids of the split being loaded: lane l holds the id of page 32*split + l.
  const int32_t* bt = P.bt_flat + rq.bt_off;
  auto fetch_pages = [&](int split) -> int {
    const int pg = split * nc::kPagesPerSplit + lane;
    return pg < rq.n_pages ? __ldg(bt + pg) : -1;
  };
  int pages_even = -1, pages_odd = -1;
  {
    const int ids = fetch_pages(item.split_begin);
    if (item.split_begin & 1) pages_odd = ids; else pages_even = ids;
  }
  // Issue load i of the item: tile t_begin + i/2, K if i is even, V if odd.
  auto issue = [&](int i) {
    const int t = t_begin + (i >> 1);
    const int split = t / TPS;
    const int tl = t - split * TPS;
    if (!(i & 1) && tl == TPS / 2 && split + 1 < item.split_end) {
      const int ids = fetch_pages(split + 1);  // needed four tiles from now
      if ((split + 1) & 1) pages_odd = ids; else pages_even = ids;
    }
    const int stage = i % R;
    issue_stage_load<D, SK>(&kv_map, stage0 + stage * C::kStageBytes, bar0 + stage * 8,
                       (split & 1) ? pages_odd : pages_even, tl * nc::kPagesPerTile,
                       min(nc::kPagesPerTile, rq.n_pages - t * nc::kPagesPerTile), P.Hkv, kvh, i & 1, lane);
  };
#pragma unroll 1
  for (int i = 0; i < R && i < n_loads; ++i) issue(i);

  float u[C::NE][4], uc[C::NE][4];
#pragma unroll
  for (int e = 0; e < C::NE; ++e) u[e][0] = u[e][1] = u[e][2] = u[e][3] = 0.f;
  float mc_a = 0.f, mc_b = 0.f, zc_a = 0.f, zc_b = 0.f;
  bool timed_out = false;

#pragma unroll 1
  for (int t = t_begin; t < t_end; ++t) {
    const int li = 2 * (t - t_begin);
    const int key0 = t * nc::kKeyTile;
    float s[8][4];
    {
      const int stage = li % R;
      if (!__all_sync(kFullMask, mbar_wait_bounded(bar0 + stage * 8, (li / R) & 1))) {
        timed_out = true;  // warp-uniform: every lane leaves together
        break;
      }
      tile_scores<D, SK>(stage0 + stage * C::kStageBytes, qa, s, 0, lane);
    }
    __syncwarp();
    if (li + R < n_loads) issue(li + R);
    uint32_t pa[4][4];
    tile_softmax_dispatch<D>(s, key0, c, r, u, pa, quad, key0 + nc::kKeyTile - 1 <= p_min, upper_rows);
    {
      const int stage = (li + 1) % R;
      if (!__all_sync(kFullMask, mbar_wait_bounded(bar0 + stage * 8, ((li + 1) / R) & 1))) {
        timed_out = true;
        break;
      }
      const uint32_t vs = stage0 + stage * C::kStageBytes;
      if (key0 + nc::kKeyTile > n_eff) zero_value_tail<D, SK>(vs, n_eff - key0, lane);
      tile_pv<D, SK>(vs, pa, u, 0, lane);
    }
    __syncwarp();
    if (li + 1 + R < n_loads) issue(li + 1 + R);

    // ---- end of a split: fold it into the running result ---------------------
    if ((t + 1) % TPS == 0 || t + 1 == t_end) {
      const int split = t / TPS;
      if (split == 0) {
#pragma unroll
        for (int e = 0; e < C::NE; ++e) {
          uc[e][0] = u[e][0]; uc[e][1] = u[e][1]; uc[e][2] = u[e][2]; uc[e][3] = u[e][3];
        }
        mc_a = r.m_a; mc_b = r.m_b; zc_a = r.z_a; zc_b = r.z_b;
      } else {
        if (r.p_a >= split * nc::kSplitLen) {  // rows that see nothing of the split keep their state
          const nc::FoldFactors f = nc::fold_scalars(mc_a, zc_a, r.m_a, r.z_a);
#pragma unroll
          for (int e = 0; e < C::NE; ++e) {
            uc[e][0] = nc::fold_u(uc[e][0], u[e][0], f);
            uc[e][1] = nc::fold_u(uc[e][1], u[e][1], f);
          }
        }
        if (r.p_b >= split * nc::kSplitLen) {
          const nc::FoldFactors f = nc::fold_scalars(mc_b, zc_b, r.m_b, r.z_b);
#pragma unroll
          for (int e = 0; e < C::NE; ++e) {
            uc[e][2] = nc::fold_u(uc[e][2], u[e][2], f);
            uc[e][3] = nc::fold_u(uc[e][3], u[e][3], f);
          }
        }
      }
#pragma unroll
      for (int e = 0; e < C::NE; ++e) u[e][0] = u[e][1] = u[e][2] = u[e][3] = 0.f;
      r.reset();
    }
  }

  if (timed_out) {
    if (lane == 0) atomicOr(P.status, kStatusTimeout);
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 2000000ull) {
    }
    return;
  }

  const float inv_a = nc::out_scale(zc_a), inv_b = nc::out_scale(zc_b);
  if (valid_a) {
    __nv_bfloat16* dst = P.out + (static_cast<size_t>(rq.q_row0 + tok_a) * P.Hq + head_a) * D + 2 * quad;
#pragma unroll
    for (int e = 0; e < C::NE; ++e)
      *reinterpret_cast<__nv_bfloat162*>(dst + 8 * e) =
          __floats2bfloat162_rn(nc::out_value(uc[e][0], inv_a), nc::out_value(uc[e][1], inv_a));
  }
  if (valid_b) {
    __nv_bfloat16* dst = P.out + (static_cast<size_t>(rq.q_row0 + tok_b) * P.Hq + head_b) * D + 2 * quad;
#pragma unroll
    for (int e = 0; e < C::NE; ++e)
      *reinterpret_cast<__nv_bfloat162*>(dst + 8 * e) =
          __floats2bfloat162_rn(nc::out_value(uc[e][2], inv_b), nc::out_value(uc[e][3], inv_b));
  }
}

}  // namespace vosti
