// Attention tile loop, one warp per (work item, KV head).
//
// Every warp is an independent worker: it owns a private ring of shared-memory
// stages fed by its own TMA page gathers (one mbarrier per stage), walks the
// key tiles of its item in ascending order and keeps the fp32 state (m, z, U)
// of up to 16 rows (token x head-in-group) in registers.  QK^T and PV run on
// the tensor cores (mma.sync m16n8k16, bf16 in, fp32 accumulate), head-dim and
// key chunks of 16 in ascending order.
//
//   SEQ = false (split-parallel, decode / short queries): the item is one
//         split of 512 keys; the warp writes its partial (m, z, U).
//   SEQ = true  (long queries): the item covers splits 0..K-1; the warp folds
//         each finished split into a running result with the same fold the
//         combine kernel uses, then normalises and stores bf16 output.
//
// Both follow App. A's iteration (mask, h = any visible, m_hat, alpha, A,
// z_hat, U_hat, select on h) through the shared scalar rules in nc_math.cuh.
#pragma once
#include "meta.cuh"
#include "nc_math.cuh"
#include "ptx.cuh"

namespace vosti {

constexpr int kWarpsPerCta = 4;
constexpr uint32_t kStatusTimeout = 1u;

template <int D>
struct WarpKernelCfg {
  static constexpr int kStageBytes = nc::kKeyTile * D * 2;  // one K or one V tile
  static constexpr int kStages = (D == 128) ? 3 : 6;        // per warp
  static constexpr int kHalfBytes = nc::kKeyTile * 128;     // 64 keys x 64 elements
  static constexpr int kPageBytes = nc::kPageSize * 128;    // one TMA box: 16 keys x 64 elements
  static constexpr int kSmemBytes =
      kWarpsPerCta * kStages * kStageBytes + kWarpsPerCta * kStages * 8 + 1024;
};

template <int D, bool SEQ>
__global__ void __launch_bounds__(kWarpsPerCta * 32, 1)
attn_warp_kernel(const __grid_constant__ CUtensorMap kv_map, const AttnParams P) {
  using Cfg = WarpKernelCfg<D>;
  constexpr int R = Cfg::kStages;
  constexpr int KC = D / 16;  // head-dim chunks of 16
  constexpr int NE = D / 8;   // output column tiles of 8
  constexpr int NT = nc::kKeyTile / 8;
  constexpr int TPS = nc::kTilesPerSplit;
  constexpr unsigned FULL = 0xffffffffu;

  extern __shared__ uint8_t smem_raw[];
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int quad = lane & 3;
  const int worker = blockIdx.x * kWarpsPerCta + warp;
  if (worker >= P.n_workers) return;  // warps never synchronise with one another

  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t stage0 = base + warp * R * Cfg::kStageBytes;
  const uint32_t bar0 = base + kWarpsPerCta * R * Cfg::kStageBytes + warp * R * 8;

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

  // Rows of this thread: rho and rho + 8 of the 16-row group.
  const int row_a = item.row_group * nc::kRowsPerGroup + (lane >> 2);
  const int row_b = row_a + 8;
  const int tok_a = row_a / G, tok_b = row_b / G;
  const bool valid_a = tok_a < rq.q_len, valid_b = tok_b < rq.q_len;
  const int p_a = valid_a ? rq.start + tok_a : -1;  // padding rows see nothing
  const int p_b = valid_b ? rq.start + tok_b : -1;
  const int head_a = kvh * G + row_a % G, head_b = kvh * G + row_b % G;
  const int last_tok = min(rq.q_len - 1, (item.row_group * nc::kRowsPerGroup + 15) / G);
  const int p_max = rq.start + last_tok;
  const int n_eff = rq.start + rq.q_len;  // slots at or beyond this hold nothing we may read

  const int t_begin = item.split_begin * TPS;
  const int t_end = min(item.split_end * TPS, p_max / nc::kKeyTile + 1);
  const int n_loads = 2 * (t_end - t_begin);

  // Query fragments (A operand), loaded once.
  uint32_t qa[KC][4];
  {
    const __nv_bfloat16* qr_a =
        P.q + (static_cast<size_t>(rq.q_row0 + tok_a) * P.Hq + head_a) * D + 2 * quad;
    const __nv_bfloat16* qr_b =
        P.q + (static_cast<size_t>(rq.q_row0 + tok_b) * P.Hq + head_b) * D + 2 * quad;
#pragma unroll
    for (int kc = 0; kc < KC; ++kc) {
      qa[kc][0] = valid_a ? *reinterpret_cast<const uint32_t*>(qr_a + 16 * kc) : 0u;
      qa[kc][1] = valid_b ? *reinterpret_cast<const uint32_t*>(qr_b + 16 * kc) : 0u;
      qa[kc][2] = valid_a ? *reinterpret_cast<const uint32_t*>(qr_a + 16 * kc + 8) : 0u;
      qa[kc][3] = valid_b ? *reinterpret_cast<const uint32_t*>(qr_b + 16 * kc + 8) : 0u;
    }
  }

  // Page ids of the split being loaded: lane l holds the id of page 32*split + l.
  const int32_t* bt = P.bt_flat + rq.bt_off;
  auto fetch_pages = [&](int split) -> int {
    const int pg = split * nc::kPagesPerSplit + lane;
    return pg < rq.n_pages ? __ldg(bt + pg) : -1;
  };
  int pages_even = -1, pages_odd = -1;
  {
    const int first = item.split_begin;
    const int ids = fetch_pages(first);
    if (first & 1) pages_odd = ids; else pages_even = ids;
  }

  // Issue load i of the item: tile t_begin + i/2, K if i is even, V if odd.
  auto issue = [&](int i) {
    const int t = t_begin + (i >> 1);
    const int is_v = i & 1;
    const int split = t / TPS;
    const int tl = t - split * TPS;
    if (!is_v && tl == TPS / 2 && split + 1 < item.split_end) {
      const int ids = fetch_pages(split + 1);  // needed four tiles from now
      if ((split + 1) & 1) pages_odd = ids; else pages_even = ids;
    }
    const int ids = (split & 1) ? pages_odd : pages_even;
    const int stage = i % R;
    const uint32_t dst = stage0 + stage * Cfg::kStageBytes;
    const uint32_t bar = bar0 + stage * 8;
    const int n_valid = min(nc::kPagesPerTile, rq.n_pages - t * nc::kPagesPerTile);
    if (lane == 0) {
      fence_proxy_async();
      mbar_expect_tx(bar, n_valid * nc::kPageSize * D * 2);
    }
#pragma unroll
    for (int j = 0; j < nc::kPagesPerTile; ++j) {
      const int page = __shfl_sync(FULL, ids, tl * nc::kPagesPerTile + j);
      if (lane == 0 && j < n_valid) {
        const int32_t y = ((page * P.Hkv + kvh) * 2 + is_v) * nc::kPageSize;
#pragma unroll
        for (int h = 0; h < D / 64; ++h)
          tma_load_2d(dst + h * Cfg::kHalfBytes + j * Cfg::kPageBytes, &kv_map, h * 64, y, bar);
      }
    }
  };

#pragma unroll 1
  for (int i = 0; i < R && i < n_loads; ++i) issue(i);

  // State of the current split and (SEQ only) of the running fold.
  float u[NE][4];
  float m_a, m_b, z_a, z_b;
  float uc[SEQ ? NE : 1][4];
  float mc_a = 0.f, mc_b = 0.f, zc_a = 0.f, zc_b = 0.f;
  auto reset_split = [&]() {
#pragma unroll
    for (int e = 0; e < NE; ++e) u[e][0] = u[e][1] = u[e][2] = u[e][3] = 0.f;
    m_a = m_b = -INFINITY;
    z_a = z_b = 0.f;
  };
  reset_split();

  // ldmatrix lane addressing inside a stage (128-byte swizzle: the 16-byte
  // chunk index of a 128-byte row is XORed with the row index mod 8).
  const int lm_mat = lane >> 3, lm_row = lane & 7;
  bool timed_out = false;

#pragma unroll 1
  for (int t = t_begin; t < t_end; ++t) {
    const int li = 2 * (t - t_begin);
    const int key0 = t * nc::kKeyTile;

    // ---- S = Q K^T ---------------------------------------------------------
    {
      const int stage = li % R;
      if (!__all_sync(FULL, mbar_wait_bounded(bar0 + stage * 8, (li / R) & 1))) {
        timed_out = true;  // warp-uniform: every lane leaves together
        break;
      }
    }
    float s[NT][4];
    {
      const uint32_t ks = stage0 + (li % R) * Cfg::kStageBytes;
#pragma unroll
      for (int n = 0; n < NT; ++n) {
        s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
        const int key = n * 8 + lm_row;
#pragma unroll
        for (int cp = 0; cp < KC / 2; ++cp) {
          const int x = 4 * cp + lm_mat;
          const uint32_t addr =
              ks + (x >> 3) * Cfg::kHalfBytes + key * 128 + (((x & 7) ^ (key & 7)) << 4);
          uint32_t b0, b1, b2, b3;
          ldsm_x4(addr, b0, b1, b2, b3);
          mma_bf16_16816(s[n], qa[2 * cp], b0, b1);
          mma_bf16_16816(s[n], qa[2 * cp + 1], b2, b3);
        }
      }
    }
    __syncwarp();
    if (li + R < n_loads) issue(li + R);

    // ---- mask, online softmax ----------------------------------------------
    const bool h_a = key0 <= p_a, h_b = key0 <= p_b;
    float mx_a = -INFINITY, mx_b = -INFINITY;
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      const int j = key0 + n * 8 + 2 * quad;
      mx_a = fmaxf(mx_a, j <= p_a ? s[n][0] : -INFINITY);
      mx_a = fmaxf(mx_a, j + 1 <= p_a ? s[n][1] : -INFINITY);
      mx_b = fmaxf(mx_b, j <= p_b ? s[n][2] : -INFINITY);
      mx_b = fmaxf(mx_b, j + 1 <= p_b ? s[n][3] : -INFINITY);
    }
    mx_a = fmaxf(mx_a, __shfl_xor_sync(FULL, mx_a, 1));
    mx_a = fmaxf(mx_a, __shfl_xor_sync(FULL, mx_a, 2));
    mx_b = fmaxf(mx_b, __shfl_xor_sync(FULL, mx_b, 1));
    mx_b = fmaxf(mx_b, __shfl_xor_sync(FULL, mx_b, 2));
    const float mn_a = h_a ? nc::new_max(m_a, mx_a, c) : m_a;
    const float mn_b = h_b ? nc::new_max(m_b, mx_b, c) : m_b;
    const float al_a = h_a ? nc::rescale(m_a, mn_a) : 1.0f;
    const float al_b = h_b ? nc::rescale(m_b, mn_b) : 1.0f;
    const float ng_a = -mn_a, ng_b = -mn_b;
    float w_a[16], w_b[16];
#pragma unroll
    for (int n = 0; n < NT; ++n) {
      const int j = key0 + n * 8 + 2 * quad;
      w_a[2 * n] = j <= p_a ? nc::weight(s[n][0], c, ng_a) : 0.f;
      w_a[2 * n + 1] = j + 1 <= p_a ? nc::weight(s[n][1], c, ng_a) : 0.f;
      w_b[2 * n] = j <= p_b ? nc::weight(s[n][2], c, ng_b) : 0.f;
      w_b[2 * n + 1] = j + 1 <= p_b ? nc::weight(s[n][3], c, ng_b) : 0.f;
    }
    {
      float ps_a = nc::quad_partial(w_a), ps_b = nc::quad_partial(w_b);
      // (s0 + s1) + (s2 + s3): xor 1 pairs quads (0,1) and (2,3), xor 2 joins them.
      ps_a = __fadd_rn(ps_a, __shfl_xor_sync(FULL, ps_a, 1));
      ps_a = __fadd_rn(ps_a, __shfl_xor_sync(FULL, ps_a, 2));
      ps_b = __fadd_rn(ps_b, __shfl_xor_sync(FULL, ps_b, 1));
      ps_b = __fadd_rn(ps_b, __shfl_xor_sync(FULL, ps_b, 2));
      z_a = h_a ? nc::z_update(z_a, al_a, ps_a) : z_a;
      z_b = h_b ? nc::z_update(z_b, al_b, ps_b) : z_b;
      m_a = mn_a;
      m_b = mn_b;
    }
#pragma unroll
    for (int e = 0; e < NE; ++e) {
      u[e][0] = nc::u_rescale(u[e][0], al_a);
      u[e][1] = nc::u_rescale(u[e][1], al_a);
      u[e][2] = nc::u_rescale(u[e][2], al_b);
      u[e][3] = nc::u_rescale(u[e][3], al_b);
    }
    uint32_t pa[NT / 2][4];
#pragma unroll
    for (int kc = 0; kc < NT / 2; ++kc) {
      __nv_bfloat162 t0 = __floats2bfloat162_rn(w_a[4 * kc], w_a[4 * kc + 1]);
      __nv_bfloat162 t1 = __floats2bfloat162_rn(w_b[4 * kc], w_b[4 * kc + 1]);
      __nv_bfloat162 t2 = __floats2bfloat162_rn(w_a[4 * kc + 2], w_a[4 * kc + 3]);
      __nv_bfloat162 t3 = __floats2bfloat162_rn(w_b[4 * kc + 2], w_b[4 * kc + 3]);
      pa[kc][0] = *reinterpret_cast<uint32_t*>(&t0);
      pa[kc][1] = *reinterpret_cast<uint32_t*>(&t1);
      pa[kc][2] = *reinterpret_cast<uint32_t*>(&t2);
      pa[kc][3] = *reinterpret_cast<uint32_t*>(&t3);
    }

    // ---- U += P V ----------------------------------------------------------
    {
      const int stage = (li + 1) % R;
      if (!__all_sync(FULL, mbar_wait_bounded(bar0 + stage * 8, ((li + 1) / R) & 1))) {
        timed_out = true;
        break;
      }
    }
    const uint32_t vs = stage0 + ((li + 1) % R) * Cfg::kStageBytes;
    if (key0 + nc::kKeyTile > n_eff) {
      // Tail tile: value rows at or beyond n_eff were not loaded or hold
      // whatever the pool had; zero them so that a zero weight times a
      // non-finite value cannot poison the row.
      const int first = n_eff - key0;  // 1..63
      const int n_chunks = (nc::kKeyTile - first) * 8 * (D / 64);
      for (int x = lane; x < n_chunks; x += 32) {
        const int half = x / ((nc::kKeyTile - first) * 8);
        const int y = x - half * (nc::kKeyTile - first) * 8;
        const uint32_t addr = vs + half * Cfg::kHalfBytes + (first + (y >> 3)) * 128 + ((y & 7) << 4);
        asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(addr), "r"(0u) : "memory");
      }
      __syncwarp();
    }
#pragma unroll
    for (int e = 0; e < NE; e += 2) {
#pragma unroll
      for (int kc = 0; kc < NT / 2; ++kc) {
        const int key = kc * 16 + (lm_mat & 1) * 8 + lm_row;
        const int x = e + (lm_mat >> 1);
        const uint32_t addr =
            vs + (x >> 3) * Cfg::kHalfBytes + key * 128 + (((x & 7) ^ (key & 7)) << 4);
        uint32_t b0, b1, b2, b3;
        ldsm_x4_trans(addr, b0, b1, b2, b3);
        mma_bf16_16816(u[e], pa[kc], b0, b1);
        mma_bf16_16816(u[e + 1], pa[kc], b2, b3);
      }
    }
    __syncwarp();
    if (li + 1 + R < n_loads) issue(li + 1 + R);

    // ---- end of a split ------------------------------------------------------
    if constexpr (SEQ) {
      if ((t + 1) % TPS == 0 || t + 1 == t_end) {
        const int split = t / TPS;
        const bool vis_a = p_a >= split * nc::kSplitLen, vis_b = p_b >= split * nc::kSplitLen;
        if (split == 0) {
#pragma unroll
          for (int e = 0; e < NE; ++e) {
            uc[e][0] = u[e][0]; uc[e][1] = u[e][1]; uc[e][2] = u[e][2]; uc[e][3] = u[e][3];
          }
          mc_a = m_a; mc_b = m_b; zc_a = z_a; zc_b = z_b;
        } else {
          if (vis_a) {
            const nc::FoldFactors f = nc::fold_scalars(mc_a, zc_a, m_a, z_a);
#pragma unroll
            for (int e = 0; e < NE; ++e) {
              uc[e][0] = nc::fold_u(uc[e][0], u[e][0], f);
              uc[e][1] = nc::fold_u(uc[e][1], u[e][1], f);
            }
          }
          if (vis_b) {
            const nc::FoldFactors f = nc::fold_scalars(mc_b, zc_b, m_b, z_b);
#pragma unroll
            for (int e = 0; e < NE; ++e) {
              uc[e][2] = nc::fold_u(uc[e][2], u[e][2], f);
              uc[e][3] = nc::fold_u(uc[e][3], u[e][3], f);
            }
          }
        }
        reset_split();
      }
    }
  }

  if (timed_out) {
    if (lane == 0) atomicOr(P.status, kStatusTimeout);
    // Give copies still in flight a bounded chance to land before the CTA's
    // shared memory can be handed to another block.
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 2000000ull) {
    }
    return;
  }

  if constexpr (!SEQ) {
    // Partial (m, z, U) of split `split_begin` for the rows that see it.
    const int split = item.split_begin;
    const int rows = rq.q_len * G;
    const int64_t slab = rq.part_base + (static_cast<int64_t>(kvh) * rq.n_splits + split) * rows;
    if (valid_a && p_a >= split * nc::kSplitLen) {
      float* dst = P.ws_u + (slab + row_a) * D + 2 * quad;
#pragma unroll
      for (int e = 0; e < NE; ++e) *reinterpret_cast<float2*>(dst + 8 * e) = make_float2(u[e][0], u[e][1]);
      if (quad == 0) P.ws_mz[slab + row_a] = make_float2(m_a, z_a);
    }
    if (valid_b && p_b >= split * nc::kSplitLen) {
      float* dst = P.ws_u + (slab + row_b) * D + 2 * quad;
#pragma unroll
      for (int e = 0; e < NE; ++e) *reinterpret_cast<float2*>(dst + 8 * e) = make_float2(u[e][2], u[e][3]);
      if (quad == 0) P.ws_mz[slab + row_b] = make_float2(m_b, z_b);
    }
  } else {
    const float inv_a = nc::out_scale(zc_a), inv_b = nc::out_scale(zc_b);
    if (valid_a) {
      __nv_bfloat16* dst =
          P.out + (static_cast<size_t>(rq.q_row0 + tok_a) * P.Hq + head_a) * D + 2 * quad;
#pragma unroll
      for (int e = 0; e < NE; ++e)
        *reinterpret_cast<__nv_bfloat162*>(dst + 8 * e) = __floats2bfloat162_rn(
            nc::out_value(uc[e][0], inv_a), nc::out_value(uc[e][1], inv_a));
    }
    if (valid_b) {
      __nv_bfloat16* dst =
          P.out + (static_cast<size_t>(rq.q_row0 + tok_b) * P.Hq + head_b) * D + 2 * quad;
#pragma unroll
      for (int e = 0; e < NE; ++e)
        *reinterpret_cast<__nv_bfloat162*>(dst + 8 * e) = __floats2bfloat162_rn(
            nc::out_value(uc[e][2], inv_b), nc::out_value(uc[e][3], inv_b));
    }
  }
}

// Cross-split combine for split-parallel rows: one warp per (token, query
// head) folds the partials of splits 0..floor(p / L_S) left to right, then
// normalises.  Order depends on the split index only.
template <int D>
__global__ void __launch_bounds__(128) combine_kernel(const AttnParams P) {
  constexpr int V = D / 32;  // floats per lane
  const int lane = threadIdx.x & 31;
  const int widx = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (widx >= P.n_split_tokens * P.Hq) return;
  const int2 rt = P.split_tokens[widx / P.Hq];
  const int head = widx % P.Hq;
  const ReqMeta rq = P.reqs[rt.x];
  const int kvh = head / P.G;
  const int row = rt.y * P.G + head % P.G;
  const int rows = rq.q_len * P.G;
  const int p = rq.start + rt.y;
  const int n_splits = p / nc::kSplitLen + 1;
  const int64_t slab0 = rq.part_base + static_cast<int64_t>(kvh) * rq.n_splits * rows + row;

  float uc[V];
  float mc, zc;
  {
    const float2 mz = P.ws_mz[slab0];
    mc = mz.x;
    zc = mz.y;
    const float* src = P.ws_u + slab0 * D + lane * V;
    if constexpr (V == 4) {
      const float4 x = *reinterpret_cast<const float4*>(src);
      uc[0] = x.x; uc[1] = x.y; uc[2] = x.z; uc[3] = x.w;
    } else {
      const float2 x = *reinterpret_cast<const float2*>(src);
      uc[0] = x.x; uc[1] = x.y;
    }
  }
#pragma unroll 4
  for (int k = 1; k < n_splits; ++k) {
    const int64_t slab = slab0 + static_cast<int64_t>(k) * rows;
    const float2 mz = P.ws_mz[slab];
    float uk[V];
    const float* src = P.ws_u + slab * D + lane * V;
    if constexpr (V == 4) {
      const float4 x = *reinterpret_cast<const float4*>(src);
      uk[0] = x.x; uk[1] = x.y; uk[2] = x.z; uk[3] = x.w;
    } else {
      const float2 x = *reinterpret_cast<const float2*>(src);
      uk[0] = x.x; uk[1] = x.y;
    }
    const nc::FoldFactors f = nc::fold_scalars(mc, zc, mz.x, mz.y);
#pragma unroll
    for (int i = 0; i < V; ++i) uc[i] = nc::fold_u(uc[i], uk[i], f);
  }
  const float inv = nc::out_scale(zc);
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
  const int slot = P.slot[tok];
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

}  // namespace vosti
