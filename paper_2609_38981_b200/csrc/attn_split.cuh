// Split-parallel attention (decode, speculative and other short queries): a
// persistent kernel, one CTA per SM, eight (or four, or two) independent warp
// workers per CTA.
//
// A worker draws (item, KV head) tickets from a global counter.  An item is one
// KV split (512 keys) of one 16-row group of a request; the worker walks its
// key tiles in ascending order and writes the partial (m, z, U) of the rows
// that see the split.  Each worker owns a ring of shared-memory stages filled
// by its own TMA page gathers; the load stream runs ahead of the consumer
// across item boundaries, so the ring stays full while one item ends and the
// next begins.  Which worker runs which item, and when, has no effect on the
// bits: partials are folded later in split order.
#pragma once
#include "meta.cuh"
#include "tile_math.cuh"

namespace vosti {

// Eight workers per SM (two per scheduler, so one worker's instruction latency
// hides behind the other's); each owns kStages stages of 32 keys (K or V).
// With few items (a small batch) a CTA runs fewer workers, each with a deeper ring: a worker's
// speed is then bound by the bytes it keeps in flight, not by its share of the SM.
//
// NARROW (four workers, each with the eight-worker ring): the CTA takes half of an SM's shared
// memory and registers, so that a CTA of the tensor-memory tile kernel fits beside it.  Used when a
// tile kernel follows in the same call: the two then run side by side (the split-parallel rows are
// bound by HBM, the tiles by the tensor pipe and the SFU), see launch_attention().
template <int D, int WARPS = 8, bool NARROW = false>
struct SplitKernelCfg {
  static_assert(WARPS == 8 || WARPS == 4 || WARPS == 2, "workers per CTA");
  static_assert(!NARROW || WARPS == 4, "the narrow variant has four workers");
  static constexpr int kWarps = WARPS;
  // With eight workers a ring of three 32-key stages is what the shared memory allows; with fewer,
  // a stage is a whole 64-key tile (K or V): half as many TMA instructions and barrier probes.
  static constexpr int kStageKeys = (WARPS == 8 || NARROW) ? 32 : 64;
  static constexpr int kStages = NARROW ? 3 : ((D == 128) ? 24 : 48) / WARPS / (kStageKeys / 32);
  static constexpr int kSmemBytes =
      kWarps * kStages * TileCfg<D, kStageKeys>::kStageBytes + kWarps * kStages * 8 + 1024;
};

template <int D, int WARPS = 8, bool NARROW = false>
__global__ void __launch_bounds__(WARPS * 32, 1)
attn_split_kernel(const __grid_constant__ CUtensorMap kv_map, const AttnParams P) {  // kv_map: the 3-D page map
  constexpr bool PM = true;  // stages are page-major: one TMA box per (page, K|V)
  constexpr int SK = SplitKernelCfg<D, WARPS, NARROW>::kStageKeys;
  using C = TileCfg<D, SK>;
  constexpr int kWarpsPerCta = SplitKernelCfg<D, WARPS, NARROW>::kWarps;
  constexpr int R = SplitKernelCfg<D, WARPS, NARROW>::kStages;
  constexpr int TPS = nc::kTilesPerSplit;
  constexpr int LPT = 2 * C::kParts;  // loads per tile: K parts then V parts

  extern __shared__ uint8_t smem_raw[];
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int quad = lane & 3;
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

  const int G = P.G;
  const float c = P.c;
  // A device-planned call reads items a kernel earlier in the stream wrote: nothing before it is done.
  if (P.counts != nullptr) griddep_wait();

  // ---- tickets ---------------------------------------------------------------
  // Producer-side description of an item: enough to issue its loads.
  struct Desc {
    uint32_t ticket;
    int kvh, t_begin, n_loads, n_pages, ids;
    int split_tile0;  // first key tile of the item's split (t_begin may lie after it under a window)
  };
  auto read_item = [&](uint32_t ticket) -> SplitItem {
    const int4* src = reinterpret_cast<const int4*>(P.split_items + ticket / P.Hkv);
    const int4 a = __ldg(src), b = __ldg(src + 1), d = __ldg(src + 2);
    SplitItem si;
    si.q_row0 = a.x; si.q_len = a.y; si.start = a.z; si.n_pages = a.w;
    si.bt_index = b.x; si.split = b.y; si.row_group = b.z; si.n_splits = b.w;
    si.part_base = (static_cast<int64_t>(static_cast<uint32_t>(d.y)) << 32) | static_cast<uint32_t>(d.x);
    si.req = d.z; si.first_split = d.w;
    return si;
  };
  // The first ticket of worker w is w itself; later ones come from the counter.
  const uint32_t n_static = gridDim.x * kWarpsPerCta;
  auto draw = [&](Desc& d, bool first) -> bool {
    uint32_t t = blockIdx.x * kWarpsPerCta + warp;
    if (!first) {
      if (lane == 0) t = n_static + atomicAdd(P.ticket, 1u);
      t = __shfl_sync(kFullMask, t, 0);
    }
    const uint32_t n_workers = P.counts != nullptr ? static_cast<uint32_t>(__ldg(P.counts)) : static_cast<uint32_t>(P.n_workers);
    if (t >= n_workers) return false;
    const SplitItem si = read_item(t);
    int t_end, t_first;
    if (si.req < 0) {  // packed rows: every row sees the whole split
      t_end = (si.split + 1) * TPS;
      t_first = 0;
    } else {
      const int last_tok = min(si.q_len - 1, (si.row_group * nc::kRowsPerGroup + 15) / G);
      t_end = min((si.split + 1) * TPS, (si.start + last_tok) / nc::kKeyTile + 1);
      // under a sliding window the group's first row needs nothing before this tile
      const int first_tok = (si.row_group * nc::kRowsPerGroup) / G;
      t_first = nc::first_key(si.start + first_tok, P.window) / nc::kKeyTile;
    }
    d.ticket = t;
    d.kvh = static_cast<int>(t % P.Hkv);
    d.split_tile0 = si.split * TPS;
    d.t_begin = max(si.split * TPS, t_first);
    d.n_loads = LPT * (t_end - d.t_begin);
    d.n_pages = si.n_pages;
    d.ids = (si.split * nc::kPagesPerSplit + lane < si.n_pages) ? __ldg(P.bt_flat + si.bt_index + lane) : -1;
    if (P.counts != nullptr) {  // nobody has looked at these page ids yet: report strays, read page 0 instead
      // (entries wholly before the window of the request's first row are not looked at at all:
      // the caller may have given those pages back; page 0 stands in where a load still covers them)
      const int pg = si.split * nc::kPagesPerSplit + lane;
      if (pg < nc::first_key(si.start, P.window) / nc::kPageSize) d.ids = 0;
      const bool stray = d.ids < -1 || d.ids >= P.num_pages || (d.ids == -1 && pg < si.n_pages);
      if (__any_sync(kFullMask, stray) && lane == 0) atomicOr(P.status, kStatusBadMetadata);
      if (stray) d.ids = 0;
    }
    return true;
  };
  auto leave = [&]() {
    if (lane == 0) {
      __threadfence();
      const uint32_t d = atomicAdd(P.done, 1u);
      if (d == gridDim.x * kWarpsPerCta - 1) {  // last worker out resets the counters
        *P.ticket = 0u;
        *P.done = 0u;
        __threadfence();
      }
    }
  };

  Desc cur, nxt;
  nxt.ticket = 0; nxt.kvh = 0; nxt.t_begin = 0; nxt.n_loads = 0; nxt.n_pages = 0; nxt.ids = -1;
  if (!draw(cur, true)) {
    leave();
    return;
  }
  bool has_nxt = true;      // assumed until the second draw says otherwise
  bool drew_second = false;
  griddep_wait();           // the pool (appended tokens) and Q come from earlier work in the stream
  // The kernel after this one may be scheduled from here on (where an SM has room, or as this
  // grid's CTAs retire).  What it reads of this kernel's results it reads after its own
  // griddep_wait(); a tile kernel that reads none of them starts at once, and everything before
  // this kernel in the stream is complete by then, because every worker has waited for it above.
  griddep_launch();

  // ---- load stream -------------------------------------------------------------
  uint32_t g_issue = 0, g_cons = 0;  // loads issued / consumed since kernel start
  int ahead = 0;                     // 0: issuing for cur, 1: for nxt, 2: nxt fully issued
  int prod_li = 0;                   // next load of the item being issued
  bool prod_done = false;
  auto issue_one = [&]() -> bool {
    if (prod_done || ahead == 2 || g_issue - g_cons >= static_cast<uint32_t>(R)) return false;
    if (ahead == 1 && !drew_second) return false;  // nxt not drawn yet (first item only)
    const int kvh = ahead ? nxt.kvh : cur.kvh;
    const int t_begin = ahead ? nxt.t_begin : cur.t_begin;
    const int n_loads = ahead ? nxt.n_loads : cur.n_loads;
    const int n_pages = ahead ? nxt.n_pages : cur.n_pages;
    const int ids = ahead ? nxt.ids : cur.ids;
    const int split_tile0 = ahead ? nxt.split_tile0 : cur.split_tile0;
    const int tl = t_begin - split_tile0 + prod_li / LPT;  // tile within the split
    const int tw = prod_li / LPT;                           // tile within the item
    const int sub = prod_li - tw * LPT;    // 0 .. kParts-1: K parts, then V parts
    const int is_v = sub >= C::kParts;
    const int part = sub - is_v * C::kParts;
    const int first_page = tl * nc::kPagesPerTile + part * C::kPagesPerStage;  // within the split
    const int stage = g_issue % R;
    issue_stage_load<D, SK, PM>(&kv_map, stage0 + stage * C::kStageBytes, bar0 + stage * 8, ids, first_page,
                            max(0, min(C::kPagesPerStage, n_pages - (split_tile0 * nc::kPagesPerTile + first_page))),
                            P.Hkv, kvh, is_v, lane);
    ++g_issue;
    if (++prod_li == n_loads) {
      prod_li = 0;
      ++ahead;
      if (ahead == 1 && !has_nxt) prod_done = true;
    }
    return true;
  };

  bool timed_out = false;
  while (true) {
    while (issue_one()) {
    }
    // ---- consumer set-up for `cur` -----------------------------------------------
    const SplitItem si = read_item(cur.ticket);
    const int kvh = cur.kvh;
    // The warp's 16 rows: a row group of one request, or packed rows of several requests.
    const bool packed = si.req < 0;
    bool valid_a, valid_b, upper_rows;
    const __nv_bfloat16 *q_a, *q_b;
    int64_t out_a, out_b;  // partial rows the two rows write
    int n_eff, p_min, lo_top, lo_first;
    RowPair r;
    if (packed) {
      const int ra = lane >> 2, rb = ra + 8;
      valid_a = ra < si.q_len;
      valid_b = rb < si.q_len;
      const int4* rows = reinterpret_cast<const int4*>(P.packed_rows) + static_cast<size_t>(-1 - si.req) * 16;
      const int4 da = __ldg(rows + (valid_a ? ra : 0)), db = __ldg(rows + (valid_b ? rb : 0));
      r.p_a = valid_a ? da.y : -1;
      r.p_b = valid_b ? db.y : -1;
      r.lo_a = r.lo_b = nc::kNoLowerBound;
      q_a = P.q + (static_cast<size_t>(da.x & 0xffffff) * P.Hq + kvh * G + (da.x >> 24)) * D;
      q_b = P.q + (static_cast<size_t>(db.x & 0xffffff) * P.Hq + kvh * G + (db.x >> 24)) * D;
      out_a = valid_a ? da.z + static_cast<int64_t>(kvh) * da.w : -1;
      out_b = valid_b ? db.z + static_cast<int64_t>(kvh) * db.w : -1;
      n_eff = 0x7fffffff;                           // a complete split: no tail to clear
      p_min = (si.split + 1) * nc::kSplitLen;       // every key of the split is visible to every row
      lo_top = lo_first = nc::kNoLowerBound;
      upper_rows = si.q_len > 8;
    } else {
      const int row_a = si.row_group * nc::kRowsPerGroup + (lane >> 2);
      const int row_b = row_a + 8;
      const int tok_a = row_a / G, tok_b = row_b / G;
      valid_a = tok_a < si.q_len;
      valid_b = tok_b < si.q_len;
      r.p_a = valid_a ? si.start + tok_a : -1;
      r.p_b = valid_b ? si.start + tok_b : -1;
      r.lo_a = nc::window_lo(r.p_a, P.window);
      r.lo_b = nc::window_lo(r.p_b, P.window);
      q_a = P.q + (static_cast<size_t>(si.q_row0 + tok_a) * P.Hq + kvh * G + row_a % G) * D;
      q_b = P.q + (static_cast<size_t>(si.q_row0 + tok_b) * P.Hq + kvh * G + row_b % G) * D;
      // partial (m, z, U) rows of this split, written only by rows that see some of it
      const int64_t slab = si.part_base + (static_cast<int64_t>(kvh) * si.n_splits + (si.split - si.first_split)) *
                                              (static_cast<int64_t>(si.q_len) * G);
      const int first_key = si.split * nc::kSplitLen, last_key = first_key + nc::kSplitLen - 1;
      out_a = (valid_a && r.p_a >= first_key && r.lo_a < last_key) ? slab + row_a : -1;
      out_b = (valid_b && r.p_b >= first_key && r.lo_b < last_key) ? slab + row_b : -1;
      n_eff = si.start + si.q_len;
      // schedule-only facts about the group: lowest and highest real position (a tile between the
      // highest row's window start and the lowest row's position is visible to every real row),
      // and whether rows 8..15 hold real rows
      p_min = si.start + (si.row_group * nc::kRowsPerGroup) / G;
      const int p_top = si.start + min(si.q_len - 1, (si.row_group * nc::kRowsPerGroup + 15) / G);
      lo_top = nc::window_lo(p_top, P.window);
      lo_first = nc::window_lo(p_min, P.window);  // keys up to here are invisible to the whole group
      upper_rows = (si.row_group * nc::kRowsPerGroup + 8) / G < si.q_len;
    }
    r.reset();
    uint32_t qa[C::KC][4];
    load_q_frags<D>(qa, q_a, q_b, valid_a, valid_b, quad);
    float u[C::NE][4];
#pragma unroll
    for (int e = 0; e < C::NE; ++e) u[e][0] = u[e][1] = u[e][2] = u[e][3] = 0.f;
    if (!drew_second) {  // first item: its loads are already in flight, now draw the next one
      drew_second = true;
      has_nxt = draw(nxt, false);
      if (ahead == 1 && !has_nxt) prod_done = true;
    }

    const int n_tiles = cur.n_loads / LPT;
#pragma unroll 1
    for (int tile = 0; tile < n_tiles; ++tile) {
      const int key0 = (cur.t_begin + tile) * nc::kKeyTile;
      float s[8][4];
#pragma unroll
      for (int part = 0; part < C::kParts; ++part) {
        const int stage = g_cons % R;
        if (!__all_sync(kFullMask, mbar_wait_bounded(bar0 + stage * 8, (g_cons / R) & 1))) {
          timed_out = true;  // warp-uniform: every lane leaves together
          break;
        }
        tile_scores<D, SK, PM>(stage0 + stage * C::kStageBytes, qa, s, part * (SK / 8), lane);
        __syncwarp();
        ++g_cons;
        issue_one();
      }
      if (timed_out) break;
      uint32_t pa[4][4];
      tile_softmax_dispatch<D>(s, key0, c, r, u, pa, quad, key0 + nc::kKeyTile - 1 <= p_min && key0 > lo_top,
                               upper_rows);
#pragma unroll
      for (int part = 0; part < C::kParts; ++part) {
        const int stage = g_cons % R;
        if (!__all_sync(kFullMask, mbar_wait_bounded(bar0 + stage * 8, (g_cons / R) & 1))) {
          timed_out = true;
          break;
        }
        const uint32_t vs = stage0 + stage * C::kStageBytes;
        const int part_key0 = key0 + part * SK;
        if (part_key0 + SK > n_eff) zero_value_tail<D, SK, PM>(vs, max(0, n_eff - part_key0), lane);
        if (part_key0 <= lo_first) zero_value_rows<D, SK, PM>(vs, 0, min(SK, lo_first - part_key0 + 1), lane);
        tile_pv<D, SK, PM>(vs, pa, u, part * (SK / 16), lane);
        __syncwarp();
        ++g_cons;
        issue_one();
      }
      if (timed_out) break;
    }
    if (timed_out) break;

    // ---- partial (m, z, U) of this split for the rows that see it -----------------
    if (out_a >= 0) {
      float* dst = P.ws_u + out_a * D + 2 * quad;
#pragma unroll
      for (int e = 0; e < C::NE; ++e) *reinterpret_cast<float2*>(dst + 8 * e) = make_float2(u[e][0], u[e][1]);
      if (quad == 0) P.ws_mz[out_a] = make_float2(r.m_a, r.z_a);
    }
    if (out_b >= 0) {
      float* dst = P.ws_u + out_b * D + 2 * quad;
#pragma unroll
      for (int e = 0; e < C::NE; ++e) *reinterpret_cast<float2*>(dst + 8 * e) = make_float2(u[e][2], u[e][3]);
      if (quad == 0) P.ws_mz[out_b] = make_float2(r.m_b, r.z_b);
    }
    if (!has_nxt) break;
    cur = nxt;
    --ahead;
    has_nxt = draw(nxt, false);
    if (ahead == 1 && !has_nxt) prod_done = true;
  }

  if (timed_out) {
    if (lane == 0) atomicOr(P.status, kStatusTimeout);
    // Give copies still in flight a bounded chance to land before the CTA's
    // shared memory can be handed to another block.
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 2000000ull) {
    }
  }
  leave();
}

}  // namespace vosti
