// Tile attention for long queries (prefill chunks): one CTA per (128-row tile,
// KV head), two CTAs per SM, QK^T and PV on the 5th-generation tensor cores
// (tcgen05.mma, M = 128) with the accumulators in tensor memory, K/V tiles
// gathered from the page pool by TMA.
//
// It executes the same numerical contract as the split-parallel kernel: key
// tiles of 64 in ascending order; S from head-dim chunks of 16 ascending with a
// fresh accumulator; the scalar softmax rules of nc_math.cuh applied by one
// thread per row (all 64 lanes of the row in its registers, so the pinned
// row-sum order is a matter of adding in that order); U rescaled by alpha and
// then accumulated over key chunks of 16 ascending; at every 512-key split
// boundary the finished split is folded into the running result with
// fold_scalars / fold_u.  tcgen05.mma and mma.sync.m16n8k16 give bit-identical
// sums for the same chunk order (measured on B200), which is what lets this
// kernel and the warp-MMA kernels agree bit for bit.
//
// Work on a row is divided between two threads so that neither chain is long:
//   * a softmax thread reads the row's 64 scores, applies the scalar rules
//     (maximum, alpha, exponentials, pinned row sum), publishes alpha and writes
//     the bf16 weights over the scores;
//   * a correction thread takes alpha and rescales the row's U accumulator when
//     some alpha of its warp is not 1, zero-fills value rows no query row may
//     see, and at the end of every split folds the split into the running
//     result (and, at the end of the row, normalises and stores it).
// (With the lazy reference maximum of the contract alpha is 1 in the common
// case, so the correction thread's per-tile work is a handshake; the thread is
// there for the rare rescale and for the fold.)
// Roles by warpgroup (384 threads): 0 = softmax, 1 = correction, 2 = { K
// producer, V producer, -, MMA issuer }.  Registers are moved from warpgroup 2 to
// the others with setmaxnreg.  The MMAs of the one issuing thread run in issue
// order, which the aliasing of weights over scores relies on.
// Two such CTAs share an SM (half of its shared memory, tensor memory and
// registers each) and know nothing of each other: while one of them waits --
// for its softmax, or for the split fold, which moves 128 KB between tensor
// memory and L2 -- the other one keeps the tensor and MUFU pipes busy.  The two
// 128-row halves of a 256-row work item are neighbouring CTAs, so the K/V tiles
// the second one asks for are in L2 already.
// Tensor memory (256 columns per CTA): S x2 (64 each; the bf16 weights P are
// written over the first 32 columns of the S buffer they were computed from)
// and U (D).  The running fold U_c lives in global memory (per CTA a
// [D/4][128 rows] array of float4, so that a warp's rows are contiguous; touched
// once per split): there is no room for it on chip.  A correction thread asks
// for three 16-column chunks of its row's running fold ahead of their use, with
// cache-global loads and stores (the array is streamed; L1 would only be churned).
// When this kernel is launched right behind a split-parallel kernel of the same
// call it starts without waiting for it and waits before it ends instead
// (AttnParams::beside_split): the two kernels then share the SMs.
// Measured and not kept (all bitwise correct): copying a finished split out and
// folding it behind the next split's tiles doubles the traffic through the SM's
// load/store path and is slower; dividing a row's key columns between two
// threads (two symmetric warpgroups that exchange half-row maxima and sums
// through shared memory) makes the hand-over part of every tile's chain and is
// slower too; so is keeping the first 16 to 48 columns of the running fold in the
// correction thread's registers (it has none to spare: the spills cost more than
// the traffic saved).
#pragma once
#include "meta.cuh"
#include "tcgen05.cuh"
#include "tile_math.cuh"

namespace vosti {
template <int D>
struct TileKernelCfg {
  static constexpr int kItemRows = 256;                      // rows of a work item: two CTAs
  static constexpr int kTileRows = 128;
  static constexpr int kThreads = 384;
  static constexpr int kStages = 2;                          // K+V tile pairs in flight
  static constexpr int kQBytes = kTileRows * D * 2;          // [half][row][128 B]
  static constexpr int kKBytes = nc::kKeyTile * D * 2;       // [half][key][128 B]
  static constexpr int kStageBytes = 2 * kKBytes;            // K then V
  static constexpr int kAlphaBytes = 2 * kTileRows * 4;      // alpha[buffer][row]
  static constexpr int kMzBytes = 2 * kTileRows * 8;         // (m, z)[split parity][row]
  static constexpr int kBarBytes = 512;
  static constexpr int kSmemBytes = kQBytes + kStages * kStageBytes + kAlphaBytes + kMzBytes + kBarBytes + 1024;
  // Registers per thread after the roles have split.  The total must not exceed what the CTA
  // was given at launch (384 threads x 80 registers): a warpgroup asking for more than the
  // others have released waits for ever.
  static constexpr int kRegsLaunch = 80;
  static constexpr int kRegsSoftmax = 112;
  static constexpr int kRegsCorrection = 104;
  static constexpr int kRegsOther = 24;
  static constexpr int kFoldAhead = 3;  // chunks of 16 running-fold columns requested ahead of their use
  static constexpr int kRegsAfterSplit = 128 * (kRegsSoftmax + kRegsCorrection + kRegsOther);
  static_assert(kRegsAfterSplit <= kThreads * kRegsLaunch, "register split exceeds the launch allocation");
  // tensor-memory columns
  static constexpr uint32_t kTmemCols = 256;
  static constexpr uint32_t kColS = 0;    // buffer b: S / P at 64 b
  static constexpr uint32_t kColU = 128;  // U
};

template <int N>
__device__ __forceinline__ void reg_alloc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N>
__device__ __forceinline__ void reg_dealloc() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }

// PACKED = false: a CTA is one 128-row half of a 256-row item of one request; it walks the key
// tiles its rows see, folds split by split and writes the output rows.
// PACKED = true (shared-split packing): a CTA is up to 128 rows of *different* requests that name
// the same pages for one complete split; every row sees every key of the split; the CTA walks
// that split's eight tiles and writes each row's partial (m, z, U) where the split-parallel
// kernel would have written it, for combine_kernel to fold.  Same tiles, same scalar rules,
// same accumulation order per row: the partial is bit for bit the one a 16-row item produces.
template <int D, bool PACKED = false>
__global__ void __launch_bounds__(TileKernelCfg<D>::kThreads, 2)
attn_tile_kernel(const __grid_constant__ CUtensorMap kv_map, const AttnParams P) {
  using Cfg = TileKernelCfg<D>;
  constexpr int NS = Cfg::kStages;
  constexpr int TPS = nc::kTilesPerSplit;
  constexpr int KT = nc::kKeyTile;
  constexpr int TR = Cfg::kTileRows;
  constexpr uint32_t kAbortAfterNs = 1000000000u;

  // CTA -> (work item, KV head, half of the item); packed: CTA -> (packed tile, KV head)
  const int G = P.G;
  const int unit = PACKED ? blockIdx.x : (blockIdx.x >> 1);
  const int kvh = unit % P.Hkv;
  ReqMeta rq;
  int row0, rows, n_eff, n_tiles, T0, lo_first;
  const PackedRow* prow = nullptr;  // packed: the CTA's 128 row records
  if constexpr (PACKED) {
    const int4 ti = P.tile_pack_items[unit / P.Hkv];  // {first page id's index in the flat table, split, rows, -}
    prow = P.tile_rows + static_cast<size_t>(unit / P.Hkv) * TR;
    rq = ReqMeta{};
    rq.bt_off = ti.x - ti.y * nc::kPagesPerSplit;       // so that page index arithmetic stays absolute
    rq.n_pages = (ti.y + 1) * nc::kPagesPerSplit;
    row0 = 0;
    rows = ti.z;
    n_eff = (ti.y + 1) * nc::kSplitLen;                 // a complete split: no tail
    n_tiles = (ti.y + 1) * TPS;
    T0 = ti.y * TPS;
    lo_first = nc::window_lo(0, 0);
  } else {
    const vosti_work_item item = P.items[unit / P.Hkv];
    rq = P.reqs[item.req];
    row0 = item.row_group * nc::kRowsPerGroup + (blockIdx.x & 1) * TR;  // first row of this CTA's tile
    rows = rq.q_len * G;
    if (row0 >= rows) return;  // the item's second half does not exist
    n_eff = rq.start + rq.q_len;
    n_tiles = (rq.start + min(rq.q_len - 1, (row0 + TR - 1) / G)) / KT + 1;  // key tiles walked
    // Under a sliding window nothing before the first visible key of the tile's first row is
    // needed: the walk starts at key tile T0 (rows whose own window starts later take identity
    // steps until it does).  Stages, S buffers and barrier phases are indexed by t - T0.
    const int p_first = rq.start + row0 / G;
    T0 = nc::first_key(p_first, P.window) / KT;
    lo_first = nc::window_lo(p_first, P.window);  // keys up to here are invisible to every row
  }

  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* sbase = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t q_smem = base;
  const uint32_t kv_smem = base + Cfg::kQBytes;
  constexpr int kXchgOff = Cfg::kQBytes + NS * Cfg::kStageBytes;
  float* alpha_s = reinterpret_cast<float*>(sbase + kXchgOff);                       // [b][row]
  float2* mz_s = reinterpret_cast<float2*>(sbase + kXchgOff + Cfg::kAlphaBytes);     // [kb][row]
  constexpr int kBarOff = kXchgOff + Cfg::kAlphaBytes + Cfg::kMzBytes;
  const uint32_t bars = base + kBarOff;
  volatile uint32_t* flags = reinterpret_cast<volatile uint32_t*>(sbase + kBarOff + 448);
  // barrier map (8 bytes each); per buffer b: index b
  const uint32_t k_full = bars, v_full = bars + 8 * NS, k_empty = bars + 16 * NS, v_empty = bars + 24 * NS;
  const uint32_t s_full = bars + 32 * NS, p_full = s_full + 16, pv_done = s_full + 32;
  const uint32_t a_full = s_full + 48, mz_full = s_full + 64;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int wg = warp >> 2;

  if (tid == 0) {
    for (int i = 0; i < NS; ++i) {
      mbar_init(k_full + 8 * i, 1);
      mbar_init(v_full + 8 * i, 1);
      mbar_init(k_empty + 8 * i, 1);
      mbar_init(v_empty + 8 * i, 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(s_full + 8 * i, 1);
      mbar_init(p_full + 8 * i, 2 * TR);  // softmax and correction thread of every row
      mbar_init(pv_done + 8 * i, 1);
      mbar_init(a_full + 8 * i, TR);
      mbar_init(mz_full + 8 * i, TR);
    }
    flags[0] = 0u;  // abort flag
    mbar_fence_init();
    tma_prefetch_desc(&kv_map);
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(bars + 456),
                 "r"(Cfg::kTmemCols));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
  }
  // Q tile -> shared memory, [half][row][128 B] with the 128-byte swizzle; padding rows are zero.
  if (warp < 4) {
    if (!P.beside_split) griddep_wait();
    const int r = tid;
    const int row = row0 + r;
    bool valid = row < rows;
    size_t q_row;  // (packed token row) * Hq + query head
    if constexpr (PACKED) {
      const PackedRow pr = prow[r];
      valid = pr.p >= 0;
      q_row = static_cast<size_t>(pr.q_row_g & 0xFFFFFF) * P.Hq + kvh * G + (static_cast<uint32_t>(pr.q_row_g) >> 24);
    } else {
      q_row = static_cast<size_t>(rq.q_row0 + row / G) * P.Hq + kvh * G + row % G;
    }
    const uint4* src = reinterpret_cast<const uint4*>(P.q + q_row * D);
#pragma unroll
    for (int c = 0; c < D / 8; ++c) {
      const uint4 v = valid ? __ldg(src + c) : make_uint4(0, 0, 0, 0);
      const uint32_t addr = q_smem + (c >> 3) * (TR * 128) + r * 128 + (((c & 7) ^ (r & 7)) << 4);
      asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                   : "memory");
    }
    fence_proxy_async();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(sbase + kBarOff + 456);

  // Bounded wait shared by all roles: gives up after ~1 s or as soon as another
  // thread of the CTA has given up, records the failure, and lets the caller
  // fall through to the common exit (tensor memory is still released).
  auto wait = [&](uint32_t bar, uint32_t parity) -> bool {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    for (uint32_t it = 0;; ++it) {
      if (mbar_try_wait_hint(bar, parity, 4000u)) return true;  // sleeps in hardware, no issue slots burnt
      if ((it & 63u) == 63u) {
        if (flags[0] != 0u) return false;
        if (global_timer_ns() - t0 > kAbortAfterNs) {
          flags[0] = 1u;
          atomicOr(P.status, kStatusTimeout);
          return false;
        }
      }
    }
  };
  // The same for a single thread that must react at once (the MMA issuer): polls without sleeping.
  auto wait_spin = [&](uint32_t bar, uint32_t parity) -> bool {
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
      if (mbar_test_wait(bar, parity)) return true;
      if ((it & 1023u) == 1023u) {
        if (flags[0] != 0u) return false;
        if (it == 1023u) {
          t0 = global_timer_ns();
        } else if (global_timer_ns() - t0 > kAbortAfterNs) {
          flags[0] = 1u;
          atomicOr(P.status, kStatusTimeout);
          return false;
        }
      }
    }
  };

  if (wg == 2) {
    reg_dealloc<Cfg::kRegsOther>();
    // Which warp of the group takes which role decides which scheduler it loads (warp w issues
    // on scheduler w mod 4, beside softmax warp w mod 4 and correction warp 4 + w mod 4): K producer,
    // V producer and issuer on warps 8, 9 and 11 measured 3 % faster than on 8, 10 and 9.
    if (warp == 8 || warp == 9) {
      // ================= TMA producers: warp 8 loads the K tiles, warp 9 the V tiles ========
      if (!P.beside_split) griddep_wait();
      const int is_v = warp == 9;
      const int32_t* bt = P.bt_flat + rq.bt_off;
      auto fetch_pages = [&](int split) -> int {
        const int pg = split * nc::kPagesPerSplit + lane;
        return pg < rq.n_pages ? __ldg(bt + pg) : -1;
      };
      int pages_even = -1, pages_odd = -1;
      if ((T0 / TPS) & 1) pages_odd = fetch_pages(T0 / TPS); else pages_even = fetch_pages(T0 / TPS);
      bool ok = true;
      for (int t = T0; t < n_tiles && ok; ++t) {
        const int s = (t - T0) % NS, use = (t - T0) / NS;
        const int split = t / TPS, tl = t - split * TPS;
        if ((tl == TPS / 2 || (t == T0 && tl > TPS / 2)) && (split + 1) * TPS < n_tiles) {
          const int ids = fetch_pages(split + 1);
          if ((split + 1) & 1) pages_odd = ids; else pages_even = ids;
        }
        const int ids = (split & 1) ? pages_odd : pages_even;
        const int n_valid = min(nc::kPagesPerTile, rq.n_pages - t * nc::kPagesPerTile);
        const uint32_t dst = kv_smem + s * Cfg::kStageBytes + is_v * Cfg::kKBytes;
        const uint32_t full = (is_v ? v_full : k_full) + 8 * s;
        const uint32_t empty = (is_v ? v_empty : k_empty) + 8 * s;
        if (use > 0) ok = __all_sync(kFullMask, wait(empty, (use - 1) & 1));
        if (!ok) break;
        issue_stage_load<D, KT>(&kv_map, dst, full, ids, tl * nc::kPagesPerTile, n_valid, P.Hkv, kvh, is_v, lane);
      }
    } else if (warp == 11 && lane == 0) {
      // ================= MMA issuer ==========================================================
      // One thread's MMAs run in issue order.  S of key tile t+2 overwrites the buffer whose
      // first columns PV of key tile t reads its weights from, so it is issued after that PV.
      constexpr uint32_t idesc_s = umma_idesc(128, KT, false);
      constexpr uint32_t idesc_pv = umma_idesc(128, D, true);
      bool ok = true;
      auto issue_s = [&](int t) {
        const int i = t - T0, s = i % NS, b = i & 1;
        ok = ok && wait_spin(k_full + 8 * s, (i / NS) & 1);
        if (!ok) return;
        tc_fence_after();
        const uint32_t kst = kv_smem + s * Cfg::kStageBytes;
#pragma unroll
        for (int kc = 0; kc < D / 16; ++kc) {
          const uint64_t da = smem_desc_sw128(q_smem + (kc >> 2) * (TR * 128) + (kc & 3) * 32, 16, 1024);
          const uint64_t db = smem_desc_sw128(kst + (kc >> 2) * (KT * 128) + (kc & 3) * 32, 16, 1024);
          tc_mma_ss(tmem + Cfg::kColS + b * KT, da, db, idesc_s, kc > 0 ? 1u : 0u);
        }
        tc_commit(s_full + 8 * b);
        tc_commit(k_empty + 8 * s);
      };
      issue_s(T0);
      for (int t = T0; t < n_tiles && ok; ++t) {
        if (t + 1 < n_tiles) issue_s(t + 1);
        if (!ok) break;
        const int i = t - T0, s = i % NS, b = i & 1;
        ok = wait_spin(v_full + 8 * s, (i / NS) & 1);
        if (!ok) break;
        ok = wait_spin(p_full + 8 * b, (i >> 1) & 1);
        if (!ok) break;
        tc_fence_after();
        const uint32_t vst = kv_smem + s * Cfg::kStageBytes + Cfg::kKBytes;
#pragma unroll
        for (int kc = 0; kc < KT / 16; ++kc) {
          // B = V: MN-major, 64-element halves of d KT*128 bytes apart, 8-key groups 1024 bytes apart
          const uint64_t db = smem_desc_sw128(vst + kc * 2048, KT * 128, 1024);
          // a split (and the first tile walked) starts from a fresh accumulator
          const uint32_t acc = (kc > 0 || ((t % TPS) != 0 && t != T0)) ? 1u : 0u;
          tc_mma_ts(tmem + Cfg::kColU, tmem + Cfg::kColS + b * KT + kc * 8, db, idesc_pv, acc);
        }
        tc_commit(pv_done + 8 * b);
        tc_commit(v_empty + 8 * s);
      }
    }
  } else if (wg == 0) {
    // ================= softmax: one thread per row =======================================
    reg_alloc<Cfg::kRegsSoftmax>();
    const int r = tid;                          // row of the tile = tensor-memory lane
    const int row = row0 + r;
    const bool valid = PACKED ? prow[r].p >= 0 : row < rows;
    const int p = PACKED ? prow[r].p : (valid ? rq.start + row / G : -1);  // padding rows see nothing
    const int lo = nc::window_lo(p, P.window);      // key j is visible iff lo < j <= p
    const uint32_t lane_sel = static_cast<uint32_t>(warp * 32) << 16;
    const float c = P.c;
    float m = -INFINITY, z = 0.f;
    bool ok = true;
    for (int t = T0; t < n_tiles && ok; ++t) {
      const int ti = t - T0, b = ti & 1;
      const int key0 = t * KT;
      ok = __all_sync(kFullMask, wait(s_full + 8 * b, (ti >> 1) & 1));
      if (!ok) break;
      tc_fence_after();
      uint32_t sr[64];
      {
        uint32_t lo32[32], hi32[32];
        tmem_ld32(tmem + lane_sel + Cfg::kColS + b * KT, lo32);
        tmem_ld32(tmem + lane_sel + Cfg::kColS + b * KT + 32, hi32);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) { sr[i] = lo32[i]; sr[32 + i] = hi32[i]; }
      }

      // ---- the scalar rules, lanes b = 0..63 of this row --------------------------
      // Schedule-only shortcut: when every key of the tile is visible to every real
      // row of the warp the selects all take the visible arm and are skipped.
      const bool all_visible = __all_sync(kFullMask, !valid || (key0 + KT - 1 <= p && key0 > lo));
      const bool h = all_visible || (key0 <= p && key0 + KT - 1 > lo);
      float mn, alpha;
      {
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};  // the maximum is order-free
        if (all_visible) {
#pragma unroll
          for (int i = 0; i < KT; i += 8) {
#pragma unroll
            for (int j = 0; j < 4; ++j)
              mx4[j] = nc::max3(mx4[j], __uint_as_float(sr[i + j]), __uint_as_float(sr[i + 4 + j]));
          }
        } else {
#pragma unroll
          for (int i = 0; i < KT; ++i)
            mx4[i & 3] = fmaxf(mx4[i & 3], (key0 + i <= p && key0 + i > lo) ? __uint_as_float(sr[i]) : -INFINITY);
        }
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        mn = h ? nc::new_max(m, mx, c) : m;
        alpha = h ? nc::rescale(m, mn) : 1.0f;
      }
      // the correction thread of this row can start on U while the exponentials are taken
      alpha_s[b * TR + r] = alpha;
      mbar_arrive(a_full + 8 * b);
      {
        const float ng = -mn;
        if (all_visible) {
          const uint64_t c2 = nc::pack2(c, c), ng2 = nc::pack2(ng, ng);
#pragma unroll
          for (int i = 0; i < KT; i += 2) {
            float a0, a1;
            nc::weight2(__uint_as_float(sr[i]), __uint_as_float(sr[i + 1]), c2, ng2, a0, a1);
            sr[i] = __float_as_uint(a0);
            sr[i + 1] = __float_as_uint(a1);
          }
        } else {
#pragma unroll
          for (int i = 0; i < KT; ++i)
            sr[i] = (key0 + i <= p && key0 + i > lo) ? __float_as_uint(nc::weight(__uint_as_float(sr[i]), c, ng)) : 0u;
        }
        // Pinned row sum, per half of 32 lanes: eight chains over b mod 8 (ascending b), chain pairs,
        // (P0 + P1) + (P2 + P3); then lower half + upper half.  Chains 2q and 2q+1 advance together
        // in one packed add on the adjacent lanes (8n + 2q, 8n + 2q + 1).
        float half_sum[2];
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          float part[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            uint64_t acc = nc::pack2(__uint_as_float(sr[32 * hf + 2 * q]), __uint_as_float(sr[32 * hf + 2 * q + 1]));
#pragma unroll
            for (int n = 1; n < 4; ++n)
              acc = nc::add2(acc, nc::pack2(__uint_as_float(sr[32 * hf + 8 * n + 2 * q]),
                                            __uint_as_float(sr[32 * hf + 8 * n + 2 * q + 1])));
            float e0, e1;
            nc::unpack2(acc, e0, e1);
            part[q] = __fadd_rn(e0, e1);
          }
          half_sum[hf] = nc::quad_total(part[0], part[1], part[2], part[3]);
        }
        const float total = nc::tile_total(half_sum[0], half_sum[1]);
        z = h ? nc::z_update(z, alpha, total) : z;
        m = mn;
      }
      uint32_t pk[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        __nv_bfloat162 t2 = __floats2bfloat162_rn(__uint_as_float(sr[2 * i]), __uint_as_float(sr[2 * i + 1]));
        pk[i] = *reinterpret_cast<uint32_t*>(&t2);
      }
      tmem_st32(tmem + lane_sel + Cfg::kColS + b * KT, pk);  // the weights take the place of the scores read above
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(p_full + 8 * b);

      // ---- end of a split: hand (m, z) to the correction thread, start afresh -----------
      if ((t + 1) % TPS == 0 || t + 1 == n_tiles) {
        const int kb = (t / TPS - T0 / TPS) & 1;
        mz_s[kb * TR + r] = make_float2(m, z);
        mbar_arrive(mz_full + 8 * kb);
        m = -INFINITY;
        z = 0.f;
      }
    }
  } else {
    // ================= correction: one thread per row =====================================
    reg_alloc<Cfg::kRegsCorrection>();
    const int r = tid & (TR - 1);
    const int row = row0 + r;
    const bool valid = PACKED ? prow[r].p >= 0 : row < rows;
    const int tok = row / G;
    const int p = PACKED ? prow[r].p : (valid ? rq.start + tok : -1);
    // first split the row sees; before it (and in the first split the CTA walks) the
    // running result is simply taken from the split, as the fold of the split kernels does
    const int k_first = max(nc::first_key(p, P.window) / nc::kSplitLen, T0 / TPS);
    const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
    // running fold of this tile in global memory ([D/4][128] float4: this thread owns column r),
    // and the row's place in the output
    float4* ucg = reinterpret_cast<float4*>(P.ws_uc) + static_cast<size_t>(blockIdx.x) * (D / 4) * TR + r;
    __nv_bfloat16* dst = P.out + (static_cast<size_t>(rq.q_row0 + tok) * P.Hq + kvh * G + row % G) * D;
    // packed: the row's partial slab, where the split-parallel kernel would have put it
    int64_t slab = 0;
    if constexpr (PACKED) {
      const PackedRow pr = prow[r];
      slab = static_cast<int64_t>(pr.slab_row) + static_cast<int64_t>(kvh) * pr.kvh_stride;
    }
    float mc = 0.f, zc = 0.f;
    bool ok = true;
    for (int t = T0; t < n_tiles && ok; ++t) {
      const int ti = t - T0, b = ti & 1, s = ti % NS;
      const int key0 = t * KT;
      ok = __all_sync(kFullMask, wait(a_full + 8 * b, (ti >> 1) & 1));
      if (!ok) break;
      const float alpha = alpha_s[b * TR + r];
      // The accumulator of a split's first tile is fresh: nothing to rescale.  Otherwise U is
      // rescaled unless alpha is exactly 1 for every row of the warp (u * 1 = u bit for bit;
      // with the lazy reference maximum that is the common case); it must be at rest for that:
      // PV of the previous tile done.
      if ((t % TPS) != 0 && t != T0 && !__all_sync(kFullMask, alpha == 1.0f)) {
        ok = __all_sync(kFullMask, wait(pv_done + 8 * ((ti - 1) & 1), ((ti - 1) >> 1) & 1));
        if (!ok) break;
        tc_fence_after();
#pragma unroll 1
        for (int cb = 0; cb < D; cb += 16) {
          uint32_t ur[16];
          tmem_ld16(tmem + lane_sel + Cfg::kColU + cb, ur);
          tmem_wait_ld();
          const uint64_t alpha2 = nc::pack2(alpha, alpha);
#pragma unroll
          for (int i = 0; i < 16; i += 2) {  // u * alpha, two lanes per instruction
            float u0, u1;
            nc::unpack2(nc::mul2(nc::pack2(__uint_as_float(ur[i]), __uint_as_float(ur[i + 1])), alpha2), u0, u1);
            ur[i] = __float_as_uint(u0);
            ur[i + 1] = __float_as_uint(u1);
          }
          tmem_st16(tmem + lane_sel + Cfg::kColU + cb, ur);
        }
        tmem_wait_st();
      }
      if (key0 + KT > n_eff || key0 <= lo_first) {
        // Value rows no row may see: at or beyond n_eff (not loaded, or pool garbage) in the tail
        // tile; before the window of the tile's first row (their pages may have been given back)
        // in the first tile under a sliding window.  Zero them: 0 * non-finite would poison U.
        ok = __all_sync(kFullMask, wait(v_full + 8 * s, (ti / NS) & 1));
        if (!ok) break;
        const uint32_t vst = kv_smem + s * Cfg::kStageBytes + Cfg::kKBytes;
        if (key0 + KT > n_eff) {
          const int first = n_eff - key0;
          const int per_half = (KT - first) * 8;
          for (int xx = r; xx < per_half * (D / 64); xx += TR) {
            const int half = xx / per_half, y = xx - half * per_half;
            const uint32_t addr = vst + half * (KT * 128) + (first + (y >> 3)) * 128 + ((y & 7) << 4);
            asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(addr), "r"(0u) : "memory");
          }
        }
        if (key0 <= lo_first) {
          const int per_half = min(KT, lo_first - key0 + 1) * 8;
          for (int xx = r; xx < per_half * (D / 64); xx += TR) {
            const int half = xx / per_half, y = xx - half * per_half;
            const uint32_t addr = vst + half * (KT * 128) + (y >> 3) * 128 + ((y & 7) << 4);
            asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(addr), "r"(0u) : "memory");
          }
        }
        fence_proxy_async();
      }
      tc_fence_before();
      mbar_arrive(p_full + 8 * b);

      // ---- end of a split -------------------------------------------------------------------
      if constexpr (PACKED) {
        if (t + 1 == n_tiles) {  // the split is complete: its raw (m, z, U) is the row's partial
          ok = __all_sync(kFullMask, wait(mz_full, 0));
          if (!ok) break;
          const float2 mz = mz_s[r];
          ok = __all_sync(kFullMask, wait(pv_done + 8 * b, (ti >> 1) & 1));
          if (!ok) break;
          tc_fence_after();
          if (valid) P.ws_mz[slab] = mz;
          float* pu = P.ws_u + slab * D;
#pragma unroll 1
          for (int cb = 0; cb < D; cb += 16) {
            uint32_t ur[16];
            tmem_ld16(tmem + lane_sel + Cfg::kColU + cb, ur);
            tmem_wait_ld();
            if (valid) {
#pragma unroll
              for (int i = 0; i < 16; i += 4)
                *reinterpret_cast<uint4*>(pu + cb + i) = make_uint4(ur[i], ur[i + 1], ur[i + 2], ur[i + 3]);
            }
          }
        }
      } else if ((t + 1) % TPS == 0 || t + 1 == n_tiles) {
        const int split = t / TPS;
        const int kb = (split - T0 / TPS) & 1, kuse = (split - T0 / TPS) >> 1;
        const bool resume = split > T0 / TPS;  // the CTA has stored a running result before
        const bool last = t + 1 == n_tiles;
        // The running-fold values do not depend on the PV in flight: request the first kFoldAhead
        // chunks of 16 columns now; a chunk's registers are refilled as soon as it has been used.
        constexpr int kFoldAhead = Cfg::kFoldAhead < D / 16 ? Cfg::kFoldAhead : D / 16;
        float4 uc4[4 * kFoldAhead];
        if (resume) {
#pragma unroll
          for (int i = 0; i < 4 * kFoldAhead; ++i) uc4[i] = __ldcg(ucg + static_cast<size_t>(i) * TR);
        }
        ok = __all_sync(kFullMask, wait(mz_full + 8 * kb, kuse & 1));
        if (!ok) break;
        const float2 mz = mz_s[kb * TR + r];
        ok = __all_sync(kFullMask, wait(pv_done + 8 * b, (ti >> 1) & 1));
        if (!ok) break;
        tc_fence_after();
        const bool take = split <= k_first;  // the row's first split: the running result starts from it
        const bool sees = p >= split * nc::kSplitLen;
        nc::FoldFactors f;
        f.a = 1.f;
        f.b = 0.f;
        if (take) {
          mc = mz.x;
          zc = mz.y;
        } else if (sees) {
          f = nc::fold_scalars(mc, zc, mz.x, mz.y);
        }
        const float inv = nc::out_scale(zc);  // used on the last split only
        if (last && valid && P.lse != nullptr)
          P.lse[static_cast<size_t>(rq.q_row0 + tok) * P.Hq + kvh * G + row % G] = nc::lse_value(mc, zc);
#pragma unroll
        for (int cb = 0; cb < D; cb += 16) {
          const int slot = ((cb / 16) % kFoldAhead) * 4;
          uint32_t ur[16];
          tmem_ld16(tmem + lane_sel + Cfg::kColU + cb, ur);
          tmem_wait_ld();
          float un[16];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float4 x = uc4[slot + i];
            const float u0 = __uint_as_float(ur[4 * i]), u1 = __uint_as_float(ur[4 * i + 1]);
            const float u2 = __uint_as_float(ur[4 * i + 2]), u3 = __uint_as_float(ur[4 * i + 3]);
            un[4 * i] = take ? u0 : (sees ? nc::fold_u(x.x, u0, f) : x.x);
            un[4 * i + 1] = take ? u1 : (sees ? nc::fold_u(x.y, u1, f) : x.y);
            un[4 * i + 2] = take ? u2 : (sees ? nc::fold_u(x.z, u2, f) : x.z);
            un[4 * i + 3] = take ? u3 : (sees ? nc::fold_u(x.w, u3, f) : x.w);
          }
          if (resume && cb / 16 + kFoldAhead < D / 16) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
              uc4[slot + i] = __ldcg(ucg + static_cast<size_t>((cb / 16 + kFoldAhead) * 4 + i) * TR);
          }
          if (last) {
            if (valid) {
#pragma unroll
              for (int i = 0; i < 16; i += 8) {
                uint32_t o[4];
#pragma unroll
                for (int xx = 0; xx < 4; ++xx) {
                  __nv_bfloat162 t2 = __floats2bfloat162_rn(nc::out_value(un[i + 2 * xx], inv),
                                                            nc::out_value(un[i + 2 * xx + 1], inv));
                  o[xx] = *reinterpret_cast<uint32_t*>(&t2);
                }
                *reinterpret_cast<uint4*>(dst + cb + i) = make_uint4(o[0], o[1], o[2], o[3]);
              }
            }
          } else {
#pragma unroll
            for (int i = 0; i < 4; ++i)
              __stcg(ucg + static_cast<size_t>(cb / 4 + i) * TR, make_float4(un[4 * i], un[4 * i + 1], un[4 * i + 2], un[4 * i + 3]));
          }
        }
      }
    }
  }

  // Common exit: every role ends here, also after a timeout, so tensor memory is always released.
  tc_fence_before();
  __syncthreads();
  if (P.beside_split && tid == 0) griddep_wait();  // this grid is not complete before the one beside it is
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(Cfg::kTmemCols));
}

}  // namespace vosti
