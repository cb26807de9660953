// One key tile of the attention iteration for a 16-row group held by a warp:
// S = Q K^T, mask + online softmax, U += P V.  Every kernel that walks key
// tiles calls these same functions, so the per-row operation sequence -- and
// with it the output bits -- cannot differ between drivers.
//
// Fragment conventions (mma.sync m16n8k16, bf16 in, fp32 accumulate): lane l
// owns rows rho_a = l / 4 and rho_b = rho_a + 8 of the group and, in every
// 8-column tile, columns 2 (l % 4) and 2 (l % 4) + 1.
#pragma once
#include "nc_math.cuh"
#include "ptx.cuh"

namespace vosti {

constexpr unsigned kFullMask = 0xffffffffu;

// A stage holds the K rows or the V rows of SK consecutive keys of a tile
// (SK = 64: the whole tile, SK = 32: half of it) for one KV head, laid out as
// [half (64 elements)][key 0..SK-1][128 bytes] with the 128-byte swizzle
// (16-byte chunk index XOR key mod 8).
template <int D, int SK = nc::kKeyTile>
struct TileCfg {
  static constexpr int kStageKeys = SK;
  static constexpr int kParts = nc::kKeyTile / SK;          // stages per K (or V) tile
  static constexpr int kStageBytes = SK * D * 2;
  static constexpr int kHalfBytes = SK * 128;               // SK keys x 64 elements (128 B rows)
  static constexpr int kPageBytes = nc::kPageSize * 128;    // one TMA box: 16 keys x 64 elements
  static constexpr int kPagesPerStage = SK / nc::kPageSize;
  static constexpr int KC = D / 16;                         // head-dim chunks of 16
  static constexpr int NE = D / 8;                          // output column tiles of 8
  static constexpr int NT = nc::kKeyTile / 8;               // key column tiles of 8
};

// Address of the 16-byte chunk x (0 .. D/8-1) of key row `key` inside a stage.
//   PM = false ("half-major", written by 2 KB boxes of 64 elements x 16 rows):
//        [half][key 0..SK-1][128 B]            -- the canonical layout tcgen05 descriptors need
//   PM = true ("page-major", written by ONE 4 KB box per page covering both halves):
//        [page][half][16 rows][128 B]           -- half as many TMA instructions per stage
// Either way a 128-byte row is swizzled by its row index mod 8.
template <int D, int SK, bool PM>
__device__ __forceinline__ uint32_t stage_addr(uint32_t base, int key, int x) {
  if constexpr (PM)
    return base + (key >> 4) * (D * 32) + (x >> 3) * 2048 + (key & 15) * 128 + (((x & 7) ^ (key & 7)) << 4);
  else
    return base + (x >> 3) * (SK * 128) + key * 128 + (((x & 7) ^ (key & 7)) << 4);
}

// Per-thread view of its two rows.
struct RowPair {
  int p_a, p_b;       // logical positions (-1 for padding rows: they see nothing)
  int lo_a, lo_b;     // window lower bounds: key j is visible iff lo < j <= p
  float m_a, m_b;     // running maxima, scaled (base-two) domain
  float z_a, z_b;     // running normalisers
  __device__ __forceinline__ void reset() {
    m_a = m_b = -INFINITY;
    z_a = z_b = 0.f;
  }
};

// Query fragments of the two rows (A operand), straight from global memory.
template <int D>
__device__ __forceinline__ void load_q_frags(uint32_t (&qa)[D / 16][4], const __nv_bfloat16* row_a,
                                             const __nv_bfloat16* row_b, bool valid_a, bool valid_b,
                                             int quad) {
#pragma unroll
  for (int kc = 0; kc < D / 16; ++kc) {
    qa[kc][0] = valid_a ? *reinterpret_cast<const uint32_t*>(row_a + 16 * kc + 2 * quad) : 0u;
    qa[kc][1] = valid_b ? *reinterpret_cast<const uint32_t*>(row_b + 16 * kc + 2 * quad) : 0u;
    qa[kc][2] = valid_a ? *reinterpret_cast<const uint32_t*>(row_a + 16 * kc + 8 + 2 * quad) : 0u;
    qa[kc][3] = valid_b ? *reinterpret_cast<const uint32_t*>(row_b + 16 * kc + 8 + 2 * quad) : 0u;
  }
}

// S = Q K^T for the keys of one K stage: column tiles n0 .. n0 + SK/8 - 1 of the
// tile.  Head-dim chunks of 16 in ascending order.
template <int D, int SK, bool PM = false>
__device__ __forceinline__ void tile_scores(uint32_t ks, const uint32_t (&qa)[D / 16][4],
                                            float (&s)[8][4], int n0, int lane) {
  using C = TileCfg<D, SK>;
  constexpr int NN = SK / 8;
  const int lm_mat = lane >> 3, lm_row = lane & 7;
#pragma unroll
  for (int nn = 0; nn < NN; ++nn) s[n0 + nn][0] = s[n0 + nn][1] = s[n0 + nn][2] = s[n0 + nn][3] = 0.f;
  // Chunk pair outermost, column tile innermost: consecutive MMAs feed different
  // accumulators, so their latencies overlap.  Each accumulator still receives
  // its head-dim chunks in ascending order.
#pragma unroll
  for (int cp = 0; cp < C::KC / 2; ++cp) {
    uint32_t b[NN][4];
#pragma unroll
    for (int nn = 0; nn < NN; ++nn) {
      const int key = nn * 8 + lm_row;
      const int x = 4 * cp + lm_mat;
      ldsm_x4(stage_addr<D, SK, PM>(ks, key, x), b[nn][0], b[nn][1], b[nn][2], b[nn][3]);
    }
#pragma unroll
    for (int nn = 0; nn < NN; ++nn) mma_bf16_16816(s[n0 + nn], qa[2 * cp], b[nn][0], b[nn][1]);
#pragma unroll
    for (int nn = 0; nn < NN; ++nn) mma_bf16_16816(s[n0 + nn], qa[2 * cp + 1], b[nn][2], b[nn][3]);
  }
}

// Mask, online-softmax update of (m, z), rescale of U, and the bf16 weights as
// A-operand fragments (App. A iteration: G_hat, h, m_hat, alpha, A, z_hat,
// select on h).  key0 = first key of the tile.
//
// Two schedule-only switches, neither of which can change the bits of a real
// row: MASKED = false may be used when every key of the tile is visible to
// every real row of the group (the selects would all take the visible arm);
// UPPER = false when rows 8..15 of the group are all padding (their state is
// never stored; their weights are set to zero).  The rescale of U is skipped
// when alpha is exactly 1 for every row of the warp (u * 1 = u bit for bit).
template <int D, bool MASKED, bool UPPER>
__device__ __forceinline__ void tile_softmax(const float (&s)[8][4], int key0, float c, RowPair& r,
                                             float (&u)[D / 8][4], uint32_t (&pa)[4][4], int quad) {
  using C = TileCfg<D, nc::kKeyTile>;
  const bool h_a = !MASKED || (key0 <= r.p_a && key0 + nc::kKeyTile - 1 > r.lo_a);
  const bool h_b = !MASKED || (key0 <= r.p_b && key0 + nc::kKeyTile - 1 > r.lo_b);
  float mx_a = -INFINITY, mx_b = -INFINITY;
#pragma unroll
  for (int n = 0; n < C::NT; ++n) {
    const int j = key0 + n * 8 + 2 * quad;
    mx_a = fmaxf(mx_a, (!MASKED || (j <= r.p_a && j > r.lo_a)) ? s[n][0] : -INFINITY);
    mx_a = fmaxf(mx_a, (!MASKED || (j + 1 <= r.p_a && j + 1 > r.lo_a)) ? s[n][1] : -INFINITY);
    if (UPPER) {
      mx_b = fmaxf(mx_b, (!MASKED || (j <= r.p_b && j > r.lo_b)) ? s[n][2] : -INFINITY);
      mx_b = fmaxf(mx_b, (!MASKED || (j + 1 <= r.p_b && j + 1 > r.lo_b)) ? s[n][3] : -INFINITY);
    }
  }
  mx_a = fmaxf(mx_a, __shfl_xor_sync(kFullMask, mx_a, 1));
  mx_a = fmaxf(mx_a, __shfl_xor_sync(kFullMask, mx_a, 2));
  if (UPPER) {
    mx_b = fmaxf(mx_b, __shfl_xor_sync(kFullMask, mx_b, 1));
    mx_b = fmaxf(mx_b, __shfl_xor_sync(kFullMask, mx_b, 2));
  }
  const float mn_a = h_a ? nc::new_max(r.m_a, mx_a, c) : r.m_a;
  const float mn_b = (UPPER && h_b) ? nc::new_max(r.m_b, mx_b, c) : r.m_b;
  const float al_a = h_a ? nc::rescale(r.m_a, mn_a) : 1.0f;
  const float al_b = (UPPER && h_b) ? nc::rescale(r.m_b, mn_b) : 1.0f;
  const float ng_a = -mn_a, ng_b = -mn_b;
  float w_a[16], w_b[16];
#pragma unroll
  for (int n = 0; n < C::NT; ++n) {
    const int j = key0 + n * 8 + 2 * quad;
    w_a[2 * n] = (!MASKED || (j <= r.p_a && j > r.lo_a)) ? nc::weight(s[n][0], c, ng_a) : 0.f;
    w_a[2 * n + 1] = (!MASKED || (j + 1 <= r.p_a && j + 1 > r.lo_a)) ? nc::weight(s[n][1], c, ng_a) : 0.f;
    if (UPPER) {
      w_b[2 * n] = (!MASKED || (j <= r.p_b && j > r.lo_b)) ? nc::weight(s[n][2], c, ng_b) : 0.f;
      w_b[2 * n + 1] = (!MASKED || (j + 1 <= r.p_b && j + 1 > r.lo_b)) ? nc::weight(s[n][3], c, ng_b) : 0.f;
    } else {
      w_b[2 * n] = w_b[2 * n + 1] = 0.f;
    }
  }
  // Row sum: per half of the tile, this thread's pair (two chains), then the four pairs of the
  // row: xor 1 joins pairs (0,1) and (2,3), xor 2 joins those: (P0 + P1) + (P2 + P3); then
  // lower half + upper half.
  auto row_sum = [&](const float (&w)[16]) {
    float lo_h = nc::quad_partial<0>(w), hi_h = nc::quad_partial<1>(w);
    lo_h = __fadd_rn(lo_h, __shfl_xor_sync(kFullMask, lo_h, 1));
    hi_h = __fadd_rn(hi_h, __shfl_xor_sync(kFullMask, hi_h, 1));
    lo_h = __fadd_rn(lo_h, __shfl_xor_sync(kFullMask, lo_h, 2));
    hi_h = __fadd_rn(hi_h, __shfl_xor_sync(kFullMask, hi_h, 2));
    return nc::tile_total(lo_h, hi_h);
  };
  const float ps_a = row_sum(w_a);
  r.z_a = h_a ? nc::z_update(r.z_a, al_a, ps_a) : r.z_a;
  r.m_a = mn_a;
  if (UPPER) {
    const float ps_b = row_sum(w_b);
    r.z_b = h_b ? nc::z_update(r.z_b, al_b, ps_b) : r.z_b;
    r.m_b = mn_b;
  }
  if (!__all_sync(kFullMask, al_a == 1.0f && al_b == 1.0f)) {
#pragma unroll
    for (int e = 0; e < C::NE; ++e) {
      u[e][0] = nc::u_rescale(u[e][0], al_a);
      u[e][1] = nc::u_rescale(u[e][1], al_a);
      if (UPPER) {
        u[e][2] = nc::u_rescale(u[e][2], al_b);
        u[e][3] = nc::u_rescale(u[e][3], al_b);
      }
    }
  }
#pragma unroll
  for (int kc = 0; kc < C::NT / 2; ++kc) {
    __nv_bfloat162 t0 = __floats2bfloat162_rn(w_a[4 * kc], w_a[4 * kc + 1]);
    __nv_bfloat162 t2 = __floats2bfloat162_rn(w_a[4 * kc + 2], w_a[4 * kc + 3]);
    pa[kc][0] = *reinterpret_cast<uint32_t*>(&t0);
    pa[kc][2] = *reinterpret_cast<uint32_t*>(&t2);
    if (UPPER) {
      __nv_bfloat162 t1 = __floats2bfloat162_rn(w_b[4 * kc], w_b[4 * kc + 1]);
      __nv_bfloat162 t3 = __floats2bfloat162_rn(w_b[4 * kc + 2], w_b[4 * kc + 3]);
      pa[kc][1] = *reinterpret_cast<uint32_t*>(&t1);
      pa[kc][3] = *reinterpret_cast<uint32_t*>(&t3);
    } else {
      pa[kc][1] = pa[kc][3] = 0u;
    }
  }
}

// Picks the cheapest variant that is exact for this tile.  `all_visible`: every
// key of the tile is visible to every real row; `upper_rows`: some row 8..15 is real.
template <int D>
__device__ __forceinline__ void tile_softmax_dispatch(const float (&s)[8][4], int key0, float c, RowPair& r,
                                                      float (&u)[D / 8][4], uint32_t (&pa)[4][4], int quad,
                                                      bool all_visible, bool upper_rows) {
  if (all_visible) {
    if (upper_rows) tile_softmax<D, false, true>(s, key0, c, r, u, pa, quad);
    else tile_softmax<D, false, false>(s, key0, c, r, u, pa, quad);
  } else {
    if (upper_rows) tile_softmax<D, true, true>(s, key0, c, r, u, pa, quad);
    else tile_softmax<D, true, false>(s, key0, c, r, u, pa, quad);
  }
}

// Value rows no real row of the group can see must not reach the PV product as
// they are: a zero weight times a non-finite value would poison the row (the
// paper's zero-padded out-of-range loads).  Two cases: the tail of a request
// (rows at or beyond n_eff were not loaded, or hold whatever the pool had) and,
// under a sliding window, the rows of the first tile that lie before the window
// of the group's first row (their pages may have been given back by the caller).
// Clears rows [row_begin, row_end) of the stage.
template <int D, int SK, bool PM = false>
__device__ __forceinline__ void zero_value_rows(uint32_t vs, int row_begin, int row_end, int lane) {
  const int per_half = (row_end - row_begin) * 8;
  const int n_chunks = per_half * (D / 64);
  for (int x = lane; x < n_chunks; x += 32) {
    const int half = x / per_half;
    const int y = x - half * per_half;
    // every 16-byte chunk of the row is cleared, so the swizzle inside the row does not matter
    const uint32_t addr = stage_addr<D, SK, PM>(vs, row_begin + (y >> 3), half * 8 + (y & 7));
    asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(addr), "r"(0u) : "memory");
  }
  // These generic-proxy writes precede a later TMA (async-proxy) refill of the same stage.
  fence_proxy_async();
  __syncwarp();
}
template <int D, int SK, bool PM = false>
__device__ __forceinline__ void zero_value_tail(uint32_t vs, int first_bad_row, int lane) {
  zero_value_rows<D, SK, PM>(vs, first_bad_row, SK, lane);
}

// U += P V for the keys of one V stage: key chunks kc0 .. kc0 + SK/16 - 1 of the
// tile.  Per accumulator the chunks are applied in ascending order.
template <int D, int SK, bool PM = false>
__device__ __forceinline__ void tile_pv(uint32_t vs, const uint32_t (&pa)[4][4], float (&u)[D / 8][4],
                                        int kc0, int lane) {
  using C = TileCfg<D, SK>;
  const int lm_mat = lane >> 3, lm_row = lane & 7;
  // Key chunk outermost, output column tile innermost: consecutive MMAs feed
  // different accumulators; each accumulator gets its key chunks in ascending order.
#pragma unroll
  for (int kk = 0; kk < SK / 16; ++kk) {
#pragma unroll
    for (int e = 0; e < C::NE; e += 2) {
      const int key = kk * 16 + (lm_mat & 1) * 8 + lm_row;
      const int x = e + (lm_mat >> 1);
      uint32_t b0, b1, b2, b3;
      ldsm_x4_trans(stage_addr<D, SK, PM>(vs, key, x), b0, b1, b2, b3);
      mma_bf16_16816(u[e], pa[kc0 + kk], b0, b1);
      mma_bf16_16816(u[e + 1], pa[kc0 + kk], b2, b3);
    }
  }
}

// One TMA page gather: the K or V rows of `n_valid` pages (at most SK / 16) for
// one KV head into a stage; `ids` holds one page id per lane, `first_lane` the
// lane of the stage's first page.  Called by all lanes.  Lane 0 arms the
// barrier; then every box of the stage is issued by its own lane in ONE warp
// instruction (a thread needs on the order of a hundred cycles per TMA
// instruction, so issuing the boxes one after another from a single lane makes
// the issuing warp the bottleneck).
// PM = true: `map` is the 3-D map (64 elements, rows, halves) and one box brings a whole page chunk.
template <int D, int SK, bool PM = false>
__device__ __forceinline__ void issue_stage_load(const CUtensorMap* map, uint32_t dst, uint32_t bar,
                                                 int ids, int first_lane, int n_valid, int Hkv, int kvh,
                                                 int is_v, int lane) {
  using C = TileCfg<D, SK>;
  constexpr int HALVES = PM ? 1 : D / 64;
  constexpr int BOXES = C::kPagesPerStage * HALVES;
  if (lane == 0) mbar_expect_tx(bar, n_valid * nc::kPageSize * D * 2);
  const int j = lane / HALVES, h = lane % HALVES;  // page of the stage, 64-element half
  const int page = __shfl_sync(kFullMask, ids, first_lane + (lane < BOXES ? j : 0));
  __syncwarp();
  if (lane < BOXES && j < n_valid) {
    const int32_t y = ((page * Hkv + kvh) * 2 + is_v) * nc::kPageSize;
    if constexpr (PM)
      tma_load_3d(dst + j * (D * 32), map, 0, y, 0, bar);
    else
      tma_load_2d(dst + h * C::kHalfBytes + j * C::kPageBytes, map, h * 64, y, bar);
  }
}

}  // namespace vosti
