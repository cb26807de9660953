// Batch-invariant linear layer (tcgen05.mma + TMA, persistent, warp-specialised)
// and RMS normalisation for sm_100a: include/vosti_linear.h.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "../../include/vosti_linear.h"
#include "ptx.cuh"
#include "tcgen05.cuh"

namespace vosti {
namespace {

__device__ uint32_t g_linear_status;  // bit 0: a bounded wait gave up

template <int BN>
struct LinearCfg {
  static constexpr int kBM = 128, kBK = 64;
  static constexpr int kStages = BN == 256 ? 4 : 6;
  static constexpr int kABytes = kBM * kBK * 2;   // [row][128 B], 128-byte swizzle
  static constexpr int kBBytes = BN * kBK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kEpiWarps = BN / 32;       // an epilogue thread owns 128 columns of one row
  static constexpr int kThreads = 64 + 32 * kEpiWarps;  // TMA warp, MMA warp, epilogue warps
  static constexpr int kSmemBytes = kStages * kStageBytes + 256 + 1024;
  static constexpr uint32_t kTmemCols = 2 * BN;   // two accumulators: the epilogue of a segment overlaps the next one's MMAs
};

// Frozen constants of the linear layer's numerics (hashed by vosti_linear_fingerprint).  The
// wave size is the SM count of a B200 taken as a NUMBER: it decides where segment sums are cut and
// must not follow the device the library happens to run on.
constexpr uint32_t kLinearVersion = 1;
constexpr int kSegmentWaveUnits = 148;      // (column tile, segment) units of one wave
constexpr int kSegmentMinBlocks = 16;       // a segment holds at least this many 64-wide K blocks (1024 elements)
constexpr uint32_t kRuleSegmentSum = 1;     // per segment: zero fp32 accumulator, chunks of 16 ascending; sums added left to right
constexpr int kMaxClusterSegments = 16;      // segments of a tile that a cluster can add (scheduling only)
constexpr uint32_t kRuleRmsNorm = 1;        // lane l adds its 16-byte vectors l, l+32, ... ascending with fma; butterfly; rsqrt.rn

// The K range of a weight is cut into `n_seg` segments of whole 64-wide blocks, a function of
// (N, K) alone; segment j covers blocks [j * B / n_seg, (j + 1) * B / n_seg).
struct Segments {
  int n_seg, k_blocks;
  __host__ __device__ int begin(int j) const { return static_cast<int>(static_cast<int64_t>(j) * k_blocks / n_seg); }
};
__host__ __device__ inline Segments segments_of(int64_t N, int64_t K) {
  const int k_blocks = static_cast<int>(K / 64);
  const int64_t col_tiles = N % 256 == 0 ? N / 256 : N / 128;  // columns of the widest instruction that divides N
  // as many (column tile, segment) units as fit one wave over the 148 SMs of a B200 when the batch
  // is a single row tile, but segments of at least 1024 elements: every segment costs the
  // large-batch schedule a pass over the accumulator
  int64_t want = kSegmentWaveUnits / col_tiles;
  const int64_t cap = k_blocks / kSegmentMinBlocks > 0 ? k_blocks / kSegmentMinBlocks : 1;
  if (want > cap) want = cap;
  if (want < 1) want = 1;
  return Segments{static_cast<int>(want), k_blocks};
}

// Tiles are numbered in bands of 16 row tiles, column tile by column tile inside a band, so that
// the CTAs running at the same time work on a block of about 16 x 9 tiles and both operands are
// re-read from L2 rather than from HBM.  The order in which tiles are visited has no influence
// on any output bit.
struct TileCoord {
  int m0, n0;
};
template <int BM, int BN>
__device__ __forceinline__ TileCoord tile_coord(int t, int m_tiles, int n_cols) {
  constexpr int kBand = 16;
  const int per_band = kBand * n_cols;
  const int band = t / per_band, in_band = t - band * per_band;
  const int first_m = band * kBand;
  const int rows = min(kBand, m_tiles - first_m);
  return TileCoord{(first_m + in_band % rows) * BM, (in_band / rows) * BN};
}

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// The address, in the cluster's shared window, of `addr` in the CTA of rank `rank`.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float4 ld_cluster_f4(uint32_t cluster_addr) {
  float4 v;
  // (ordered against the cluster barriers around its use by their own memory clobbers)
  asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
               : "r"(cluster_addr));
  return v;
}

// The numerical contract of an output element: for each segment of K a sum s_j that starts from
// a zero fp32 accumulator and takes the products in ascending K order (tcgen05.mma, K = 16 per
// instruction); then t = s_0, t = t + s_j for j = 1, 2, ... in fp32, round to nearest; then
// bf16(t).  Two schedules compute exactly that:
//   SPLIT = false: one CTA per SM walks output tiles and, inside a tile, the segments in order;
//     the epilogue threads keep t in registers and add each finished segment to it while the
//     MMAs of the next segment run into the other tensor-memory accumulator.
//   SPLIT = true (few row tiles, e.g. a decode batch): the unit of work is a (tile, segment)
//     pair, so that every SM streams a slice of the weight; s_j goes to a workspace and
//     linear_fold_kernel adds the segments in the same order.
//   SPLIT and CLUSTER (the same units, when a tile's segments number at most eight): the CTAs that
//     hold the segments of one tile form a cluster; each leaves its s_j in its own shared memory,
//     and after a cluster barrier CTA j adds, for its share of the tile's columns, s_0, s_1, ... in
//     that order out of the peers' shared memory and writes the bf16 result.  No workspace, no
//     second kernel, and the segment sums never travel through L2.
// Which one runs is a scheduling decision that may depend on M; the bits do not.
template <int BN, bool SPLIT, bool CLUSTER = false>
__global__ void __launch_bounds__(LinearCfg<BN>::kThreads, 1)
linear_kernel(const __grid_constant__ CUtensorMap x_map, const __grid_constant__ CUtensorMap w_map,
              __nv_bfloat16* __restrict__ y, float* __restrict__ seg_ws, int M, int N, int K) {
  using Cfg = LinearCfg<BN>;
  constexpr int NS = Cfg::kStages;
  constexpr uint32_t kAbortAfterNs = 1000000000u;
  // CLUSTER: a row of the CTA's segment sum in shared memory; the 16 bytes beyond BN floats keep
  // 16-byte accesses of consecutive rows on different banks
  constexpr uint32_t kPartRow = BN * 4 + 16;
  static_assert(!CLUSTER || 128 * kPartRow <= static_cast<uint32_t>(NS * Cfg::kStageBytes), "segment sum fits the stages");
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* sbase = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + NS * Cfg::kStageBytes;
  const uint32_t full = bars, empty = bars + 8 * NS, acc_full = bars + 16 * NS, acc_empty = acc_full + 16;
  volatile uint32_t* flags = reinterpret_cast<volatile uint32_t*>(sbase + NS * Cfg::kStageBytes + 192);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int m_tiles = (M + Cfg::kBM - 1) / Cfg::kBM;
  const int n_cols = N / BN;
  const int n_tiles = m_tiles * n_cols;
  const Segments seg = segments_of(N, K);
  // A step is one segment of one tile; a CTA's steps are numbered consecutively.  Without the
  // split a CTA owns whole tiles (steps tile-major); with it, single (tile, segment) units.
  const int n_units = SPLIT ? n_tiles * seg.n_seg : n_tiles;
  auto step_of = [&](int unit, int j, int& tile, int& sj) {
    if (SPLIT) {
      tile = unit / seg.n_seg;
      sj = unit - tile * seg.n_seg;
    } else {
      tile = unit;
      sj = j;
    }
  };
  constexpr int kStepsPerUnitSplit = 1;
  const int steps_per_unit = SPLIT ? kStepsPerUnitSplit : seg.n_seg;

  if (tid == 0) {
    for (int i = 0; i < NS; ++i) {
      mbar_init(full + 8 * i, 1);
      mbar_init(empty + 8 * i, 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(acc_full + 8 * i, 1);
      mbar_init(acc_empty + 8 * i, 32 * Cfg::kEpiWarps);
    }
    flags[0] = 0u;
    mbar_fence_init();
    tma_prefetch_desc(&x_map);
    tma_prefetch_desc(&w_map);
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(bars + 200),
                 "r"(Cfg::kTmemCols));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(sbase + NS * Cfg::kStageBytes + 200);

  // Bounded wait: gives up after ~1 s or as soon as another thread of the CTA has given up.
  auto wait = [&](uint32_t bar, uint32_t parity) -> bool {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    for (uint32_t it = 0;; ++it) {
      if (mbar_try_wait_hint(bar, parity, 2000u)) return true;
      if ((it & 63u) == 63u) {
        if (flags[0] != 0u) return false;
        if (global_timer_ns() - t0 > kAbortAfterNs) {
          flags[0] = 1u;
          atomicOr(&g_linear_status, 1u);
          return false;
        }
      }
    }
  };

  if (warp == 0) {
    // ================= TMA producer ==========================================================
    if (lane == 0) {
      griddep_wait();
      uint32_t it = 0;
      bool ok = true;
      for (int unit = blockIdx.x; unit < n_units && ok; unit += gridDim.x) {
        for (int j = 0; j < steps_per_unit && ok; ++j) {
          int tile, sj;
          step_of(unit, j, tile, sj);
          const TileCoord tc = tile_coord<Cfg::kBM, BN>(tile, m_tiles, n_cols);
          for (int kb = seg.begin(sj); kb < seg.begin(sj + 1); ++kb, ++it) {
            const uint32_t s = it % NS, use = it / NS;
            if (use > 0) ok = wait(empty + 8 * s, (use - 1) & 1);
            if (!ok) break;
            const uint32_t dst = base + s * Cfg::kStageBytes;
            mbar_expect_tx(full + 8 * s, Cfg::kStageBytes);
            tma_load_2d(dst, &x_map, kb * Cfg::kBK, tc.m0, full + 8 * s);  // rows beyond M arrive as zeros
            tma_load_2d(dst + Cfg::kABytes, &w_map, kb * Cfg::kBK, tc.n0, full + 8 * s);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ================= MMA issuer ============================================================
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc(128, BN, false);
      uint32_t it = 0, step = 0;
      bool ok = true;
      for (int unit = blockIdx.x; unit < n_units && ok; unit += gridDim.x) {
        for (int j = 0; j < steps_per_unit && ok; ++j, ++step) {
          int tile, sj;
          step_of(unit, j, tile, sj);
          const uint32_t buf = step & 1, acc_use = step >> 1;
          if (acc_use > 0) ok = wait(acc_empty + 8 * buf, (acc_use - 1) & 1);  // the epilogue has drained this accumulator
          if (!ok) break;
          tc_fence_after();
          const int kb0 = seg.begin(sj), kb1 = seg.begin(sj + 1);
          for (int kb = kb0; kb < kb1; ++kb, ++it) {
            const uint32_t s = it % NS;
            ok = wait(full + 8 * s, (it / NS) & 1);
            if (!ok) break;
            tc_fence_after();
            const uint32_t a = base + s * Cfg::kStageBytes, b = a + Cfg::kABytes;
#pragma unroll
            for (int kc = 0; kc < Cfg::kBK / 16; ++kc)
              tc_mma_ss(tmem + buf * BN, smem_desc_sw128(a + kc * 32, 16, 1024),
                        smem_desc_sw128(b + kc * 32, 16, 1024), idesc, (kb > kb0 || kc > 0) ? 1u : 0u);
            tc_commit(empty + 8 * s);
          }
          if (!ok) break;
          tc_commit(acc_full + 8 * buf);
        }
      }
    }
  } else {
    // ================= epilogue: a thread owns 128 columns of one row of the tile ===============
    const int e = warp - 2;
    const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const int r = (warp & 3) * 32 + lane;   // row of the tile = tensor-memory lane
    const int c0 = (e >> 2) * 128;          // first of the thread's columns
    float total[128];
    uint32_t step = 0;
    bool ok = true;
    for (int unit = blockIdx.x; unit < n_units && ok; unit += gridDim.x) {
      for (int j = 0; j < steps_per_unit && ok; ++j, ++step) {
        int tile, sj;
        step_of(unit, j, tile, sj);
        const uint32_t buf = step & 1;
        const TileCoord tc = tile_coord<Cfg::kBM, BN>(tile, m_tiles, n_cols);
        ok = __all_sync(0xffffffffu, wait(acc_full + 8 * buf, (step >> 1) & 1));
        if (!ok) break;
        tc_fence_after();
        const bool in_range = tc.m0 + r < M;
        if constexpr (SPLIT && CLUSTER) {
          // s_j of this unit -> this CTA's shared memory, [row][BN] fp32 with rows kPartRow bytes apart
          // (the pipeline stages are idle: the unit's MMAs are done, and the CTA has no other unit)
          const uint32_t dst = base + r * kPartRow + c0 * 4;
          const bool warp_live = tc.m0 + (warp & 3) * 32 < M;  // else: rows beyond M, never read
#pragma unroll 1
          for (int cb = 0; cb < 128 && warp_live; cb += 32) {
            uint32_t v[32];
            tmem_ld32(tmem + lane_sel + buf * BN + c0 + cb, v);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; i += 4)
              asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(dst + (cb + i) * 4), "r"(v[i]), "r"(v[i + 1]),
                           "r"(v[i + 2]), "r"(v[i + 3])
                           : "memory");
          }
        } else if (SPLIT) {
          // s_j of this unit -> workspace [column tile][segment][row][BN]
          float* dst = seg_ws + ((static_cast<size_t>(tc.n0 / BN) * seg.n_seg + sj) * M + (tc.m0 + r)) * BN + c0;
#pragma unroll 1
          for (int cb = 0; cb < 128; cb += 32) {
            uint32_t v[32];
            tmem_ld32(tmem + lane_sel + buf * BN + c0 + cb, v);
            tmem_wait_ld();
            if (cb + 32 == 128) {
              tc_fence_before();
              mbar_arrive(acc_empty + 8 * buf);
            }
            if (in_range) {
#pragma unroll
              for (int i = 0; i < 32; i += 4)
                *reinterpret_cast<uint4*>(dst + cb + i) = make_uint4(v[i], v[i + 1], v[i + 2], v[i + 3]);
            }
          }
        } else {
#pragma unroll
          for (int cb = 0; cb < 128; cb += 32) {
            uint32_t v[32];
            tmem_ld32(tmem + lane_sel + buf * BN + c0 + cb, v);
            tmem_wait_ld();
            if (cb + 32 == 128) {  // the accumulator is in registers: hand it back
              tc_fence_before();
              mbar_arrive(acc_empty + 8 * buf);
            }
            if (sj == 0) {
#pragma unroll
              for (int i = 0; i < 32; ++i) total[cb + i] = __uint_as_float(v[i]);
            } else {
#pragma unroll
              for (int i = 0; i < 32; ++i) total[cb + i] = __fadd_rn(total[cb + i], __uint_as_float(v[i]));
            }
          }
          if (sj == seg.n_seg - 1 && in_range) {
            __nv_bfloat16* dst = y + static_cast<size_t>(tc.m0 + r) * N + tc.n0 + c0;
#pragma unroll
            for (int i = 0; i < 128; i += 8) {
              uint32_t o[4];
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                __nv_bfloat162 t2 = __floats2bfloat162_rn(total[i + 2 * q], total[i + 2 * q + 1]);
                o[q] = *reinterpret_cast<uint32_t*>(&t2);
              }
              *reinterpret_cast<uint4*>(dst + i) = make_uint4(o[0], o[1], o[2], o[3]);
            }
          }
        }
      }
    }
  }

  if constexpr (SPLIT && CLUSTER) {
    // Every thread of the cluster gets here, also after a wait has given up.  First barrier: the
    // segment sums of the tile are in the shared memory of the CTAs that computed them.
    cluster_sync_all();
    if (warp >= 2) {
      const int n = seg.n_seg;                       // = CTAs of the cluster; this CTA's rank = its segment
      const int j = static_cast<int>(cluster_ctarank());
      const int g_lo = j * (BN / 8) / n, g_hi = (j + 1) * (BN / 8) / n;  // this CTA's groups of eight columns
      const int cpr = 2 * (g_hi - g_lo);             // 16-byte chunks (four columns) per row of its share
      int tile, sj;
      step_of(blockIdx.x, 0, tile, sj);
      const TileCoord tc = tile_coord<Cfg::kBM, BN>(tile, m_tiles, n_cols);
      // Consecutive threads take consecutive chunks of a row: a warp's request to a peer's shared
      // memory is one contiguous piece (scattered 16-byte requests crawl), and so is its store.
      constexpr int kStride = 32 * Cfg::kEpiWarps, kBatch = 1;  // (more chunks in flight per thread measured slower)
      const int live = min(Cfg::kBM, M - tc.m0) * cpr;  // rows beyond M hold zeros nobody wants
      for (int idx0 = tid - 64; idx0 < live; idx0 += kBatch * kStride) {
        float4 a[kBatch][kMaxClusterSegments];  // every value is requested before the first is used
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
          const int idx = idx0 + u * kStride;
          if (idx < live) {
            const int row = idx / cpr, ch = idx - row * cpr;
            const uint32_t local = base + row * kPartRow + g_lo * 32 + ch * 16;
#pragma unroll
            for (int q = 0; q < kMaxClusterSegments; ++q)
              if (q < n) a[u][q] = ld_cluster_f4(map_to_cta(local, static_cast<uint32_t>(q)));
          }
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
          const int idx = idx0 + u * kStride;
          if (idx < live) {
            const int row = idx / cpr, ch = idx - row * cpr;
            float4 t = a[u][0];
#pragma unroll
            for (int q = 1; q < kMaxClusterSegments; ++q)  // t = s_0, then t + s_1, ... : the contract's order
              if (q < n) {
                t.x = __fadd_rn(t.x, a[u][q].x); t.y = __fadd_rn(t.y, a[u][q].y);
                t.z = __fadd_rn(t.z, a[u][q].z); t.w = __fadd_rn(t.w, a[u][q].w);
              }
            if (tc.m0 + row < M) {
              __nv_bfloat162 lo2 = __floats2bfloat162_rn(t.x, t.y), hi2 = __floats2bfloat162_rn(t.z, t.w);
              *reinterpret_cast<uint2*>(y + static_cast<size_t>(tc.m0 + row) * N + tc.n0 + g_lo * 8 + ch * 4) =
                  make_uint2(*reinterpret_cast<uint32_t*>(&lo2), *reinterpret_cast<uint32_t*>(&hi2));
            }
          }
        }
      }
    }
    cluster_sync_all();  // nobody reads this CTA's shared memory any more
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(Cfg::kTmemCols));
}

// ---- the same contract on CTA pairs -------------------------------------------------------------
// Two CTAs of a cluster (the two SMs of a TPC) compute one 256 x 256 tile with tcgen05.mma
// cta_group::2: each loads its own 128 rows of x and its own 128 of the tile's 256 weight rows,
// the pair's instruction reads both halves of the weight tile, and each SM's tensor memory
// receives its 128 rows of the result.  Per SM and K block that is 32 KB from L2 instead of 48 KB,
// so six stages fit where four did.  An output element is still the same chain of K = 16
// products in ascending K order, segment by segment: the bits are those of linear_kernel
// (tested), and which kernel runs is a scheduling decision.
struct PairCfg {
  static constexpr int kBM = 128, kBN = 256, kBK = 64;   // kBM: rows per CTA; the pair's tile is 256 x 256
  static constexpr int kStages = 6;
  static constexpr int kABytes = kBM * kBK * 2;
  static constexpr int kBBytes = (kBN / 2) * kBK * 2;    // this CTA's half of the weight tile
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kEpiWarps = 8;
  static constexpr int kThreads = 64 + 32 * kEpiWarps;
  static constexpr int kSmemBytes = kStages * kStageBytes + 256 + 1024;
  static constexpr uint32_t kTmemCols = 2 * kBN;
};

// TMA load into this CTA's shared memory whose bytes are counted on the leader CTA's mbarrier.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int32_t x, int32_t y,
                                                 uint32_t leader_bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(leader_bar)
      : "memory");
}
__device__ __forceinline__ void tc_mma_ss_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrive, once the pair's MMAs issued so far have completed, on the barrier at this offset in both CTAs.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
  const uint16_t both = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::
                   "r"(bar), "h"(both)
               : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(PairCfg::kThreads, 1)
linear_pair_kernel(const __grid_constant__ CUtensorMap x_map, const __grid_constant__ CUtensorMap w_map,
                   __nv_bfloat16* __restrict__ y, int M, int N, int K) {
  using Cfg = PairCfg;
  constexpr int NS = Cfg::kStages;
  constexpr int BN = Cfg::kBN;
  constexpr uint32_t kAbortAfterNs = 1000000000u;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* sbase = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + NS * Cfg::kStageBytes;
  // full, acc_empty: the leader's copies are used; empty, acc_full: each CTA's own
  const uint32_t full = bars, empty = bars + 8 * NS, acc_full = bars + 16 * NS, acc_empty = acc_full + 16;
  volatile uint32_t* flags = reinterpret_cast<volatile uint32_t*>(sbase + NS * Cfg::kStageBytes + 192);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int m_tiles = (M + 2 * Cfg::kBM - 1) / (2 * Cfg::kBM);
  const int n_cols = N / BN;
  const int n_tiles = m_tiles * n_cols;
  const Segments seg = segments_of(N, K);

  if (tid == 0) {
    for (int i = 0; i < NS; ++i) {
      mbar_init(full + 8 * i, 1);
      mbar_init(empty + 8 * i, 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(acc_full + 8 * i, 1);
      mbar_init(acc_empty + 8 * i, 2 * Cfg::kEpiWarps);  // one arrival per epilogue warp of either CTA
    }
    flags[0] = 0u;
    mbar_fence_init();
    tma_prefetch_desc(&x_map);
    tma_prefetch_desc(&w_map);
  }
  if (warp == 1) {  // the same warp of both CTAs, the same shared-memory offset
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(bars + 200),
                 "r"(Cfg::kTmemCols));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers exist before anything is sent to them
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(sbase + NS * Cfg::kStageBytes + 200);

  auto wait = [&](uint32_t bar, uint32_t parity) -> bool {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    for (uint32_t it = 0;; ++it) {
      if (mbar_try_wait_hint(bar, parity, 2000u)) return true;
      if ((it & 63u) == 63u) {
        if (flags[0] != 0u) return false;
        if (global_timer_ns() - t0 > kAbortAfterNs) {
          flags[0] = 1u;
          atomicOr(&g_linear_status, 1u);
          return false;
        }
      }
    }
  };

  if (warp == 0) {
    // ================= TMA producer (both CTAs) ==============================================
    if (lane == 0) {
      griddep_wait();
      uint32_t it = 0;
      bool ok = true;
      for (int tile = pair; tile < n_tiles && ok; tile += n_pairs) {
        const TileCoord tc = tile_coord<2 * Cfg::kBM, BN>(tile, m_tiles, n_cols);
        for (int kb = 0; kb < seg.k_blocks; ++kb, ++it) {
          const uint32_t s = it % NS, use = it / NS;
          if (use > 0) ok = wait(empty + 8 * s, (use - 1) & 1);
          if (!ok) break;
          const uint32_t dst = base + s * Cfg::kStageBytes;
          const uint32_t leader_full = map_to_cta(full + 8 * s, 0);
          if (rank == 0) mbar_expect_tx(full + 8 * s, 2 * Cfg::kStageBytes);  // both CTAs' bytes
          tma_load_2d_pair(dst, &x_map, kb * Cfg::kBK, tc.m0 + static_cast<int>(rank) * Cfg::kBM, leader_full);
          tma_load_2d_pair(dst + Cfg::kABytes, &w_map, kb * Cfg::kBK, tc.n0 + static_cast<int>(rank) * (BN / 2),
                           leader_full);
        }
      }
    }
  } else if (warp == 1) {
    // ================= MMA issuer (one thread of the leader CTA) ==============================
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = umma_idesc(2 * Cfg::kBM, BN, false);
      uint32_t it = 0, step = 0;
      bool ok = true;
      for (int tile = pair; tile < n_tiles && ok; tile += n_pairs) {
        for (int sj = 0; sj < seg.n_seg && ok; ++sj, ++step) {
          const uint32_t buf = step & 1, acc_use = step >> 1;
          if (acc_use > 0) ok = wait(acc_empty + 8 * buf, (acc_use - 1) & 1);  // both epilogues have drained it
          if (!ok) break;
          tc_fence_after();
          const int kb0 = seg.begin(sj), kb1 = seg.begin(sj + 1);
          for (int kb = kb0; kb < kb1; ++kb, ++it) {
            const uint32_t s = it % NS;
            ok = wait(full + 8 * s, (it / NS) & 1);
            if (!ok) break;
            tc_fence_after();
            const uint32_t a = base + s * Cfg::kStageBytes, b = a + Cfg::kABytes;
#pragma unroll
            for (int kc = 0; kc < Cfg::kBK / 16; ++kc)
              tc_mma_ss_pair(tmem + buf * BN, smem_desc_sw128(a + kc * 32, 16, 1024),
                             smem_desc_sw128(b + kc * 32, 16, 1024), idesc, (kb > kb0 || kc > 0) ? 1u : 0u);
            tc_commit_pair(empty + 8 * s);
          }
          if (!ok) break;
          tc_commit_pair(acc_full + 8 * buf);
        }
      }
    }
  } else {
    // ================= epilogue (both CTAs): a thread owns 128 columns of one of its CTA's rows =
    const int e = warp - 2;
    const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const int r = (warp & 3) * 32 + lane;
    const int c0 = (e >> 2) * 128;
    float total[128];
    uint32_t step = 0;
    bool ok = true;
    for (int tile = pair; tile < n_tiles && ok; tile += n_pairs) {
      const TileCoord tc = tile_coord<2 * Cfg::kBM, BN>(tile, m_tiles, n_cols);
      const int row = tc.m0 + static_cast<int>(rank) * Cfg::kBM + r;
      for (int sj = 0; sj < seg.n_seg && ok; ++sj, ++step) {
        const uint32_t buf = step & 1;
        ok = __all_sync(0xffffffffu, wait(acc_full + 8 * buf, (step >> 1) & 1));
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int cb = 0; cb < 128; cb += 32) {
          uint32_t v[32];
          tmem_ld32(tmem + lane_sel + buf * BN + c0 + cb, v);
          tmem_wait_ld();
          if (cb + 32 == 128) {  // the accumulator is in registers: hand it back to the issuer
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(acc_empty + 8 * buf, 0));
          }
          if (sj == 0) {
#pragma unroll
            for (int i = 0; i < 32; ++i) total[cb + i] = __uint_as_float(v[i]);
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) total[cb + i] = __fadd_rn(total[cb + i], __uint_as_float(v[i]));
          }
        }
        if (sj == seg.n_seg - 1 && row < M) {
          __nv_bfloat16* dst = y + static_cast<size_t>(row) * N + tc.n0 + c0;
#pragma unroll
          for (int i = 0; i < 128; i += 8) {
            uint32_t o[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              __nv_bfloat162 t2 = __floats2bfloat162_rn(total[i + 2 * q], total[i + 2 * q + 1]);
              o[q] = *reinterpret_cast<uint32_t*>(&t2);
            }
            *reinterpret_cast<uint4*>(dst + i) = make_uint4(o[0], o[1], o[2], o[3]);
          }
        }
      }
    }
  }

  // Neither CTA leaves while the other may still send to its barriers or read its shared memory.
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1)
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(Cfg::kTmemCols));
}

// The second half of the split schedule: y = bf16(((s_0 + s_1) + s_2) + ...), eight columns per thread.
__global__ void __launch_bounds__(256) linear_fold_kernel(const float* __restrict__ seg_ws,
                                                          __nv_bfloat16* __restrict__ y, int M, int N, int bn,
                                                          int n_seg) {
  griddep_wait();
  const int64_t idx = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) * 8;
  if (idx >= static_cast<int64_t>(M) * N) return;
  const int m = static_cast<int>(idx / N), n = static_cast<int>(idx - static_cast<int64_t>(m) * N);
  const int ct = n / bn, c = n - ct * bn;
  const float* src = seg_ws + ((static_cast<size_t>(ct) * n_seg) * M + m) * bn + c;
  const size_t seg_stride = static_cast<size_t>(M) * bn;
  float t[8];
  {
    const float4 a = *reinterpret_cast<const float4*>(src), b = *reinterpret_cast<const float4*>(src + 4);
    t[0] = a.x; t[1] = a.y; t[2] = a.z; t[3] = a.w; t[4] = b.x; t[5] = b.y; t[6] = b.z; t[7] = b.w;
  }
  for (int j = 1; j < n_seg; ++j) {
    const float4 a = *reinterpret_cast<const float4*>(src + j * seg_stride);
    const float4 b = *reinterpret_cast<const float4*>(src + j * seg_stride + 4);
    t[0] = __fadd_rn(t[0], a.x); t[1] = __fadd_rn(t[1], a.y); t[2] = __fadd_rn(t[2], a.z); t[3] = __fadd_rn(t[3], a.w);
    t[4] = __fadd_rn(t[4], b.x); t[5] = __fadd_rn(t[5], b.y); t[6] = __fadd_rn(t[6], b.z); t[7] = __fadd_rn(t[7], b.w);
  }
  uint32_t o[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    __nv_bfloat162 t2 = __floats2bfloat162_rn(t[2 * q], t[2 * q + 1]);
    o[q] = *reinterpret_cast<uint32_t*>(&t2);
  }
  *reinterpret_cast<uint4*>(y + idx) = make_uint4(o[0], o[1], o[2], o[3]);
}

// One warp per row.  Lane l adds the squares of its 8-element vectors l, l + 32, ... in
// ascending order (elements of a vector in ascending order), the 32 partial sums are
// combined by a butterfly (xor 16, 8, 4, 2, 1): the order depends on K only.
__global__ void __launch_bounds__(256) rmsnorm_kernel(const __nv_bfloat16* __restrict__ x,
                                                      const __nv_bfloat16* __restrict__ w,
                                                      __nv_bfloat16* __restrict__ y, int64_t M, int K, float eps) {
  griddep_wait();
  const int64_t row = static_cast<int64_t>(blockIdx.x) * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= M) return;
  const uint4* xr = reinterpret_cast<const uint4*>(x + row * K);
  const uint4* wr = reinterpret_cast<const uint4*>(w);
  uint4* yr = reinterpret_cast<uint4*>(y + row * K);
  const int nv = K / 8;
  float ss = 0.f;
  for (int i = lane; i < nv; i += 32) {
    const uint4 v = xr[i];
    const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u[j]));
      ss = __fmaf_rn(f.x, f.x, ss);
      ss = __fmaf_rn(f.y, f.y, ss);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss = __fadd_rn(ss, __shfl_xor_sync(0xffffffffu, ss, o));
  const float inv = __frsqrt_rn(__fadd_rn(__fdiv_rn(ss, static_cast<float>(K)), eps));
  for (int i = lane; i < nv; i += 32) {
    const uint4 v = xr[i], g = wr[i];
    const uint32_t u[4] = {v.x, v.y, v.z, v.w}, gw[4] = {g.x, g.y, g.z, g.w};
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u[j]));
      const float2 h = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&gw[j]));
      __nv_bfloat162 t2 = __floats2bfloat162_rn(__fmul_rn(__fmul_rn(f.x, inv), h.x), __fmul_rn(__fmul_rn(f.y, inv), h.y));
      o[j] = *reinterpret_cast<uint32_t*>(&t2);
    }
    yr[i] = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

// A [rows, K] bf16 row-major matrix as a 2-D tensor map with boxes of 64 columns x box_rows rows.
bool make_map(EncodeTiledFn fn, CUtensorMap* map, const void* ptr, int64_t rows, int64_t K, int box_rows) {
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(K), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(K) * 2};
  const cuuint32_t box[2] = {64, static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Workspace the split schedule needs: one fp32 [M, N] slab per segment.
size_t split_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  return sizeof(float) * static_cast<size_t>(segments_of(N, K).n_seg) * M * N;
}

// Whether spreading the segments over CTAs through the workspace is expected to beat whole tiles:
// rounds of K blocks on the busiest SM, plus what the segment sums cost on their way through the
// workspace and back, in units of the time of one 64-wide K block of a tile (about 0.4 us; the sums
// cost about one block time per 190,000 of their elements, fitted to the measurements below).  Measured on the Llama-3.1-8B
// shapes: 6144 x 4096 at 384 rows 32 us split, 29 us whole; 4096 x 14336 at 256 rows 46 us split,
// 93 us whole.  Scheduling only.
inline bool split_pays(int64_t M, int64_t N, int64_t tiles, const Segments& seg, int sm_count) {
  auto rounds = [&](int64_t units) { return (units + sm_count - 1) / sm_count; };
  const int64_t per_seg = (seg.k_blocks + seg.n_seg - 1) / seg.n_seg;
  const int64_t whole = rounds(tiles) * seg.k_blocks;
  const int64_t split = rounds(tiles * seg.n_seg) * per_seg + M * N * seg.n_seg / 190000;
  return split < whole;
}

template <int BN>
vosti_status launch_linear(EncodeTiledFn fn, const void* x, const void* w, void* y, int64_t M, int64_t N, int64_t K,
                           void* workspace, size_t workspace_bytes, int sm_count, cudaStream_t stream,
                           int schedule, bool use_pairs = false) {
  using Cfg = LinearCfg<BN>;
  static bool attr_set[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return VOSTI_ERR_CUDA;
  if (!attr_set[dev]) {
    if (cudaFuncSetAttribute(linear_kernel<BN, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             Cfg::kSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(linear_kernel<BN, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             Cfg::kSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(linear_kernel<BN, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             Cfg::kSmemBytes) != cudaSuccess ||
        // clusters of nine to sixteen CTAs (a tile with as many segments) are beyond the portable size
        cudaFuncSetAttribute(linear_kernel<BN, true, true>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) !=
            cudaSuccess)
      return VOSTI_ERR_CUDA;
    attr_set[dev] = true;
  }
  alignas(64) CUtensorMap x_map, w_map;
  if (!make_map(fn, &x_map, x, M, K, Cfg::kBM) || !make_map(fn, &w_map, w, N, K, BN)) return VOSTI_ERR_CUDA;
  const int64_t tiles = ((M + Cfg::kBM - 1) / Cfg::kBM) * (N / BN);
  const Segments seg = segments_of(N, K);
  __nv_bfloat16* yb = static_cast<__nv_bfloat16*>(y);
  // Scheduling only.  Few row tiles (whole tiles would leave most SMs idle): the segments of a tile
  // are spread over CTAs -- in clusters that add the segment sums themselves when a tile has at most
  // eight segments (the portable cluster size), else through the caller's workspace if there is one.
  // Many row tiles: CTA pairs when the caller's estimate favours them, else single CTAs.
  const bool few = tiles * 2 <= sm_count;
  const bool ws_ok = workspace != nullptr && workspace_bytes >= split_workspace_bytes(M, N, K) &&
                     reinterpret_cast<uintptr_t>(workspace) % 16 == 0;
  const bool cluster_ok = seg.n_seg > 1 && seg.n_seg <= kMaxClusterSegments;
  const bool pairs_ok = BN == 256 && sm_count >= 2;
  int sched = schedule;
  if (sched == VOSTI_LINEAR_AUTO) {
    // (clusters only when all of them fit the SMs at once: a second round of one-unit CTAs costs
    // more than the persistent workspace route's second round)
    // (and of the portable size: nine CTAs to a cluster were placed eight clusters at a time and took
    // 45 us where the workspace route takes 26-36, 4096 x 14336 at 1-128 rows)
    if (few && cluster_ok && seg.n_seg <= 8 && tiles * seg.n_seg <= (sm_count / seg.n_seg) * seg.n_seg)
      sched = VOSTI_LINEAR_SPLIT_CLUSTER;
    else if (seg.n_seg > 1 && ws_ok && split_pays(M, N, tiles, seg, sm_count)) sched = VOSTI_LINEAR_SPLIT_WORKSPACE;
    // (without a workspace the large clusters still halve the time of whole tiles at those sizes)
    else if (few && cluster_ok && tiles * seg.n_seg <= sm_count) sched = VOSTI_LINEAR_SPLIT_CLUSTER;
    else if (pairs_ok && use_pairs) sched = VOSTI_LINEAR_PAIRS;
    else sched = VOSTI_LINEAR_WHOLE_TILES;
  } else if ((sched == VOSTI_LINEAR_SPLIT_CLUSTER && !cluster_ok) ||
             (sched == VOSTI_LINEAR_SPLIT_WORKSPACE && !(seg.n_seg > 1 && ws_ok)) ||
             (sched == VOSTI_LINEAR_PAIRS && !pairs_ok)) {
    return VOSTI_ERR_UNSUPPORTED_CONFIG;
  }
  if (sched == VOSTI_LINEAR_SPLIT_CLUSTER) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(tiles * seg.n_seg));  // one cluster per tile, one CTA per segment
    cfg.blockDim = dim3(Cfg::kThreads);
    cfg.dynamicSmemBytes = Cfg::kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(seg.n_seg);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, linear_kernel<BN, true, true>, x_map, w_map, yb, static_cast<float*>(nullptr),
                           static_cast<int>(M), static_cast<int>(N), static_cast<int>(K)) == cudaSuccess)
      return VOSTI_OK;
    (void)cudaGetLastError();
    if (schedule != VOSTI_LINEAR_AUTO) return VOSTI_ERR_CUDA;
    // such clusters cannot be placed on this device: the other routes remain
    sched = (seg.n_seg > 1 && ws_ok) ? VOSTI_LINEAR_SPLIT_WORKSPACE : VOSTI_LINEAR_WHOLE_TILES;
  }
  const bool split = sched == VOSTI_LINEAR_SPLIT_WORKSPACE;
  if constexpr (BN == 256) {
    const int n_pairs = sm_count / 2;
    if (sched == VOSTI_LINEAR_PAIRS) {
      static bool pair_attr_set[64] = {};
      if (!pair_attr_set[dev]) {
        if (cudaFuncSetAttribute(linear_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 PairCfg::kSmemBytes) != cudaSuccess)
          return VOSTI_ERR_CUDA;
        pair_attr_set[dev] = true;
      }
      alignas(64) CUtensorMap w_half_map;  // this CTA's 128 of the tile's 256 weight rows
      if (!make_map(fn, &w_half_map, w, N, K, BN / 2)) return VOSTI_ERR_CUDA;
      linear_pair_kernel<<<2 * n_pairs, PairCfg::kThreads, PairCfg::kSmemBytes, stream>>>(
          x_map, w_half_map, yb, static_cast<int>(M), static_cast<int>(N), static_cast<int>(K));
      return cudaGetLastError() == cudaSuccess ? VOSTI_OK : VOSTI_ERR_CUDA;
    }
  }
  if (!split) {
    const int grid = static_cast<int>(tiles < sm_count ? tiles : sm_count);
    linear_kernel<BN, false><<<grid, Cfg::kThreads, Cfg::kSmemBytes, stream>>>(
        x_map, w_map, yb, nullptr, static_cast<int>(M), static_cast<int>(N), static_cast<int>(K));
  } else {
    const int64_t units = tiles * seg.n_seg;
    const int grid = static_cast<int>(units < sm_count ? units : sm_count);
    float* ws = static_cast<float*>(workspace);
    linear_kernel<BN, true><<<grid, Cfg::kThreads, Cfg::kSmemBytes, stream>>>(
        x_map, w_map, yb, ws, static_cast<int>(M), static_cast<int>(N), static_cast<int>(K));
    // the fold may be scheduled while the segment kernel drains; it waits for it on the device
    const int64_t threads = M * N / 8;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>((threads + 255) / 256));
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, linear_fold_kernel, static_cast<const float*>(ws), yb, static_cast<int>(M),
                           static_cast<int>(N), BN, seg.n_seg) != cudaSuccess)
      return VOSTI_ERR_CUDA;
  }
  return cudaGetLastError() == cudaSuccess ? VOSTI_OK : VOSTI_ERR_CUDA;
}

}  // namespace
}  // namespace vosti

using namespace vosti;

extern "C" {

vosti_status vosti_linear_tile_shape(int64_t N, int64_t K, int32_t* b_m, int32_t* b_n, int32_t* b_k) {
  if (N <= 0 || K <= 0 || N % 128 != 0 || K % 64 != 0 || N > INT32_MAX || K > INT32_MAX)
    return VOSTI_ERR_UNSUPPORTED_CONFIG;
  if (b_m) *b_m = 128;
  if (b_n) *b_n = N % 256 == 0 ? 256 : 128;
  if (b_k) *b_k = 64;
  return VOSTI_OK;
}

int32_t vosti_linear_contract(uint32_t* words, int32_t cap) {
  const uint32_t w[] = {kLinearVersion, 128u /* B_M */, 256u /* widest B_N */, 128u /* B_N otherwise */, 64u /* B_K */,
                        static_cast<uint32_t>(kSegmentWaveUnits), static_cast<uint32_t>(kSegmentMinBlocks),
                        kRuleSegmentSum, kRuleRmsNorm};
  const int32_t n = static_cast<int32_t>(sizeof w / sizeof w[0]);
  for (int32_t i = 0; i < n && i < cap && words; ++i) words[i] = w[i];
  return n;
}

uint64_t vosti_linear_fingerprint(void) {
  uint32_t w[16];
  const int32_t n = vosti_linear_contract(w, 16);
  uint64_t h = 1469598103934665603ull;
  for (int32_t i = 0; i < n; ++i)
    for (int b = 0; b < 8; ++b) {
      h ^= (static_cast<uint64_t>(w[i]) >> (8 * b)) & 0xff;
      h *= 1099511628211ull;
    }
  return h;
}

vosti_status vosti_linear_segments(int64_t N, int64_t K, int32_t* n_segments) {
  int32_t bn = 0;
  const vosti_status shape = vosti_linear_tile_shape(N, K, nullptr, &bn, nullptr);
  if (shape != VOSTI_OK) return shape;
  if (n_segments) *n_segments = segments_of(N, K).n_seg;
  return VOSTI_OK;
}

size_t vosti_linear_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  int32_t bn = 0;
  if (M <= 0 || vosti_linear_tile_shape(N, K, nullptr, &bn, nullptr) != VOSTI_OK) return 0;
  return split_workspace_bytes(M, N, K);
}

vosti_status vosti_linear(const void* x, const void* w, void* y, int64_t M, int64_t N, int64_t K, void* workspace,
                          size_t workspace_bytes, void* cuda_stream) {
  return vosti_linear_ex(x, w, y, M, N, K, workspace, workspace_bytes, VOSTI_LINEAR_AUTO, cuda_stream);
}

vosti_status vosti_linear_ex(const void* x, const void* w, void* y, int64_t M, int64_t N, int64_t K, void* workspace,
                             size_t workspace_bytes, int32_t schedule, void* cuda_stream) {
  if (schedule < VOSTI_LINEAR_AUTO || schedule > VOSTI_LINEAR_PAIRS) return VOSTI_ERR_INVALID_ARG;
  int32_t bn = 0;
  const vosti_status shape = vosti_linear_tile_shape(N, K, nullptr, &bn, nullptr);
  if (shape != VOSTI_OK) return shape;
  if (M < 0 || M > INT32_MAX) return VOSTI_ERR_INVALID_ARG;
  if (M == 0) return VOSTI_OK;
  if (!x || !w || !y) return VOSTI_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(w) | reinterpret_cast<uintptr_t>(y)) % 16)
    return VOSTI_ERR_INVALID_ARG;
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !p)
      return VOSTI_ERR_CUDA;
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  int dev = 0, sm_count = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return VOSTI_ERR_CUDA;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (bn != 256)
    return launch_linear<128>(fn, x, w, y, M, N, K, workspace, workspace_bytes, sm_count, stream, schedule);
  // Scheduling only (the bits are the same either way): CTA pairs when there is more than one
  // row tile, the pairs have at least three rounds of 256 x 256 tiles (below that a round of
  // single CTAs is measured to be as fast or faster), and their rounds, a little cheaper each,
  // do not take longer than the single CTAs' rounds of 128 x 256 tiles.
  const int64_t m128 = (M + 127) / 128, m256 = (M + 255) / 256;
  auto rounds = [](int64_t tiles, int64_t slots) { return (tiles + slots - 1) / slots; };
  const int64_t r_single = rounds(m128 * (N / 256), sm_count);
  const int64_t r_pair = sm_count >= 2 ? rounds(m256 * (N / 256), sm_count / 2) : 0;
  const bool use_pairs = M > 128 && r_pair >= 3 && 0.93 * static_cast<double>(r_pair) <= static_cast<double>(r_single);
  return launch_linear<256>(fn, x, w, y, M, N, K, workspace, workspace_bytes, sm_count, stream, schedule, use_pairs);
}

vosti_status vosti_rmsnorm(const void* x, const void* weight, void* y, int64_t M, int64_t K, float eps,
                           void* cuda_stream) {
  if (M < 0 || K <= 0 || K % 8 != 0 || K > INT32_MAX || !(eps >= 0.0f)) return VOSTI_ERR_INVALID_ARG;
  if (M == 0) return VOSTI_OK;
  if (!x || !weight || !y) return VOSTI_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(weight) | reinterpret_cast<uintptr_t>(y)) % 16)
    return VOSTI_ERR_INVALID_ARG;
  const int64_t grid = (M + 7) / 8;
  if (grid > INT32_MAX) return VOSTI_ERR_INVALID_ARG;
  rmsnorm_kernel<<<static_cast<int>(grid), 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      static_cast<const __nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(weight),
      static_cast<__nv_bfloat16*>(y), M, static_cast<int>(K), eps);
  return cudaGetLastError() == cudaSuccess ? VOSTI_OK : VOSTI_ERR_CUDA;
}

vosti_status vosti_linear_poll_status(void* cuda_stream) {
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  uint32_t word = 0, zero = 0;
  if (cudaStreamSynchronize(stream) != cudaSuccess ||
      cudaMemcpyFromSymbol(&word, g_linear_status, sizeof word) != cudaSuccess ||
      cudaMemcpyToSymbol(g_linear_status, &zero, sizeof zero) != cudaSuccess)
    return VOSTI_ERR_CUDA;
  return (word & 1u) ? VOSTI_ERR_TIMEOUT : VOSTI_OK;
}

}  // extern "C"
