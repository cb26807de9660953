// Planning on the device, for steps that are replayed from a CUDA graph.
//
// The host planner reads the call's lengths and block tables on the CPU, which
// a captured graph cannot do: its metadata changes from replay to replay while
// the launch parameters stay what they were at capture.  Here the lengths, the
// start positions and the block tables live in device memory, and one CTA
// turns them into the records the attention kernels read -- per request
// (ReqMeta), per (row group, split) work item (SplitItem, longest first), per
// token (request, token) -- plus the counts the kernels bound their loops
// with.  Only split-parallel requests (decode, speculative queries) are
// planned this way.  The plan is a scheduling artefact: the same items as the
// host planner's, so the same partials, the same fold, the same bits.
#pragma once
#include "meta.cuh"
#include "nc_math.cuh"
#include "ptx.cuh"

namespace vosti {

// What a device plan holds, in this order, each part 16-byte aligned.
struct DevicePlanHeader {
  int32_t n_workers;        // split items x KV heads
  int32_t n_split_tokens;   // tokens the combine kernel finishes
  int32_t n_items;
  int32_t n_partial_rows;
  int32_t pad[12];
};
static_assert(sizeof(DevicePlanHeader) == 64, "header is one 64-byte record");

struct DevicePlanScratch {   // per request, between the two phases of the planner
  int32_t full_prefix;       // full-split items of the requests before this one
  int32_t part_rel[4];       // per row group, first and last split: index of that item within its bucket, or -1
  int32_t pad[3];
};

struct DevicePlanLayout {
  size_t off_reqs, off_items, off_toks, off_scratch, total;
  int64_t items_max, toks_max;
};
__host__ inline DevicePlanLayout device_plan_layout(int64_t max_batch, int64_t max_total_q, int64_t max_seq_len) {
  auto up = [](size_t x) { return (x + 15) & ~size_t{15}; };
  DevicePlanLayout L{};
  const int64_t k_max = (max_seq_len + nc::kSplitLen - 1) / nc::kSplitLen;
  L.items_max = max_batch * (nc::kSplitRowsMax / nc::kRowsPerGroup) * k_max;
  L.toks_max = max_total_q < max_batch * nc::kSplitRowsMax ? max_total_q : max_batch * nc::kSplitRowsMax;
  size_t at = sizeof(DevicePlanHeader);
  L.off_reqs = at; at += up(sizeof(ReqMeta) * max_batch);
  L.off_items = at; at += up(sizeof(SplitItem) * L.items_max);
  L.off_toks = at; at += up(sizeof(int2) * L.toks_max);
  L.off_scratch = at; at += up(sizeof(DevicePlanScratch) * max_batch);
  L.total = at;
  return L;
}

struct DevicePlanArgs {
  const int32_t* q_lens;        // device [batch]
  const int32_t* start_pos;     // device [batch]
  const int32_t* block_tables;  // device [batch][stride]
  int32_t stride, batch, max_q_len;
  int32_t G, Hkv, window;
  int64_t num_pages, max_seq_len, items_max, toks_max, part_rows_max;
  DevicePlanHeader* header;
  ReqMeta* reqs;
  SplitItem* items;
  int2* toks;
  DevicePlanScratch* scratch;
  uint32_t* status;
};

constexpr int kPlanThreads = 1024;   // at most; small batches are planned by 256 threads
constexpr int kPlanValues = 3 + nc::kTilesPerSplit;  // scanned per request, see device_plan_kernel

// Exclusive prefix sums of kPlanValues ints per thread over the CTA, all at once: a shuffle scan
// inside each warp, the warps' totals through shared memory, and every warp adds up the totals
// of the warps before it (and of all warps, for `total`) by itself.  Two barriers.
__device__ __forceinline__ void block_exclusive_scan(const int (&v)[kPlanValues], int (&pre)[kPlanValues],
                                                     int (&total)[kPlanValues], int (*warp_totals)[kPlanValues]) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
#pragma unroll
  for (int i = 0; i < kPlanValues; ++i) {
    int x = v[i];
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, x, d);
      if (lane >= d) x += y;
    }
    pre[i] = x - v[i];
    if (lane == 31) warp_totals[warp][i] = x;
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < kPlanValues; ++i) {
    const int t = lane < n_warps ? warp_totals[lane][i] : 0;
    int before = lane < warp ? t : 0, all = t;
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
      before += __shfl_xor_sync(0xffffffffu, before, d);
      all += __shfl_xor_sync(0xffffffffu, all, d);
    }
    pre[i] += before;
    total[i] = all;
  }
  __syncthreads();  // warp_totals is reused by the next chunk of requests
}

// The key tiles a 16-row group of a request walks: [t0, t1), t0 the tile of the first key its
// first row sees (0 without a sliding window).  Its items are the splits k0 .. k1 - 1; the first
// and the last may hold fewer than eight of those tiles, the ones between are full.
struct GroupSpan {
  int t0, t1, k0, k1;
  __device__ __forceinline__ int tiles_in(int k) const {
    return min(t1, (k + 1) * nc::kTilesPerSplit) - max(t0, k * nc::kTilesPerSplit);
  }
  // full-split items: [f0, f1)
  __device__ __forceinline__ int f0() const { return k0 + (tiles_in(k0) < nc::kTilesPerSplit ? 1 : 0); }
  __device__ __forceinline__ int f1() const {
    return max(f0(), k1 - ((k1 - 1 > k0 || tiles_in(k0) == nc::kTilesPerSplit) && tiles_in(k1 - 1) < nc::kTilesPerSplit ? 1 : 0));
  }
  // partial items: the first split if it is not full; the last split if it is another one and not full
  __device__ __forceinline__ bool first_partial() const { return tiles_in(k0) < nc::kTilesPerSplit; }
  __device__ __forceinline__ bool last_partial() const { return k1 - 1 > k0 && tiles_in(k1 - 1) < nc::kTilesPerSplit; }
};
__device__ __forceinline__ GroupSpan group_span(int st, int q, int G, int x, int window) {
  const int first_tok = (x * nc::kRowsPerGroup) / G;
  const int last_tok = min(q - 1, (x * nc::kRowsPerGroup + nc::kRowsPerGroup - 1) / G);
  GroupSpan sp;
  sp.t0 = nc::first_key(st + first_tok, window) / nc::kKeyTile;
  sp.t1 = (st + last_tok) / nc::kKeyTile + 1;
  sp.k0 = sp.t0 / nc::kTilesPerSplit;
  sp.k1 = (sp.t1 + nc::kTilesPerSplit - 1) / nc::kTilesPerSplit;
  return sp;
}

// A request as the planner accepts it: lengths outside the premises make it empty (and set
// the status bit), so that no later kernel reads or writes on its behalf.
__device__ __forceinline__ bool plan_request(const DevicePlanArgs& A, int r, int& q, int& st) {
  q = A.q_lens[r];
  st = A.start_pos[r];
  const int64_t n_eff = int64_t{st} + q;
  const bool ok = q >= 0 && st >= 0 && q <= A.max_q_len && int64_t{q} * A.G <= nc::kSplitRowsMax &&
                  n_eff <= A.max_seq_len && (n_eff + nc::kPageSize - 1) / nc::kPageSize <= A.stride;
  if (!ok) q = 0;
  return ok;
}

static __global__ void __launch_bounds__(kPlanThreads) device_plan_kernel(const DevicePlanArgs A) {
  constexpr int TPS = nc::kTilesPerSplit;
  // scanned per request: [0] tokens, [1] partial rows, [2] full-split items, [3 + t] row groups whose
  // last split has t tiles, t = 1..7 ([3] unused)
  constexpr int NV = kPlanValues;
  __shared__ int warp_totals[32][NV];
  __shared__ int bucket_base[TPS + 1];
  __shared__ int bad;
  // full_prefix of every request, for the binary searches of phase B2 (global scratch beyond 1024 requests)
  __shared__ int full_prefix_s[kPlanThreads];
  const bool prefix_in_smem = A.batch <= kPlanThreads;
  const int tid = threadIdx.x, n_threads = blockDim.x;
  if (tid == 0) bad = 0;
  griddep_wait();  // the metadata may come from a kernel earlier in the stream
  __syncthreads();

  // ---- phase A: per request counts, prefix sums, ReqMeta -------------------------------------
  int carry[NV];  // totals of the chunks of requests already scanned (the same in every thread)
#pragma unroll
  for (int i = 0; i < NV; ++i) carry[i] = 0;
  for (int r0 = 0; r0 < A.batch; r0 += n_threads) {
    const int r = r0 + tid;
    int q = 0, st = 0;
    int v[NV];
#pragma unroll
    for (int i = 0; i < NV; ++i) v[i] = 0;
    int part_bucket[4] = {0, 0, 0, 0};  // per group: tiles of its partial first / last split, 0 = none
    int first_split = 0, n_splits = 0;
    if (r < A.batch) {
      if (!plan_request(A, r, q, st)) bad = 1;
      if (q > 0) {
        const int rows = q * A.G;
        const int groups = (rows + nc::kRowsPerGroup - 1) / nc::kRowsPerGroup;
        first_split = nc::first_key(st, A.window) / nc::kSplitLen;
        n_splits = (st + q - 1) / nc::kSplitLen + 1 - first_split;
        v[0] = q;
        v[1] = A.Hkv * n_splits * rows;
#pragma unroll
        for (int x = 0; x < 2; ++x) {
          if (x >= groups) continue;
          const GroupSpan sp = group_span(st, q, A.G, x, A.window);
          v[2] += sp.f1() - sp.f0();
          if (sp.first_partial()) part_bucket[2 * x] = sp.tiles_in(sp.k0);
          if (sp.last_partial()) part_bucket[2 * x + 1] = sp.tiles_in(sp.k1 - 1);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int t = 1; t < TPS; ++t) v[3 + t] += part_bucket[i] == t ? 1 : 0;
      }
    }
    int pre[NV], total[NV];
    block_exclusive_scan(v, pre, total, warp_totals);
    if (r < A.batch) {
      ReqMeta m;
      m.q_row0 = carry[0] + pre[0];
      m.q_len = q;
      m.start = st;
      m.n_pages = q > 0 ? (st + q + nc::kPageSize - 1) / nc::kPageSize : 0;
      m.bt_off = r * A.stride;
      m.n_splits = n_splits;
      m.first_split = first_split;
      m.pad = 0;
      m.part_base = carry[1] + pre[1];
      A.reqs[r] = m;
      DevicePlanScratch s;
      s.full_prefix = carry[2] + pre[2];
      if (prefix_in_smem) full_prefix_s[r] = s.full_prefix;
      // a request's partial items that fall into one bucket follow one another there
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        s.part_rel[i] = -1;
        if (part_bucket[i] == 0) continue;
        int same_before = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) same_before += (j < i && part_bucket[j] == part_bucket[i]) ? 1 : 0;
#pragma unroll
        for (int t = 1; t < TPS; ++t)
          if (part_bucket[i] == t) s.part_rel[i] = carry[3 + t] + pre[3 + t] + same_before;
      }
      s.pad[0] = s.pad[1] = s.pad[2] = 0;
      A.scratch[r] = s;
      for (int i = 0; i < q; ++i)
        if (m.q_row0 + i < A.toks_max) A.toks[m.q_row0 + i] = make_int2(r, i);
    }
#pragma unroll
    for (int i = 0; i < NV; ++i) carry[i] += total[i];
  }
  __syncthreads();  // ReqMeta and scratch of every request are written; `bad` is final

  // ---- totals, capacity, bucket bases (longest first: full items, then 7-tile tails, ...) ------
  const int total_q = carry[0], part_rows = carry[1], n_full = carry[2];
  int n_items = n_full;
  for (int t = 1; t < TPS; ++t) n_items += carry[3 + t];
  const bool fits = total_q <= A.toks_max && n_items <= A.items_max && part_rows <= A.part_rows_max &&
                    part_rows >= 0 && n_items >= 0;
  if (tid == 0) {
    int o = n_full;
    bucket_base[TPS] = 0;
    for (int t = TPS - 1; t >= 1; --t) {
      bucket_base[t] = o;
      o += carry[3 + t];
    }
    DevicePlanHeader h = {};
    h.n_items = fits ? n_items : 0;
    h.n_workers = h.n_items * A.Hkv;
    h.n_split_tokens = fits ? total_q : 0;
    h.n_partial_rows = fits ? part_rows : 0;
    *A.header = h;
    if (bad || !fits) atomicOr(A.status, kStatusBadMetadata);
  }
  __syncthreads();
  if (!fits) return;

  auto make_item = [&](const ReqMeta& m, int r, int k, int x) {
    SplitItem si;
    si.q_row0 = m.q_row0;
    si.q_len = m.q_len;
    si.start = m.start;
    si.n_pages = m.n_pages;
    si.bt_index = m.bt_off + k * nc::kPagesPerSplit;
    si.split = k;
    si.row_group = x;
    si.n_splits = m.n_splits;
    si.part_base = m.part_base;
    si.req = r;
    si.first_split = m.first_split;
    return si;
  };

  // ---- phase B1: the last split of every row group, by bucket ---------------------------------
  for (int r = tid; r < A.batch; r += n_threads) {
    const ReqMeta m = A.reqs[r];
    if (m.q_len == 0) continue;
    const DevicePlanScratch s = A.scratch[r];
    const int groups = (m.q_len * A.G + nc::kRowsPerGroup - 1) / nc::kRowsPerGroup;
    for (int x = 0; x < groups; ++x) {
      const GroupSpan sp = group_span(m.start, m.q_len, A.G, x, A.window);
      if (s.part_rel[2 * x] >= 0)
        A.items[bucket_base[sp.tiles_in(sp.k0)] + s.part_rel[2 * x]] = make_item(m, r, sp.k0, x);
      if (s.part_rel[2 * x + 1] >= 0)
        A.items[bucket_base[sp.tiles_in(sp.k1 - 1)] + s.part_rel[2 * x + 1]] = make_item(m, r, sp.k1 - 1, x);
    }
  }
  // ---- phase B2: full-split items, one thread per item (request by binary search) --------------
  for (int j = tid; j < n_full; j += n_threads) {
    int lo = 0, hi = A.batch - 1;  // last request whose full_prefix <= j and that owns full items
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      const int at_mid = prefix_in_smem ? full_prefix_s[mid] : A.scratch[mid].full_prefix;
      if (at_mid <= j) lo = mid; else hi = mid - 1;
    }
    const int r = lo;
    const ReqMeta m = A.reqs[r];
    const int local = j - (prefix_in_smem ? full_prefix_s[r] : A.scratch[r].full_prefix);
    const int groups = (m.q_len * A.G + nc::kRowsPerGroup - 1) / nc::kRowsPerGroup;
    int fa[2] = {0, 0}, fb[2] = {0, 0};  // full-split items of the groups: [fa, fb)
    for (int x = 0; x < groups; ++x) {
      const GroupSpan sp = group_span(m.start, m.q_len, A.G, x, A.window);
      fa[x] = sp.f0();
      fb[x] = sp.f1();
    }
    int k, x;
    if (groups == 2 && fa[0] == fa[1]) {
      // split outermost, row group innermost, as the host planner orders them: the two groups
      // that read a split get neighbouring tickets
      const int both = min(fb[0], fb[1]) - fa[0];
      if (local < 2 * both) {
        k = fa[0] + (local >> 1);
        x = local & 1;
      } else {
        k = fa[0] + both + (local - 2 * both);
        x = fb[0] > fb[1] ? 0 : 1;
      }
    } else {  // one group, or ranges that start apart (a sliding window): group by group
      const int n0 = fb[0] - fa[0];
      x = local < n0 ? 0 : 1;
      k = x == 0 ? fa[0] + local : fa[1] + (local - n0);
    }
    A.items[j] = make_item(m, r, k, x);
  }
}

// KV append from a device plan: one warp per (request, token slot < max_q_len, KV head).
struct AppendPlannedParams {
  const __nv_bfloat16* k_new;
  const __nv_bfloat16* v_new;
  __nv_bfloat16* pool;
  const ReqMeta* reqs;
  const int32_t* block_tables;
  int32_t batch, max_q_len, Hkv;
  int64_t num_pages;
  uint32_t* status;
};
template <int D>
__global__ void __launch_bounds__(128) kv_append_planned_kernel(const AppendPlannedParams P) {
  const int lane = threadIdx.x & 31;
  const int64_t widx = static_cast<int64_t>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
  griddep_wait();  // the plan, and earlier readers of the pool
  if (widx >= static_cast<int64_t>(P.batch) * P.max_q_len * P.Hkv) return;
  const int kvh = static_cast<int>(widx % P.Hkv);
  const int i = static_cast<int>((widx / P.Hkv) % P.max_q_len);
  const int r = static_cast<int>(widx / (static_cast<int64_t>(P.Hkv) * P.max_q_len));
  const ReqMeta m = P.reqs[r];
  if (i >= m.q_len) return;
  const int pos = m.start + i;
  const int page = P.block_tables[static_cast<size_t>(m.bt_off) + pos / nc::kPageSize];
  if (page < 0 || page >= P.num_pages) {  // nothing is written through a page id outside the pool
    if (lane == 0) atomicOr(P.status, kStatusBadMetadata);
    return;
  }
  const int within = pos % nc::kPageSize;
  const int tok = m.q_row0 + i;
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
