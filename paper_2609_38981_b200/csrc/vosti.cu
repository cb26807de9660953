// libvosti: C ABI, host-side validation and work planning, kernel launches.
// Entry points are declared and documented in include/vosti.h.
#include <algorithm>
#include <chrono>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <utility>
#include <vector>

#include "attn_split.cuh"
#include "attn_tile.cuh"
#include "aux_kernels.cuh"
#include "device_plan.cuh"
#include "selftest_mma.cuh"

namespace vosti {
namespace {

constexpr int kHostSlots = 8;        // ring of pinned staging buffers
constexpr int kPackedTileRows = 128;  // rows of a packed tile: one CTA of the tile kernel
constexpr int64_t kTilePackMinRowSplits = 2048;  // rows x splits of such groups from which the extra launch pays
constexpr int kTilePackMinRows = 48;  // rows sharing a split from which packing goes through the tile kernel
constexpr int kHostSteps = 3;        // host-buffer steps that may be in flight (vosti_step_host_async)
constexpr size_t kAlign = 1024;
constexpr int kTileRows = 256;       // rows of one tile-kernel work item (16 row groups)

size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }

bool geometry_ok(const vosti_config& c) {
  if (c.head_dim != 64 && c.head_dim != 128) return false;
  if (c.page_size != nc::kPageSize) return false;
  if (c.n_q_heads <= 0 || c.n_kv_heads <= 0 || c.n_q_heads % c.n_kv_heads) return false;
  const int g = c.n_q_heads / c.n_kv_heads;
  if (g != 1 && g != 2 && g != 4 && g != 8 && g != 16) return false;
  if (c.num_pages <= 0 || c.max_batch <= 0 || c.max_total_q <= 0 || c.max_seq_len <= 0) return false;
  // TMA row coordinates are 32-bit: rows = pages * kv_heads * 2 * 16.
  if (c.num_pages * c.n_kv_heads >= (int64_t{1} << 26)) return false;
  if (c.max_seq_len >= (int64_t{1} << 30) || c.max_total_q >= (int64_t{1} << 27)) return false;
  return true;
}

// Sizes derived from the configuration alone.
struct Limits {
  int64_t k_max;         // splits of the longest sequence
  int64_t pages_max;     // page-table entries one call can carry
  int64_t items_max;
  int64_t part_rows_max;
  size_t meta_bytes;     // one metadata blob (attention or append)
  // workspace offsets
  size_t off_status, off_meta, off_part_u, off_part_mz, off_uc, off_stage, stage_q, stage_kv, total;
};

Limits limits_of(const vosti_config& c) {
  Limits L{};
  const int64_t G = c.n_q_heads / c.n_kv_heads;
  L.k_max = (c.max_seq_len + nc::kSplitLen - 1) / nc::kSplitLen;
  L.pages_max = int64_t{c.max_batch} * ((c.max_seq_len + nc::kPageSize - 1) / nc::kPageSize);
  const int64_t groups_split = (nc::kSplitRowsMax + nc::kRowsPerGroup - 1) / nc::kRowsPerGroup;
  const int64_t items_split = int64_t{c.max_batch} * groups_split * L.k_max;
  const int64_t items_seq = (c.max_total_q * G + kTileRows - 1) / kTileRows + c.max_batch;
  L.items_max = items_split + items_seq;
  const int64_t rows_by_batch = int64_t{c.max_batch} * nc::kSplitRowsMax;
  const int64_t rows_by_total = c.max_total_q * G;
  L.part_rows_max = std::min(rows_by_batch, rows_by_total) * c.n_kv_heads * L.k_max;
  // packed rows (shared-split packing only): 16 per packed item, and packing never adds items
  const int64_t packed_rows_max = (c.flags & VOSTI_FLAG_PACK_SHARED_SPLITS) ? 16 * items_split : 0;
  // packed tiles: a group that takes this route has at least kTilePackMinRows rows, so a tile of
  // kPackedTileRows records stands for at least kTilePackMinRows / 16 sixteen-row items
  const int64_t packed_tiles_max =
      (c.flags & VOSTI_FLAG_PACK_SHARED_SPLITS) ? items_split / (kTilePackMinRows / 16) + 1 : 0;
  const size_t attn_blob = align_up(sizeof(PackedRow) * packed_rows_max, 16) +
                           align_up(sizeof(PackedRow) * kPackedTileRows * packed_tiles_max, 16) +
                           align_up(sizeof(int4) * packed_tiles_max, 16) +
                           align_up(sizeof(ReqMeta) * c.max_batch, 16) +
                           align_up(sizeof(SplitItem) * items_split, 16) +
                           align_up(sizeof(vosti_work_item) * items_seq, 16) +
                           align_up(sizeof(int32_t) * L.pages_max, 16) +
                           align_up(sizeof(int2) * c.max_total_q, 16);
  const size_t append_blob = align_up(sizeof(int32_t) * c.max_total_q, 16);
  L.meta_bytes = align_up(std::max(attn_blob, append_blob));
  size_t at = 0;
  L.off_status = at; at += kAlign;
  L.off_meta = at; at += L.meta_bytes * kHostSlots;  // one region per staging slot
  L.off_part_u = at; at += align_up(sizeof(float) * L.part_rows_max * c.head_dim);
  L.off_part_mz = at; at += align_up(sizeof(float2) * L.part_rows_max);
  L.off_uc = at;  // running fold of the tile kernel: one 256-row fp32 tile per (item, KV head)
  at += align_up(sizeof(float) * items_seq * c.n_kv_heads * kTileRows * c.head_dim);
  const size_t qbytes = sizeof(__nv_bfloat16) * c.max_total_q * c.n_q_heads * c.head_dim;
  const size_t kbytes = sizeof(__nv_bfloat16) * c.max_total_q * c.n_kv_heads * c.head_dim;
  // staging of the host-buffer steps: one set of (q, out, k_new, v_new) per step in flight
  L.stage_q = align_up(qbytes);
  L.stage_kv = align_up(kbytes);
  L.off_stage = at; at += kHostSteps * (2 * L.stage_q + 2 * L.stage_kv);
  L.total = at;
  return L;
}

// A (request, complete split) pair that could share its split with other requests.
struct PackCand {
  uint64_t key;  // from the split's index and its first and last page id
  int32_t req, split;
};

struct Plan {
  std::vector<vosti_work_item> items;  // split-parallel items first
  std::vector<std::pair<int64_t, vosti_work_item>> seq_scratch;
  int64_t n_split = 0;
  int64_t n_partial_rows = 0;
};

// First key a row at position p sees under a sliding window w (0: no window).
inline int64_t first_visible_key(int64_t p, int64_t w) { return (w > 0 && p - w + 1 > 0) ? p - w + 1 : 0; }

// The plan of one request depends on its own (q_len, start), the window and the
// geometry.  A split-parallel item is one (16-row group, split) pair whose keys
// some row of the group sees: splits from the one holding the first visible key
// of the group's first row to the one holding the last row's position.  Items
// are ordered longest first (by key tiles walked): split-parallel items by an
// 8-bucket counting sort, sequential ones by a stable sort on the precomputed
// tile count, so the order is reproducible.
vosti_status plan_requests(const vosti_config& c, const int32_t* q_lens, const int32_t* start_pos,
                           const int32_t* seq_lens, int32_t batch, int32_t window, Plan* plan,
                           int64_t* part_base) {
  if (batch < 0 || window < 0 || (batch > 0 && (!q_lens || !start_pos || !seq_lens))) return VOSTI_ERR_INVALID_ARG;
  if (batch > c.max_batch) return VOSTI_ERR_OUT_OF_RANGE;
  const int G = c.n_q_heads / c.n_kv_heads;
  constexpr int TPS = nc::kTilesPerSplit;
  constexpr int kGroupsMax = nc::kSplitRowsMax / nc::kRowsPerGroup;
  // key tiles [t0, t1) a row group walks, and how many of them fall into split k
  struct Span {
    int64_t t0, t1;
    int64_t k0() const { return t0 / TPS; }
    int64_t k1() const { return (t1 + TPS - 1) / TPS; }
    int64_t tiles_in(int64_t k) const { return std::min(t1, (k + 1) * TPS) - std::max(t0, k * TPS); }
  };
  auto span_of = [&](int64_t st, int64_t q, int64_t first_row, int64_t n_rows) -> Span {
    const int64_t first_tok = first_row / G;
    const int64_t last_tok = std::min<int64_t>(q - 1, (first_row + n_rows - 1) / G);
    return Span{first_visible_key(st + first_tok, window) / nc::kKeyTile, (st + last_tok) / nc::kKeyTile + 1};
  };
  int64_t total_q = 0, n_split = 0, n_seq = 0, part_rows = 0;
  int64_t bucket[TPS + 1] = {0};  // bucket[t] = split items that walk t tiles
  // pass 1: premises, counts
  for (int r = 0; r < batch; ++r) {
    const int64_t q = q_lens[r], st = start_pos[r], n = seq_lens[r];
    if (q < 0 || st < 0 || st + q > n || n > c.max_seq_len) return VOSTI_ERR_OUT_OF_RANGE;
    total_q += q;
    if (q == 0) continue;
    const int64_t rows = q * G;
    const int64_t groups = (rows + nc::kRowsPerGroup - 1) / nc::kRowsPerGroup;
    if (rows <= nc::kSplitRowsMax) {
      if (part_base) part_base[r] = part_rows;
      const int64_t first_split = first_visible_key(st, window) / nc::kSplitLen;
      part_rows += int64_t{c.n_kv_heads} * ((st + q - 1) / nc::kSplitLen + 1 - first_split) * rows;
      for (int64_t g = 0; g < groups; ++g) {
        const Span sp = span_of(st, q, g * nc::kRowsPerGroup, nc::kRowsPerGroup);
        const int64_t k0 = sp.k0(), k1 = sp.k1();
        bucket[sp.tiles_in(k0)] += 1;
        if (k1 - k0 >= 2) {
          bucket[sp.tiles_in(k1 - 1)] += 1;
          bucket[TPS] += k1 - k0 - 2;
        }
        n_split += k1 - k0;
      }
    } else {
      if (part_base) part_base[r] = 0;
      n_seq += (rows + kTileRows - 1) / kTileRows;
    }
  }
  if (total_q > c.max_total_q) return VOSTI_ERR_OUT_OF_RANGE;
  plan->items.resize(static_cast<size_t>(n_split + n_seq));
  plan->seq_scratch.clear();
  int64_t at[TPS + 1];
  {
    int64_t o = 0;
    for (int t = TPS; t >= 1; --t) {
      at[t] = o;
      o += bucket[t];
    }
  }
  // pass 2: fill
  vosti_work_item* out = plan->items.data();
  for (int r = 0; r < batch; ++r) {
    const int64_t q = q_lens[r], st = start_pos[r];
    if (q == 0) continue;
    const int64_t rows = q * G;
    const bool split_parallel = rows <= nc::kSplitRowsMax;
    // split-parallel requests: one item per (16-row group, split); others: one per 256-row tile
    const int64_t rows_per_item = split_parallel ? nc::kRowsPerGroup : kTileRows;
    const int n_row_items = static_cast<int>((rows + rows_per_item - 1) / rows_per_item);
    if (split_parallel) {
      // Split outermost, row group innermost: the (at most two) row groups that read the
      // same split get neighbouring tickets, run at about the same time on different SMs,
      // and the second read of the split's K/V is served by L2 instead of HBM.
      Span sp[kGroupsMax];
      int64_t k_lo = INT64_MAX, k_hi = 0;
      for (int x = 0; x < n_row_items; ++x) {
        sp[x] = span_of(st, q, int64_t{x} * rows_per_item, rows_per_item);
        k_lo = std::min(k_lo, sp[x].k0());
        k_hi = std::max(k_hi, sp[x].k1());
      }
      for (int64_t k = k_lo; k < k_hi; ++k)
        for (int x = 0; x < n_row_items; ++x)
          if (k >= sp[x].k0() && k < sp[x].k1())
            out[at[sp[x].tiles_in(k)]++] = {r, x, static_cast<int32_t>(k), static_cast<int32_t>(k + 1)};
    } else {
      for (int x = 0; x < n_row_items; ++x) {
        const Span sp = span_of(st, q, int64_t{x} * rows_per_item, rows_per_item);
        const int first_group = x * (kTileRows / nc::kRowsPerGroup);
        plan->seq_scratch.push_back({sp.t1 - sp.t0, vosti_work_item{r, first_group, static_cast<int32_t>(sp.k0()),
                                                                    static_cast<int32_t>(sp.k1())}});
      }
    }
  }
  std::stable_sort(plan->seq_scratch.begin(), plan->seq_scratch.end(),
                   [](const auto& a, const auto& b) { return a.first > b.first; });
  for (size_t i = 0; i < plan->seq_scratch.size(); ++i) out[n_split + i] = plan->seq_scratch[i].second;
  plan->n_split = n_split;
  plan->n_partial_rows = part_rows;
  return VOSTI_OK;
}

uint64_t fnv1a(uint64_t h, uint64_t x) {
  for (int i = 0; i < 8; ++i) {
    h ^= (x >> (8 * i)) & 0xff;
    h *= 1099511628211ull;
  }
  return h;
}

// One staging slot: a pinned host buffer, its own device metadata region, an
// event for "copy done" and one for "kernels that read the region are done".
struct HostSlot {
  uint8_t* pinned = nullptr;
  uint8_t* device = nullptr;
  cudaEvent_t copied = nullptr;
  cudaEvent_t released = nullptr;
  bool in_flight = false;
  bool has_release = false;
};

// One host-buffer step in flight: its staging set in the workspace and the three
// points of its life (inputs on the device, kernels done, output on the host).
struct HostStep {
  cudaEvent_t in_done = nullptr;
  cudaEvent_t computed = nullptr;
  cudaEvent_t out_done = nullptr;
  int64_t ticket = -1;  // -1: nothing pending in this set
};

}  // namespace
}  // namespace vosti

using namespace vosti;

struct vosti_ctx {
  vosti_config cfg;
  Limits lim;
  int device = 0;
  int sm_count = 1;
  alignas(64) CUtensorMap kv_map;    // 2-D: (d, rows), box 64 x 16: half-major stages (tile kernel)
  alignas(64) CUtensorMap kv_map3;   // 3-D: (64, rows, d/64), box 64 x 16 x d/64: page-major stages (split kernel)
  HostSlot slots[kHostSlots];
  int next_slot = 0;
  cudaStream_t copy_stream = nullptr;  // metadata uploads overlap the previous call's kernels
  cudaStream_t in_stream = nullptr;    // host-buffer steps: inputs of the next step while this one computes
  cudaStream_t out_stream = nullptr;   // host-buffer steps: output of the last step while this one computes
  HostStep host_steps[kHostSteps];
  int64_t host_steps_issued = 0;
  uint8_t* ws = nullptr;
  int64_t launches = 0;
  Plan plan;                       // reused across calls: no allocation in steady state
  std::vector<int64_t> part_base;
  std::vector<PackCand> cands;     // shared-split packing scratch
  std::vector<int64_t> pk_off;     // per request: first entry of its complete splits in pk_mark
  std::vector<uint8_t> pk_mark;    // 1: the (request, split) pair is served by packed items
  std::vector<int32_t> pk_table, pk_next, pk_head, pk_tail;  // grouping of the candidates by key
  std::vector<PackedRow> pk_tile_rows;   // packed tiles (groups of many rows, run by the tile kernel): 128 rows each
  std::vector<uint8_t> pk_member;        // per candidate: same page ids as the first of its group
  std::vector<uint8_t> pk_keep;          // per request: some group is served from its page ids
  std::vector<int64_t> pk_group_stats;   // per sharing group: members, rows together, 16-row tiles apart
  std::vector<int4> pk_tile_items;       // per packed tile {index of the split's first page id, split, rows, 0}
  int64_t last_packed_tiles = 0;
  int64_t last_split_items = 0, last_packed_items = 0, last_tile_items = 0;  // schedule of the last attention call
  // host time spent inside vosti_kv_append and the attention entry points (steady clock)
  int64_t host_ns = 0, host_calls = 0;
  // profiling of the dominant kernel
  int profile_mode = 0;
  std::vector<cudaEvent_t> ev_start, ev_stop;
  size_t ev_used = 0;
};

namespace {

// Adds the lifetime of the scope to the context's host-time account.
struct HostTimer {
  vosti_ctx* ctx;
  std::chrono::steady_clock::time_point t0;
  explicit HostTimer(vosti_ctx* c) : ctx(c), t0(std::chrono::steady_clock::now()) {}
  ~HostTimer() {
    if (!ctx) return;
    ctx->host_ns += std::chrono::duration_cast<std::chrono::nanoseconds>(std::chrono::steady_clock::now() - t0).count();
    ++ctx->host_calls;
  }
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

vosti_status build_kv_map(vosti_ctx* ctx) {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !fn)
    return VOSTI_ERR_CUDA;
  const vosti_config& c = ctx->cfg;
  // The pool as a 2-D bf16 tensor: rows = (page, kv_head, K|V, slot), columns = head_dim.
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(c.head_dim),
                              static_cast<cuuint64_t>(c.num_pages) * c.n_kv_heads * 2 * c.page_size};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(c.head_dim) * 2};
  const cuuint32_t box[2] = {64, static_cast<cuuint32_t>(c.page_size)};  // 128 bytes x one page
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = reinterpret_cast<EncodeTiledFn>(fn)(
      &ctx->kv_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, c.kv_pool, dims, strides, box, estr,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return VOSTI_ERR_CUDA;
  // The same pool with the two 64-element halves of a row as a third dimension (its stride,
  // 128 bytes, is smaller than the row stride: the encoder accepts that), so that one box
  // of 64 x 16 x d/64 brings a whole 4 KB (page, head, K|V) chunk as [half][16 rows][128 B].
  const cuuint64_t dims3[3] = {64, dims[1], static_cast<cuuint64_t>(c.head_dim / 64)};
  const cuuint64_t strides3[2] = {static_cast<cuuint64_t>(c.head_dim) * 2, 128};
  const cuuint32_t box3[3] = {64, static_cast<cuuint32_t>(c.page_size), static_cast<cuuint32_t>(c.head_dim / 64)};
  const cuuint32_t estr3[3] = {1, 1, 1};
  const CUresult r3 = reinterpret_cast<EncodeTiledFn>(fn)(
      &ctx->kv_map3, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, c.kv_pool, dims3, strides3, box3, estr3,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r3 == CUDA_SUCCESS ? VOSTI_OK : VOSTI_ERR_CUDA;
}

// Claim the next pinned staging buffer, waiting for its previous copy if needed.
vosti_status claim_slot(vosti_ctx* ctx, HostSlot** out) {
  HostSlot* s = &ctx->slots[ctx->next_slot];
  ctx->next_slot = (ctx->next_slot + 1) % kHostSlots;
  if (s->in_flight) {
    if (cudaEventSynchronize(s->copied) != cudaSuccess) return VOSTI_ERR_CUDA;
    s->in_flight = false;
  }
  *out = s;
  return VOSTI_OK;
}

// Upload a slot's blob on the copy stream and make `stream` wait for it.  The
// copy itself waits until the kernels that last read the slot's device region
// have finished.
vosti_status push_blob(vosti_ctx* ctx, HostSlot* s, size_t bytes, cudaStream_t stream) {
  cudaStream_t cs = ctx->copy_stream;
  if (s->has_release && cudaStreamWaitEvent(cs, s->released, 0) != cudaSuccess) return VOSTI_ERR_CUDA;
  if (cudaMemcpyAsync(s->device, s->pinned, bytes, cudaMemcpyHostToDevice, cs) != cudaSuccess)
    return VOSTI_ERR_CUDA;
  if (cudaEventRecord(s->copied, cs) != cudaSuccess) return VOSTI_ERR_CUDA;
  s->in_flight = true;
  // The stream waits for the copy.  (Polling the event until the copy has landed, so that no wait
  // node sits in front of the attention kernel, cost the host 11 us per call and gained the GPU
  // nothing measurable: the kernel behind the node is the step's longest.)
  if (cudaStreamWaitEvent(stream, s->copied, 0) != cudaSuccess) return VOSTI_ERR_CUDA;
  return VOSTI_OK;
}

// Mark the point on `stream` after which the slot's device region may be overwritten.
vosti_status release_slot(HostSlot* s, cudaStream_t stream) {
  if (cudaEventRecord(s->released, stream) != cudaSuccess) return VOSTI_ERR_CUDA;
  s->has_release = true;
  return VOSTI_OK;
}

// Launch with programmatic stream serialization: the grid may be scheduled
// while its predecessor in the stream drains; the kernel calls griddep_wait()
// before touching anything the predecessor wrote.
template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kernel)(KArgs...), int grid, int block, size_t smem,
                             cudaStream_t stream, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

template <int D>
vosti_status launch_attention(vosti_ctx* ctx, const AttnParams& base, int64_t n_split, int64_t n_seq,
                              cudaStream_t stream, bool run_partials = true, bool run_combine = true,
                              int64_t n_packed_tiles = 0) {
  using Cfg = SplitKernelCfg<D>;
  const int Hkv = ctx->cfg.n_kv_heads;
  const bool prof = ctx->profile_mode != 0;
  auto timed = [&](int mode, auto&& launch) {
    const bool rec = prof && ctx->profile_mode == mode;
    if (rec) {
      if (ctx->ev_used == ctx->ev_start.size()) {
        cudaEvent_t a, b;
        cudaEventCreate(&a);
        cudaEventCreate(&b);
        ctx->ev_start.push_back(a);
        ctx->ev_stop.push_back(b);
      }
      cudaEventRecord(ctx->ev_start[ctx->ev_used], stream);
    }
    launch();
    if (rec) cudaEventRecord(ctx->ev_stop[ctx->ev_used++], stream);
    ++ctx->launches;
  };
  // A tile kernel that follows a split-parallel kernel reads nothing that kernel writes, and the two
  // are bound by different things (HBM; tensor pipe and SFU).  They run side by side: the split
  // kernel in its narrow form, which leaves half of every SM to one CTA of the tile kernel, releases
  // its successor as soon as its own inputs are complete; the tile kernel starts without waiting
  // and waits before it ends (AttnParams::beside_split).  Scheduling only: no bits depend on it.
  // (With event pairs around the kernels they run one after the other, in their usual forms.)
  const int64_t tile_ctas = (n_seq > 0 ? 2 * n_seq : n_packed_tiles) * Hkv;
  const bool side_by_side = n_split > 0 && run_partials && !prof && tile_ctas >= ctx->sm_count / 2 &&
                            !(ctx->cfg.flags & VOSTI_FLAG_NO_OVERLAP);
  // The narrow form pays when the tile kernel has CTAs for the place beside it for as long as the
  // split kernel runs (measured: mixed chunked-prefill step 501 -> 485 us narrow, 493 us not); a short
  // tile kernel rather fills the SMs that the split kernel's CTAs leave (packed prefix-sharing step
  // 56.8 us narrow, 55.2 us not).
  const bool narrow = tile_ctas >= 2 * ctx->sm_count;
  if (n_split > 0 && run_partials) {
    AttnParams p = base;
    p.n_workers = static_cast<int32_t>(n_split * Hkv);
    // persistent: one CTA per SM, warps draw (item, KV head) tickets; with few of them, fewer
    // workers per CTA with deeper rings (scheduling only)
    timed(1, [&] {
      if (side_by_side && narrow) {
        using CN = SplitKernelCfg<D, 4, true>;
        launch_dependent(attn_split_kernel<D, 4, true>, std::min((p.n_workers + 3) / 4, ctx->sm_count), 128,
                         CN::kSmemBytes, stream, ctx->kv_map3, p);
      } else if (p.n_workers <= 2 * ctx->sm_count) {
        using C2 = SplitKernelCfg<D, 2>;
        launch_dependent(attn_split_kernel<D, 2>, std::min((p.n_workers + 1) / 2, ctx->sm_count), 64, C2::kSmemBytes,
                         stream, ctx->kv_map3, p);
      } else if (p.n_workers <= 4 * ctx->sm_count ||
                 (p.n_workers > 8 * ctx->sm_count && p.n_workers <= 13 * ctx->sm_count)) {
        // (also between one and one and a half rounds of eight workers per SM, where the second round
        // would be mostly empty: four faster workers per SM balance better -- measured 2-5 % on decode
        // batches of 32-48 requests; beyond 13 tickets per SM -- the packed prefix-sharing batch has
        // 13.8 -- eight workers are faster again, 59 against 68 us on that batch)
        using C4 = SplitKernelCfg<D, 4>;
        launch_dependent(attn_split_kernel<D, 4>, std::min((p.n_workers + 3) / 4, ctx->sm_count), 128, C4::kSmemBytes,
                         stream, ctx->kv_map3, p);
      } else {
        const int grid = std::min((p.n_workers + Cfg::kWarps - 1) / Cfg::kWarps, ctx->sm_count);
        launch_dependent(attn_split_kernel<D>, grid, Cfg::kWarps * 32, Cfg::kSmemBytes, stream, ctx->kv_map3, p);
      }
    });
  }
  if (n_seq > 0 && run_partials) {
    AttnParams p = base;
    p.n_workers = static_cast<int32_t>(n_seq * Hkv);
    p.beside_split = side_by_side ? 1 : 0;
    using TileCfg_ = TileKernelCfg<D>;
    timed(2, [&] {
      // two CTAs (128 rows each) per item and KV head
      launch_dependent(attn_tile_kernel<D>, 2 * p.n_workers, TileCfg_::kThreads, TileCfg_::kSmemBytes, stream,
                       ctx->kv_map, p);
    });
  }
  if (n_packed_tiles > 0 && run_partials) {
    AttnParams p = base;
    p.n_workers = static_cast<int32_t>(n_packed_tiles * Hkv);
    p.beside_split = (side_by_side && n_seq == 0) ? 1 : 0;  // behind another tile kernel: the usual wait
    using TileCfg_ = TileKernelCfg<D>;
    timed(2, [&] {
      // one CTA per packed tile (up to 128 rows that share a split) and KV head
      launch_dependent(attn_tile_kernel<D, true>, p.n_workers, TileCfg_::kThreads, TileCfg_::kSmemBytes, stream,
                       ctx->kv_map, p);
    });
  }
  if (base.n_split_tokens > 0 && run_combine) {
    const int warps = base.n_split_tokens * base.Hq;
    timed(3, [&] { launch_dependent(combine_kernel<D>, (warps + 3) / 4, 128, 0, stream, base); });
  }
  return cudaGetLastError() == cudaSuccess ? VOSTI_OK : VOSTI_ERR_CUDA;
}

// Context-parallel decode: phase 0 = everything on this GPU; phase 1 = the partials of the splits
// this rank owns (split k belongs to rank k mod world); phase 2 = the fold over all splits.
struct CpMode {
  int phase = 0, rank = 0, world = 1;
};
vosti_status attention_impl(vosti_ctx* ctx, const void* q, void* out, float* lse, const int32_t* q_lens,
                            const int32_t* start_pos, const int32_t* seq_lens, const int32_t* block_tables,
                            int32_t block_table_stride, int32_t batch, float softmax_scale, int32_t window,
                            CpMode cp, void* cuda_stream);

template <int D>
vosti_status set_kernel_attributes() {
  using Cfg = SplitKernelCfg<D>;
  if (cudaFuncSetAttribute(attn_split_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           Cfg::kSmemBytes) != cudaSuccess ||
      cudaFuncSetAttribute(attn_split_kernel<D, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           SplitKernelCfg<D, 4>::kSmemBytes) != cudaSuccess ||
      cudaFuncSetAttribute(attn_split_kernel<D, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           SplitKernelCfg<D, 2>::kSmemBytes) != cudaSuccess ||
      cudaFuncSetAttribute(attn_split_kernel<D, 4, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           SplitKernelCfg<D, 4, true>::kSmemBytes) != cudaSuccess ||
      // the SM keeps its largest shared-memory partition, so that a tile CTA fits beside this kernel's
      cudaFuncSetAttribute(attn_split_kernel<D, 4, true>, cudaFuncAttributePreferredSharedMemoryCarveout,
                           cudaSharedmemCarveoutMaxShared) != cudaSuccess)
    return VOSTI_ERR_CUDA;
  if (cudaFuncSetAttribute(attn_tile_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           TileKernelCfg<D>::kSmemBytes) != cudaSuccess ||
      cudaFuncSetAttribute(attn_tile_kernel<D>, cudaFuncAttributePreferredSharedMemoryCarveout,
                           cudaSharedmemCarveoutMaxShared) != cudaSuccess)
    return VOSTI_ERR_CUDA;
  if (cudaFuncSetAttribute(attn_tile_kernel<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           TileKernelCfg<D>::kSmemBytes) != cudaSuccess ||
      cudaFuncSetAttribute(attn_tile_kernel<D, true>, cudaFuncAttributePreferredSharedMemoryCarveout,
                           cudaSharedmemCarveoutMaxShared) != cudaSuccess)
    return VOSTI_ERR_CUDA;
  // The tile kernel moves registers between its warpgroups; a request for more than the CTA
  // was given at launch would block for ever, so refuse to run a build where that could happen.
  cudaFuncAttributes attr;
  if (cudaFuncGetAttributes(&attr, attn_tile_kernel<D>) != cudaSuccess) return VOSTI_ERR_CUDA;
  if (attr.numRegs * TileKernelCfg<D>::kThreads < TileKernelCfg<D>::kRegsAfterSplit) return VOSTI_ERR_UNSUPPORTED_CONFIG;
  if (cudaFuncGetAttributes(&attr, attn_tile_kernel<D, true>) != cudaSuccess) return VOSTI_ERR_CUDA;
  if (attr.numRegs * TileKernelCfg<D>::kThreads < TileKernelCfg<D>::kRegsAfterSplit) return VOSTI_ERR_UNSUPPORTED_CONFIG;
  return VOSTI_OK;
}

}  // namespace

extern "C" {

const char* vosti_status_string(vosti_status s) {
  switch (s) {
    case VOSTI_OK: return "ok";
    case VOSTI_ERR_INVALID_ARG: return "invalid argument";
    case VOSTI_ERR_UNSUPPORTED_CONFIG: return "unsupported configuration";
    case VOSTI_ERR_OUT_OF_RANGE: return "length or page id out of range";
    case VOSTI_ERR_WORKSPACE: return "workspace too small or misaligned";
    case VOSTI_ERR_CUDA: return "CUDA call failed";
    case VOSTI_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

void vosti_constants(int32_t* key_tile, int32_t* split_len, int32_t* rows_per_group) {
  if (key_tile) *key_tile = nc::kKeyTile;
  if (split_len) *split_len = nc::kSplitLen;
  if (rows_per_group) *rows_per_group = nc::kRowsPerGroup;
}

// Everything that decides output bits, in a fixed order: the version, the frozen sizes and one
// id per rule of the numerical contract (nc_math.cuh).  vosti_fingerprint hashes exactly this list.
static int32_t contract_words(uint32_t* w) {
  int32_t n = 0;
  w[n++] = nc::kVersion;
  w[n++] = nc::kKeyTile;
  w[n++] = nc::kSplitLen;
  w[n++] = nc::kRowsPerGroup;
  w[n++] = nc::kSplitRowsMax;
  w[n++] = nc::kPageSize;
  w[n++] = nc::kRuleExponent;
  w[n++] = nc::kRuleMaximum;
  float step = nc::kLazyMaxStep;
  uint32_t step_bits;
  std::memcpy(&step_bits, &step, sizeof step_bits);
  w[n++] = step_bits;
  w[n++] = nc::kRuleRowSum;
  w[n++] = nc::kRuleFold;
  w[n++] = nc::kRuleReciprocal;
  w[n++] = nc::kRuleZeroSign;
  w[n++] = nc::kRuleMmaChunks;
  w[n++] = nc::kRuleLse;
  return n;
}

int32_t vosti_contract(uint32_t* words, int32_t cap) {
  uint32_t w[32];
  const int32_t n = contract_words(w);
  for (int32_t i = 0; i < n && i < cap && words; ++i) words[i] = w[i];
  return n;
}

uint64_t vosti_fingerprint(const vosti_ctx* ctx) {
  uint32_t w[32];
  const int32_t n = contract_words(w);
  uint64_t h = 1469598103934665603ull;
  for (int32_t i = 0; i < n; ++i) h = fnv1a(h, w[i]);
  if (ctx) {
    h = fnv1a(h, static_cast<uint64_t>(ctx->cfg.head_dim));
    h = fnv1a(h, static_cast<uint64_t>(ctx->cfg.page_size));
  }
  return h;
}

size_t vosti_workspace_bytes(const vosti_config* config) {
  if (!config || !geometry_ok(*config)) return 0;
  return limits_of(*config).total;
}

vosti_status vosti_plan(const vosti_config* config, const int32_t* q_lens, const int32_t* start_pos,
                        const int32_t* seq_lens, int32_t batch, vosti_work_item* items, int64_t cap,
                        int64_t* n_items, int64_t* n_split, int64_t* n_partial_rows) {
  return vosti_plan_ex(config, q_lens, start_pos, seq_lens, batch, 0, items, cap, n_items, n_split,
                       n_partial_rows);
}

vosti_status vosti_plan_ex(const vosti_config* config, const int32_t* q_lens, const int32_t* start_pos,
                           const int32_t* seq_lens, int32_t batch, int32_t window, vosti_work_item* items,
                           int64_t cap, int64_t* n_items, int64_t* n_split, int64_t* n_partial_rows) {
  if (!config || cap < 0 || (cap > 0 && !items)) return VOSTI_ERR_INVALID_ARG;
  if (!geometry_ok(*config)) return VOSTI_ERR_UNSUPPORTED_CONFIG;
  Plan plan;
  const vosti_status st = plan_requests(*config, q_lens, start_pos, seq_lens, batch, window, &plan, nullptr);
  if (st != VOSTI_OK) return st;
  const int64_t n = static_cast<int64_t>(plan.items.size());
  for (int64_t i = 0; i < std::min(n, cap); ++i) items[i] = plan.items[i];
  if (n_items) *n_items = n;
  if (n_split) *n_split = plan.n_split;
  if (n_partial_rows) *n_partial_rows = plan.n_partial_rows;
  return VOSTI_OK;
}

vosti_status vosti_create(vosti_ctx** out, const vosti_config* config) {
  if (!out || !config) return VOSTI_ERR_INVALID_ARG;
  *out = nullptr;
  if (!geometry_ok(*config)) return VOSTI_ERR_UNSUPPORTED_CONFIG;
  if (!config->kv_pool || !config->workspace) return VOSTI_ERR_INVALID_ARG;
  const Limits lim = limits_of(*config);
  if (config->workspace_bytes < lim.total || reinterpret_cast<uintptr_t>(config->workspace) % kAlign)
    return VOSTI_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(config->kv_pool) % kAlign) return VOSTI_ERR_INVALID_ARG;
  vosti_ctx* ctx = new (std::nothrow) vosti_ctx();
  if (!ctx) return VOSTI_ERR_INVALID_ARG;
  ctx->cfg = *config;
  ctx->lim = lim;
  ctx->ws = static_cast<uint8_t*>(config->workspace);
  vosti_status st = VOSTI_OK;
  if (cudaGetDevice(&ctx->device) != cudaSuccess ||
      cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, ctx->device) != cudaSuccess)
    st = VOSTI_ERR_CUDA;
  if (st == VOSTI_OK) st = build_kv_map(ctx);
  if (st == VOSTI_OK) st = config->head_dim == 128 ? set_kernel_attributes<128>() : set_kernel_attributes<64>();
  if (st == VOSTI_OK && cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking) != cudaSuccess)
    st = VOSTI_ERR_CUDA;
  if (st == VOSTI_OK && (cudaStreamCreateWithFlags(&ctx->in_stream, cudaStreamNonBlocking) != cudaSuccess ||
                         cudaStreamCreateWithFlags(&ctx->out_stream, cudaStreamNonBlocking) != cudaSuccess))
    st = VOSTI_ERR_CUDA;
  for (int i = 0; st == VOSTI_OK && i < kHostSteps; ++i) {
    HostStep& h = ctx->host_steps[i];
    if (cudaEventCreateWithFlags(&h.in_done, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h.computed, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h.out_done, cudaEventDisableTiming) != cudaSuccess)
      st = VOSTI_ERR_CUDA;
  }
  for (int i = 0; st == VOSTI_OK && i < kHostSlots; ++i) {
    ctx->slots[i].device = ctx->ws + lim.off_meta + static_cast<size_t>(i) * lim.meta_bytes;
    if (cudaHostAlloc(reinterpret_cast<void**>(&ctx->slots[i].pinned), lim.meta_bytes, cudaHostAllocDefault) !=
            cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->slots[i].copied, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->slots[i].released, cudaEventDisableTiming) != cudaSuccess)
      st = VOSTI_ERR_CUDA;
  }
  if (st == VOSTI_OK && cudaMemset(ctx->ws + lim.off_status, 0, kAlign) != cudaSuccess) st = VOSTI_ERR_CUDA;
  if (st == VOSTI_OK && cudaDeviceSynchronize() != cudaSuccess) st = VOSTI_ERR_CUDA;
  if (st != VOSTI_OK) {
    vosti_destroy(ctx);
    return st;
  }
  *out = ctx;
  return VOSTI_OK;
}

vosti_status vosti_destroy(vosti_ctx* ctx) {
  if (!ctx) return VOSTI_OK;
  for (auto& s : ctx->slots) {
    if (s.in_flight) cudaEventSynchronize(s.copied);
    if (s.copied) cudaEventDestroy(s.copied);
    if (s.released) cudaEventDestroy(s.released);
    if (s.pinned) cudaFreeHost(s.pinned);
  }
  for (cudaStream_t cs : {ctx->in_stream, ctx->out_stream, ctx->copy_stream}) {
    if (!cs) continue;
    cudaStreamSynchronize(cs);
    cudaStreamDestroy(cs);
  }
  for (auto& h : ctx->host_steps)
    for (cudaEvent_t e : {h.in_done, h.computed, h.out_done})
      if (e) cudaEventDestroy(e);
  for (auto e : ctx->ev_start) cudaEventDestroy(e);
  for (auto e : ctx->ev_stop) cudaEventDestroy(e);
  delete ctx;
  return VOSTI_OK;
}

vosti_status vosti_kv_append(vosti_ctx* ctx, const void* k_new, const void* v_new, const int32_t* q_lens,
                             const int32_t* start_pos, const int32_t* block_tables,
                             int32_t block_table_stride, int32_t batch, void* cuda_stream) {
  if (!ctx || batch < 0 || block_table_stride < 0) return VOSTI_ERR_INVALID_ARG;
  if (batch > 0 && (!q_lens || !start_pos || !block_tables)) return VOSTI_ERR_INVALID_ARG;
  if (batch > ctx->cfg.max_batch) return VOSTI_ERR_OUT_OF_RANGE;
  HostTimer host_timer(ctx);
  const vosti_config& c = ctx->cfg;
  int64_t total = 0;
  for (int r = 0; r < batch; ++r) {
    if (q_lens[r] < 0 || start_pos[r] < 0) return VOSTI_ERR_OUT_OF_RANGE;
    total += q_lens[r];
  }
  if (total > c.max_total_q) return VOSTI_ERR_OUT_OF_RANGE;
  if (total == 0) return VOSTI_OK;
  if (!k_new || !v_new) return VOSTI_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(k_new) | reinterpret_cast<uintptr_t>(v_new)) % 16) return VOSTI_ERR_INVALID_ARG;
  // Few tokens (decode): the slot list rides in the kernel parameters, no upload.
  const bool inline_slots = total <= AppendParams::kInlineSlots;
  AppendParams p;
  HostSlot* slot = nullptr;
  vosti_status st = VOSTI_OK;
  int32_t* dst = p.inline_slot;
  if (!inline_slots) {
    st = claim_slot(ctx, &slot);
    if (st != VOSTI_OK) return st;
    dst = reinterpret_cast<int32_t*>(slot->pinned);
  }
  int64_t t = 0;
  for (int r = 0; r < batch; ++r) {
    const int32_t* row = block_tables + static_cast<size_t>(r) * block_table_stride;
    for (int i = 0; i < q_lens[r]; ++i, ++t) {
      const int64_t pos = int64_t{start_pos[r]} + i;
      const int64_t blk = pos / c.page_size;
      if (blk >= block_table_stride) return VOSTI_ERR_OUT_OF_RANGE;
      const int64_t page = row[blk];
      if (page < 0 || page >= c.num_pages) return VOSTI_ERR_OUT_OF_RANGE;
      dst[t] = static_cast<int32_t>(page * c.page_size + pos % c.page_size);
    }
  }
  if (c.flags & VOSTI_FLAG_CHECK_WRITE_SLOTS) {
    std::vector<int32_t> sorted(dst, dst + total);
    std::sort(sorted.begin(), sorted.end());
    if (std::adjacent_find(sorted.begin(), sorted.end()) != sorted.end()) return VOSTI_ERR_OUT_OF_RANGE;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (!inline_slots) {
    st = push_blob(ctx, slot, sizeof(int32_t) * total, stream);
    if (st != VOSTI_OK) return st;
  }
  p.k_new = static_cast<const __nv_bfloat16*>(k_new);
  p.v_new = static_cast<const __nv_bfloat16*>(v_new);
  p.pool = static_cast<__nv_bfloat16*>(c.kv_pool);
  p.slot = inline_slots ? nullptr : reinterpret_cast<const int32_t*>(slot->device);
  p.n_tokens = static_cast<int32_t>(total);
  p.Hkv = c.n_kv_heads;
  const int64_t warps = total * c.n_kv_heads;
  const int grid = static_cast<int>((warps + 3) / 4);
  if (c.head_dim == 128)
    launch_dependent(kv_append_kernel<128>, grid, 128, 0, stream, p);
  else
    launch_dependent(kv_append_kernel<64>, grid, 128, 0, stream, p);
  ++ctx->launches;
  if (cudaGetLastError() != cudaSuccess) return VOSTI_ERR_CUDA;
  return inline_slots ? VOSTI_OK : release_slot(slot, stream);
}

vosti_status vosti_paged_attention(vosti_ctx* ctx, const void* q, void* out, const int32_t* q_lens,
                                   const int32_t* start_pos, const int32_t* seq_lens,
                                   const int32_t* block_tables, int32_t block_table_stride, int32_t batch,
                                   float softmax_scale, void* cuda_stream) {
  return vosti_paged_attention_ex(ctx, q, out, nullptr, q_lens, start_pos, seq_lens, block_tables,
                                  block_table_stride, batch, softmax_scale, 0, cuda_stream);
}

vosti_status vosti_paged_attention_ex(vosti_ctx* ctx, const void* q, void* out, float* lse, const int32_t* q_lens,
                                      const int32_t* start_pos, const int32_t* seq_lens,
                                      const int32_t* block_tables, int32_t block_table_stride, int32_t batch,
                                      float softmax_scale, int32_t window, void* cuda_stream) {
  return attention_impl(ctx, q, out, lse, q_lens, start_pos, seq_lens, block_tables, block_table_stride, batch,
                        softmax_scale, window, CpMode{}, cuda_stream);
}

vosti_status vosti_cp_partial(vosti_ctx* ctx, const void* q, const int32_t* q_lens, const int32_t* start_pos,
                              const int32_t* seq_lens, const int32_t* block_tables, int32_t block_table_stride,
                              int32_t batch, float softmax_scale, int32_t cp_rank, int32_t cp_world,
                              size_t* u_offset, size_t* u_bytes, size_t* mz_offset, size_t* mz_bytes,
                              void* cuda_stream) {
  if (cp_world < 1 || cp_rank < 0 || cp_rank >= cp_world) return VOSTI_ERR_INVALID_ARG;
  CpMode cp;
  cp.phase = 1;
  cp.rank = cp_rank;
  cp.world = cp_world;
  const vosti_status st = attention_impl(ctx, q, nullptr, nullptr, q_lens, start_pos, seq_lens, block_tables,
                                         block_table_stride, batch, softmax_scale, 0, cp, cuda_stream);
  if (st != VOSTI_OK) return st;
  if (u_offset) *u_offset = ctx->lim.off_part_u;
  if (u_bytes) *u_bytes = sizeof(float) * static_cast<size_t>(ctx->plan.n_partial_rows) * ctx->cfg.head_dim;
  if (mz_offset) *mz_offset = ctx->lim.off_part_mz;
  if (mz_bytes) *mz_bytes = sizeof(float2) * static_cast<size_t>(ctx->plan.n_partial_rows);
  return VOSTI_OK;
}

vosti_status vosti_cp_segments(const vosti_config* config, const int32_t* q_lens, const int32_t* start_pos,
                               const int32_t* seq_lens, int32_t batch, int32_t cp_rank, int32_t cp_world,
                               int64_t* segments, int64_t cap, int64_t* n_segments, int64_t* n_partial_rows) {
  if (!config || cap < 0 || (cap > 0 && !segments)) return VOSTI_ERR_INVALID_ARG;
  if (cp_world < 1 || cp_rank < 0 || cp_rank >= cp_world) return VOSTI_ERR_INVALID_ARG;
  if (!geometry_ok(*config)) return VOSTI_ERR_UNSUPPORTED_CONFIG;
  Plan plan;
  std::vector<int64_t> part_base(static_cast<size_t>(std::max(batch, 0)));
  const vosti_status st = plan_requests(*config, q_lens, start_pos, seq_lens, batch, 0, &plan, part_base.data());
  if (st != VOSTI_OK) return st;
  if (static_cast<int64_t>(plan.items.size()) != plan.n_split) return VOSTI_ERR_UNSUPPORTED_CONFIG;  // long queries
  const int64_t G = config->n_q_heads / config->n_kv_heads;
  int64_t n = 0;
  // The partial rows of request r, KV head h, split k are rows [base, base + rows) with
  // base = part_base[r] + (h * n_splits + k) * rows; split k belongs to rank k mod world.
  for (int r = 0; r < batch; ++r) {
    if (q_lens[r] == 0) continue;
    const int64_t rows = int64_t{q_lens[r]} * G;
    const int64_t n_splits = (int64_t{start_pos[r]} + q_lens[r] - 1) / nc::kSplitLen + 1;
    for (int64_t h = 0; h < config->n_kv_heads; ++h)
      for (int64_t k = cp_rank; k < n_splits; k += cp_world) {
        if (n < cap) {
          segments[2 * n] = part_base[r] + (h * n_splits + k) * rows;
          segments[2 * n + 1] = rows;
        }
        ++n;
      }
  }
  if (n_segments) *n_segments = n;
  if (n_partial_rows) *n_partial_rows = plan.n_partial_rows;
  return VOSTI_OK;
}

vosti_status vosti_cp_combine(vosti_ctx* ctx, void* out, float* lse, const int32_t* q_lens,
                              const int32_t* start_pos, const int32_t* seq_lens, int32_t batch, void* cuda_stream) {
  CpMode cp;
  cp.phase = 2;
  return attention_impl(ctx, nullptr, out, lse, q_lens, start_pos, seq_lens, nullptr, 0, batch, 1.0f, 0, cp,
                        cuda_stream);
}

}  // extern "C"

namespace {

// Shared-split packing (scheduling only).  Candidates: complete splits (all 512 keys below every
// row of the request) of split-parallel requests.  Requests whose 32 page ids of a split agree
// (compared in the caller's block tables) form a group, served from its first member's ids.  The
// rows of a group of two or more are laid out 16 to a packed item of the split-parallel kernel, if
// that saves tiles, or -- large groups, when they add up to enough work -- 128 to a packed tile of
// the tile kernel (ctx->pk_tile_rows / pk_tile_items).  Writes the 16-row packed rows at
// `packed_rows`, one SplitItem per packed item at the front of `split_items`, marks the (request,
// split) pairs it has taken over in ctx->pk_mark and the first members in ctx->pk_keep, and
// returns the number of 16-row packed items.  Items and tiles name their group's first request
// where the index into the flat page table will go: the caller patches that in once the table is
// laid out.
int64_t pack_shared_splits(vosti_ctx* ctx, const ReqMeta* reqs, int32_t batch, int G, const int32_t* block_tables,
                           int32_t block_table_stride, PackedRow* packed_rows, SplitItem* split_items) {
  // page ids of split k of request r, in the caller's table (not validated here: a group is served
  // from its first member's ids, which are validated when they are copied)
  auto ids_of = [&](int r, int64_t k) {
    return block_tables + static_cast<size_t>(r) * block_table_stride + k * nc::kPagesPerSplit;
  };
  std::vector<int64_t>& pk_off = ctx->pk_off;
  std::vector<uint8_t>& pk_mark = ctx->pk_mark;
  int64_t n_split_final = 0, n_packed_items = 0;
  std::vector<PackCand>& cands = ctx->cands;
  cands.clear();
  ctx->pk_tile_rows.clear();
  ctx->pk_tile_items.clear();
  pk_off.assign(static_cast<size_t>(batch) + 1, 0);
  for (int r = 0; r < batch; ++r) {
    const ReqMeta& m = reqs[r];
    const int64_t complete =
        (m.q_len > 0 && int64_t{m.q_len} * G <= nc::kSplitRowsMax) ? m.start / nc::kSplitLen : 0;
    pk_off[r + 1] = pk_off[r] + complete;
    for (int64_t k = 0; k < complete; ++k) {
      const int32_t* ids = ids_of(r, k);
      // Grouping key: the split index with its first and last page id.  Two requests that share
      // the whole split agree on it; agreement on all 32 ids is checked when groups are formed.
      const uint64_t key = ((static_cast<uint64_t>(static_cast<uint32_t>(ids[0])) << 32) |
                            static_cast<uint32_t>(ids[nc::kPagesPerSplit - 1])) * 0x9E3779B97F4A7C15ull +
                           static_cast<uint64_t>(k);
      cands.push_back({key, r, static_cast<int32_t>(k)});
    }
  }
  pk_mark.assign(static_cast<size_t>(pk_off[batch]), 0);
  // Group the candidates by key without sorting: an open-addressing table from key to group, the
  // members of a group chained in the order they were generated (ascending request index).
  const int n = static_cast<int>(cands.size());
  int table_size = 64;
  while (table_size < 2 * n) table_size *= 2;
  std::vector<int32_t>& table = ctx->pk_table;
  std::vector<int32_t>& next = ctx->pk_next;
  std::vector<int32_t>& head = ctx->pk_head;
  std::vector<int32_t>& tail = ctx->pk_tail;
  table.assign(static_cast<size_t>(table_size), -1);
  next.assign(static_cast<size_t>(n), -1);
  head.clear();
  tail.clear();
  for (int i = 0; i < n; ++i) {
    uint32_t h = static_cast<uint32_t>((cands[i].key * 0xD6E8FEB86659FD93ull) >> 40) & (table_size - 1);
    while (table[h] >= 0 && cands[head[table[h]]].key != cands[i].key) h = (h + 1) & (table_size - 1);
    if (table[h] < 0) {
      table[h] = static_cast<int32_t>(head.size());
      head.push_back(i);
      tail.push_back(i);
    } else {
      next[tail[table[h]]] = i;
      tail[table[h]] = i;
    }
  }
  auto same_pages = [&](const PackCand& a, const PackCand& b) {
    return a.split == b.split &&
           std::memcmp(ids_of(a.req, a.split), ids_of(b.req, b.split), sizeof(int32_t) * nc::kPagesPerSplit) == 0;
  };
  std::vector<uint8_t>& member = ctx->pk_member;  // per candidate: it has the page ids of its group's first one
  member.assign(static_cast<size_t>(n), 0);
  ctx->pk_keep.assign(static_cast<size_t>(batch), 0);
  // What each group amounts to.  Groups of kTilePackMinRows rows or more could go through the tile
  // kernel; that costs one more launch per call, so it is done only when the rows x splits they
  // hold add up to enough work (or the context asks for it always).
  struct GroupStat {
    int members;
    int64_t rows_together, tiles_apart;
  };
  std::vector<int64_t>& stats = ctx->pk_group_stats;  // three numbers per group
  stats.assign(3 * head.size(), 0);
  int64_t tile_row_splits = 0;
  for (size_t g = 0; g < head.size(); ++g) {
    const int lo = head[g];
    if (next[lo] < 0) continue;  // alone
    GroupStat gs{0, 0, 0};
    for (int i = lo; i >= 0; i = next[i])
      if (i == lo || same_pages(cands[i], cands[lo])) {
        member[i] = 1;
        const int64_t rows = int64_t{reqs[cands[i].req].q_len} * G;
        ++gs.members;
        gs.rows_together += rows;
        gs.tiles_apart += (rows + nc::kRowsPerGroup - 1) / nc::kRowsPerGroup;
      }
    stats[3 * g] = gs.members;
    stats[3 * g + 1] = gs.rows_together;
    stats[3 * g + 2] = gs.tiles_apart;
    if (gs.members >= 2 && gs.rows_together >= kTilePackMinRows) tile_row_splits += gs.rows_together;
  }
  const bool through_tiles =
      (ctx->cfg.flags & VOSTI_FLAG_PACK_THROUGH_TILES) || tile_row_splits >= kTilePackMinRowSplits;
  for (size_t g = 0; g < head.size(); ++g) {
    const int lo = head[g];
    if (next[lo] < 0) continue;  // alone
    // members: the very same split and page ids as the first (a key collision stays unpacked);
    // packing must save tiles: fewer 16-row tiles together than one request at a time, or
    // enough rows for the 128-row tiles of the tile kernel
    const int64_t members = stats[3 * g], rows_together = stats[3 * g + 1], tiles_apart = stats[3 * g + 2];
    if (members < 2) continue;
    const bool to_tiles = through_tiles && rows_together >= kTilePackMinRows;
    if (!to_tiles && (rows_together + nc::kRowsPerGroup - 1) / nc::kRowsPerGroup >= tiles_apart) continue;
    const int first_req = cands[lo].req;  // the group is served from this request's page ids
    ctx->pk_keep[first_req] = 1;
    if (to_tiles) {
      // Many rows share the split: 128 to a tile of the tensor-memory kernel, which reads the
      // split once per 128 rows instead of once per 16.
      std::vector<PackedRow>& trows = ctx->pk_tile_rows;
      const int split = cands[lo].split;
      const int64_t n_tiles = (rows_together + kPackedTileRows - 1) / kPackedTileRows;
      const size_t first_row = trows.size();
      trows.resize(first_row + static_cast<size_t>(n_tiles) * kPackedTileRows);
      for (size_t i = first_row + static_cast<size_t>(rows_together); i < trows.size(); ++i)
        trows[i] = PackedRow{0, -1, 0, 0};  // padding rows of the last tile see nothing
      for (int64_t t = 0; t < n_tiles; ++t)
        ctx->pk_tile_items.push_back(make_int4(
            first_req, split,  // .x becomes an index into the flat table once that is laid out
            static_cast<int>(std::min<int64_t>(kPackedTileRows, rows_together - t * kPackedTileRows)), 0));
      PackedRow* pr = trows.data() + first_row;  // real rows are contiguous; only the last tile has padding
      for (int i = lo; i >= 0; i = next[i]) {
        if (!member[i]) continue;
        const ReqMeta& m = reqs[cands[i].req];
        pk_mark[static_cast<size_t>(pk_off[cands[i].req] + split)] = 1;
        const int rows = m.q_len * G;
        const int32_t slab0 = static_cast<int32_t>(m.part_base + int64_t{split} * rows);
        const int32_t stride = m.n_splits * rows;
        int row = 0;
        for (int tok = 0; tok < m.q_len; ++tok)
          for (int g = 0; g < G; ++g, ++row, ++pr) {
            pr->q_row_g = (m.q_row0 + tok) | (g << 24);
            pr->p = m.start + tok;
            pr->slab_row = slab0 + row;
            pr->kvh_stride = stride;
          }
      }
      continue;
    }
    int in_item = 0;
    auto close_item = [&]() {
      PackedRow* rows16 = packed_rows + n_packed_items * 16;
      for (int i = in_item; i < 16; ++i) rows16[i] = PackedRow{0, -1, 0, 0};
      SplitItem& si = split_items[n_split_final++];
      si = SplitItem{};
      si.q_len = in_item;  // rows in use
      si.n_pages = reqs[first_req].n_pages;
      si.bt_index = first_req;  // becomes an index into the flat table once that is laid out
      si.split = cands[lo].split;
      si.req = static_cast<int32_t>(-1 - n_packed_items);
      ++n_packed_items;
      in_item = 0;
    };
    for (int i = lo; i >= 0; i = next[i]) {
      if (!member[i]) continue;
      const ReqMeta& m = reqs[cands[i].req];
      const int k = cands[i].split;
      pk_mark[static_cast<size_t>(pk_off[cands[i].req] + k)] = 1;
      const int rows = m.q_len * G;
      const int32_t slab0 = static_cast<int32_t>(m.part_base + int64_t{k} * rows);
      int row = 0;
      for (int tok = 0; tok < m.q_len; ++tok)
        for (int g = 0; g < G; ++g, ++row) {
          PackedRow& pr = packed_rows[n_packed_items * 16 + in_item];
          pr.q_row_g = (m.q_row0 + tok) | (g << 24);
          pr.p = m.start + tok;
          pr.slab_row = slab0 + row;
          pr.kvh_stride = m.n_splits * rows;
          if (++in_item == 16) close_item();
        }
    }
    if (in_item > 0) close_item();
  }
  return n_packed_items;
}

vosti_status attention_impl(vosti_ctx* ctx, const void* q, void* out, float* lse, const int32_t* q_lens,
                            const int32_t* start_pos, const int32_t* seq_lens, const int32_t* block_tables,
                            int32_t block_table_stride, int32_t batch, float softmax_scale, int32_t window,
                            CpMode cp, void* cuda_stream) {
  if (!ctx || batch < 0 || block_table_stride < 0 || window < 0) return VOSTI_ERR_INVALID_ARG;
  if (!(softmax_scale >= 0.0f) || !std::isfinite(softmax_scale)) return VOSTI_ERR_INVALID_ARG;
  if (batch > 0 && !block_tables && cp.phase != 2) return VOSTI_ERR_INVALID_ARG;
  HostTimer host_timer(ctx);
  const vosti_config& c = ctx->cfg;
  Plan& plan = ctx->plan;
  std::vector<int64_t>& part_base = ctx->part_base;
  part_base.resize(static_cast<size_t>(std::max(batch, 0)));
  vosti_status st = plan_requests(c, q_lens, start_pos, seq_lens, batch, window, &plan, part_base.data());
  if (st != VOSTI_OK) return st;
  if (plan.items.empty()) return VOSTI_OK;
  // context-parallel phases exist for split-parallel requests only (decode, speculative queries)
  if (cp.phase != 0 && static_cast<int64_t>(plan.items.size()) != plan.n_split) return VOSTI_ERR_UNSUPPORTED_CONFIG;
  if ((cp.phase != 2 && !q) || (cp.phase != 1 && !out)) return VOSTI_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(out)) % 16) return VOSTI_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(lse) % 4) return VOSTI_ERR_INVALID_ARG;
  if (static_cast<int64_t>(plan.items.size()) > ctx->lim.items_max ||
      plan.n_partial_rows > ctx->lim.part_rows_max)
    return VOSTI_ERR_WORKSPACE;

  HostSlot* slot = nullptr;
  st = claim_slot(ctx, &slot);
  if (st != VOSTI_OK) return st;
  // Blob: [ReqMeta x batch][SplitItem x n_split][sequential items][flat page ids][split tokens]
  const int G = c.n_q_heads / c.n_kv_heads;
  const int64_t n_seq = static_cast<int64_t>(plan.items.size()) - plan.n_split;
  uint8_t* blob = slot->pinned;
  size_t at = 0;
  ReqMeta* reqs = reinterpret_cast<ReqMeta*>(blob + at);
  const size_t off_reqs = at;
  at += align_up(sizeof(ReqMeta) * batch, 16);
  const size_t off_split = at;
  SplitItem* split_items = reinterpret_cast<SplitItem*>(blob + at);
  at += align_up(sizeof(SplitItem) * plan.n_split, 16);
  const size_t off_items = at;
  std::memcpy(blob + at, plan.items.data() + plan.n_split, sizeof(vosti_work_item) * n_seq);
  at += align_up(sizeof(vosti_work_item) * n_seq, 16);
  int64_t row0 = 0, n_split_tokens = 0;
  for (int r = 0; r < batch; ++r) {
    ReqMeta& m = reqs[r];
    m.q_row0 = static_cast<int32_t>(row0);
    m.q_len = q_lens[r];
    m.start = start_pos[r];
    m.n_pages = 0;
    m.bt_off = 0;
    m.n_splits = 0;
    m.first_split = 0;
    m.pad = 0;
    m.part_base = part_base[r];
    row0 += q_lens[r];
    if (q_lens[r] == 0) continue;
    const int64_t n_eff = int64_t{start_pos[r]} + q_lens[r];
    const int64_t n_pages = (n_eff + c.page_size - 1) / c.page_size;
    if (cp.phase != 2 && (n_pages > block_table_stride ||
                          (int64_t{seq_lens[r]} + c.page_size - 1) / c.page_size > block_table_stride))
      return VOSTI_ERR_OUT_OF_RANGE;
    m.n_pages = static_cast<int32_t>(n_pages);
    m.first_split = cp.phase == 2 ? 0 : static_cast<int32_t>(first_visible_key(start_pos[r], window) / nc::kSplitLen);
    m.n_splits = static_cast<int32_t>((n_eff - 1) / nc::kSplitLen + 1) - m.first_split;
    if (int64_t{q_lens[r]} * G <= nc::kSplitRowsMax) n_split_tokens += q_lens[r];
  }

  // ---- shared-split packing (scheduling only): packed items first in the item list (they walk a
  // whole split: the longest kind), the others follow in plan order.  It groups on the caller's
  // tables, before the flat table is laid out, so that pages only packed items read need not be
  // copied for every member of a group. -------------------------------------------------------
  int64_t n_split_final = 0, n_packed_items = 0, n_packed_tiles = 0;
  size_t off_packed = 0, off_tile_rows = 0, off_tile_items = 0;
  std::vector<int64_t>& pk_off = ctx->pk_off;
  std::vector<uint8_t>& pk_mark = ctx->pk_mark;
  const bool packing = (c.flags & VOSTI_FLAG_PACK_SHARED_SPLITS) && window == 0 && cp.phase == 0 && plan.n_split > 1 &&
                       plan.n_partial_rows < (int64_t{1} << 31) && row0 < (int64_t{1} << 24) && G <= 128;
  if (packing) {
    off_packed = at;
    n_packed_items = pack_shared_splits(ctx, reqs, batch, G, block_tables, block_table_stride,
                                        reinterpret_cast<PackedRow*>(blob + at), split_items);
    n_split_final = n_packed_items;
    at += align_up(sizeof(PackedRow) * 16 * n_packed_items, 16);
    n_packed_tiles = static_cast<int64_t>(ctx->pk_tile_items.size());
  }

  // ---- the flat page-id table ------------------------------------------------------------------
  const size_t off_bt = at;
  int32_t* bt_flat = reinterpret_cast<int32_t*>(blob + at);
  int64_t bt_used = 0;
  for (int r = 0; r < batch && cp.phase != 2; ++r) {  // the fold reads no pages
    ReqMeta& m = reqs[r];
    if (q_lens[r] == 0) continue;
    const int64_t n_pages = m.n_pages;
    const int32_t* row = block_tables + static_cast<size_t>(r) * block_table_stride;
    // Pages that lie wholly before the window of the request's first row are never
    // visible: their table entries are not read (the caller may have freed them);
    // page 0 stands in where a tile load still covers them.
    const int64_t first_page = first_visible_key(start_pos[r], window) / c.page_size;
    // The leading splits of a request that packed items serve are read from the first member of
    // their group: this request's ids for them are not needed on the device (they equal that
    // member's, which are copied and checked), unless it is such a first member itself.
    int64_t skip = 0;
    if ((n_packed_items > 0 || n_packed_tiles > 0) && !ctx->pk_keep[r]) {
      const int64_t complete = pk_off[r + 1] - pk_off[r];
      int64_t lead = 0;
      while (lead < complete && pk_mark[static_cast<size_t>(pk_off[r] + lead)]) ++lead;
      skip = lead * nc::kPagesPerSplit;
    }
    m.bt_off = static_cast<int32_t>(bt_used - skip);
    if (skip == 0 && first_page == 0 && cp.phase == 0) {
      // the common case: the whole row, copied and range-checked without a branch per entry
      // (page | (limit - page)) is negative exactly when page < 0 or page > limit
      const int32_t limit = static_cast<int32_t>(c.num_pages - 1);
      int32_t* dst = bt_flat + bt_used;
      int32_t bad = 0;
      for (int64_t b = 0; b < n_pages; ++b) {
        const int32_t page = row[b];
        bad |= page | (limit - page);
        dst[b] = page;
      }
      if (bad < 0) return VOSTI_ERR_OUT_OF_RANGE;
      bt_used += n_pages;
      continue;
    }
    for (int64_t b = skip; b < first_page; ++b) bt_flat[bt_used + b - skip] = 0;
    for (int64_t b = std::max(skip, first_page); b < n_pages; ++b) {
      // a context-parallel rank holds (and names) only the pages of the splits it owns
      if (cp.phase == 1 && (b / nc::kPagesPerSplit) % cp.world != cp.rank) {
        bt_flat[bt_used + b - skip] = 0;
        continue;
      }
      const int32_t page = row[b];
      if (page < 0 || page >= c.num_pages) return VOSTI_ERR_OUT_OF_RANGE;
      bt_flat[bt_used + b - skip] = page;
    }
    bt_used += n_pages - skip;
  }
  at += align_up(sizeof(int32_t) * bt_used, 16);
  if (packing) {
    // packed items and tiles named their group's first request: now its ids have a place
    for (int64_t i = 0; i < n_packed_items; ++i)
      split_items[i].bt_index = reqs[split_items[i].bt_index].bt_off + split_items[i].split * nc::kPagesPerSplit;
    for (int4& ti : ctx->pk_tile_items) ti.x = reqs[ti.x].bt_off + ti.y * nc::kPagesPerSplit;
    if (n_packed_tiles > 0) {
      off_tile_rows = at;
      std::memcpy(blob + at, ctx->pk_tile_rows.data(), sizeof(PackedRow) * ctx->pk_tile_rows.size());
      at += align_up(sizeof(PackedRow) * ctx->pk_tile_rows.size(), 16);
      off_tile_items = at;
      std::memcpy(blob + at, ctx->pk_tile_items.data(), sizeof(int4) * ctx->pk_tile_items.size());
      at += align_up(sizeof(int4) * ctx->pk_tile_items.size(), 16);
    }
  }
  for (int64_t i = 0; i < plan.n_split; ++i) {
    const vosti_work_item& it = plan.items[i];
    const ReqMeta& m = reqs[it.req];
    if ((n_packed_items > 0 || n_packed_tiles > 0) && int64_t{it.split_begin} < pk_off[it.req + 1] - pk_off[it.req] &&
        pk_mark[static_cast<size_t>(pk_off[it.req] + it.split_begin)])
      continue;  // served by packed items
    if (cp.phase == 2 || (cp.phase == 1 && it.split_begin % cp.world != cp.rank)) continue;  // not this rank's split
    SplitItem& si = split_items[n_split_final++];
    si.q_row0 = m.q_row0;
    si.q_len = m.q_len;
    si.start = m.start;
    si.n_pages = m.n_pages;
    si.bt_index = m.bt_off + it.split_begin * nc::kPagesPerSplit;
    si.split = it.split_begin;
    si.row_group = it.row_group;
    si.n_splits = m.n_splits;
    si.part_base = m.part_base;
    si.req = it.req;
    si.first_split = m.first_split;
  }
  const size_t off_tok = at;
  int2* toks = reinterpret_cast<int2*>(blob + at);
  {
    int64_t x = 0;
    for (int r = 0; r < batch; ++r)
      if (q_lens[r] > 0 && int64_t{q_lens[r]} * G <= nc::kSplitRowsMax)
        for (int i = 0; i < q_lens[r]; ++i) toks[x++] = make_int2(r, i);
  }
  at += align_up(sizeof(int2) * n_split_tokens, 16);

  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  st = push_blob(ctx, slot, at, stream);
  if (st != VOSTI_OK) return st;

  uint8_t* dmeta = slot->device;
  AttnParams p;
  p.beside_split = 0;
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.out = static_cast<__nv_bfloat16*>(out);
  p.reqs = reinterpret_cast<const ReqMeta*>(dmeta + off_reqs);
  p.items = reinterpret_cast<const vosti_work_item*>(dmeta + off_items);
  p.split_items = reinterpret_cast<const SplitItem*>(dmeta + off_split);
  p.packed_rows = reinterpret_cast<const PackedRow*>(dmeta + off_packed);
  p.ticket = reinterpret_cast<uint32_t*>(ctx->ws + ctx->lim.off_status + 64);
  p.done = reinterpret_cast<uint32_t*>(ctx->ws + ctx->lim.off_status + 128);
  p.bt_flat = reinterpret_cast<const int32_t*>(dmeta + off_bt);
  p.split_tokens = reinterpret_cast<const int2*>(dmeta + off_tok);
  p.ws_u = reinterpret_cast<float*>(ctx->ws + ctx->lim.off_part_u);
  p.ws_mz = reinterpret_cast<float2*>(ctx->ws + ctx->lim.off_part_mz);
  p.ws_uc = reinterpret_cast<float*>(ctx->ws + ctx->lim.off_uc);
  p.status = reinterpret_cast<uint32_t*>(ctx->ws + ctx->lim.off_status);
  p.n_workers = 0;
  p.n_split_tokens = static_cast<int32_t>(n_split_tokens);
  p.Hq = c.n_q_heads;
  p.Hkv = c.n_kv_heads;
  p.G = G;
  p.c = static_cast<float>(static_cast<double>(softmax_scale) * 1.4426950408889634074);
  p.window = window;
  p.lse = lse;
  p.counts = nullptr;
  p.num_pages = 0;
  p.tile_pack_items = n_packed_tiles > 0 ? reinterpret_cast<const int4*>(dmeta + off_tile_items) : nullptr;
  p.tile_rows = n_packed_tiles > 0 ? reinterpret_cast<const PackedRow*>(dmeta + off_tile_rows) : nullptr;
  ctx->last_packed_tiles = n_packed_tiles;
  ctx->last_split_items = n_split_final;
  ctx->last_packed_items = n_packed_items;
  ctx->last_tile_items = n_seq + n_packed_tiles;
  if (cp.phase == 1) {
    // Slabs of splits other ranks own stay zero, so that a sum over ranks assembles all partials.
    if (cudaMemsetAsync(p.ws_u, 0, sizeof(float) * static_cast<size_t>(plan.n_partial_rows) * c.head_dim, stream) !=
            cudaSuccess ||
        cudaMemsetAsync(p.ws_mz, 0, sizeof(float2) * static_cast<size_t>(plan.n_partial_rows), stream) != cudaSuccess)
      return VOSTI_ERR_CUDA;
  }
  st = c.head_dim == 128
           ? launch_attention<128>(ctx, p, n_split_final, n_seq, stream, cp.phase != 2, cp.phase != 1, n_packed_tiles)
           : launch_attention<64>(ctx, p, n_split_final, n_seq, stream, cp.phase != 2, cp.phase != 1, n_packed_tiles);
  if (st != VOSTI_OK) return st;
  return release_slot(slot, stream);
}

}  // namespace

extern "C" {

vosti_status vosti_step_host_wait(vosti_ctx* ctx, int64_t ticket) {
  if (!ctx || ticket < 0 || ticket >= ctx->host_steps_issued) return VOSTI_ERR_INVALID_ARG;
  HostStep& h = ctx->host_steps[ticket % kHostSteps];
  if (h.ticket != ticket) return VOSTI_OK;  // a later step took the set, which waited for this one first
  h.ticket = -1;
  return cudaEventSynchronize(h.out_done) == cudaSuccess ? VOSTI_OK : VOSTI_ERR_CUDA;
}

vosti_status vosti_step_host_async(vosti_ctx* ctx, const void* q_host, void* out_host, const void* k_new_host,
                                   const void* v_new_host, const int32_t* q_lens, const int32_t* start_pos,
                                   const int32_t* seq_lens, const int32_t* block_tables,
                                   int32_t block_table_stride, int32_t batch, float softmax_scale,
                                   void* cuda_stream, int64_t* ticket) {
  if (!ctx || batch < 0 || !ticket) return VOSTI_ERR_INVALID_ARG;
  if (batch > 0 && !q_lens) return VOSTI_ERR_INVALID_ARG;
  const vosti_config& c = ctx->cfg;
  int64_t total = 0;
  for (int r = 0; r < batch; ++r) {
    if (q_lens[r] < 0) return VOSTI_ERR_OUT_OF_RANGE;
    total += q_lens[r];
  }
  if (total > c.max_total_q) return VOSTI_ERR_OUT_OF_RANGE;
  if (total > 0 && (!q_host || !out_host || !k_new_host || !v_new_host)) return VOSTI_ERR_INVALID_ARG;
  // The set of the step issued kHostSteps ago is reused: that step must be wholly done.
  HostStep& h = ctx->host_steps[ctx->host_steps_issued % kHostSteps];
  if (h.ticket >= 0) {
    const vosti_status w = vosti_step_host_wait(ctx, h.ticket);
    if (w != VOSTI_OK) return w;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const size_t qbytes = sizeof(__nv_bfloat16) * total * c.n_q_heads * c.head_dim;
  const size_t kbytes = sizeof(__nv_bfloat16) * total * c.n_kv_heads * c.head_dim;
  uint8_t* dq = ctx->ws + ctx->lim.off_stage +
                (ctx->host_steps_issued % kHostSteps) * (2 * ctx->lim.stage_q + 2 * ctx->lim.stage_kv);
  uint8_t* dout = dq + ctx->lim.stage_q;
  uint8_t* dk = dout + ctx->lim.stage_q;
  uint8_t* dv = dk + ctx->lim.stage_kv;
  if (total > 0) {
    // Inputs go up on their own stream, so that they overlap the kernels of the step before.
    if (cudaMemcpyAsync(dq, q_host, qbytes, cudaMemcpyHostToDevice, ctx->in_stream) != cudaSuccess ||
        cudaMemcpyAsync(dk, k_new_host, kbytes, cudaMemcpyHostToDevice, ctx->in_stream) != cudaSuccess ||
        cudaMemcpyAsync(dv, v_new_host, kbytes, cudaMemcpyHostToDevice, ctx->in_stream) != cudaSuccess ||
        cudaEventRecord(h.in_done, ctx->in_stream) != cudaSuccess ||
        cudaStreamWaitEvent(stream, h.in_done, 0) != cudaSuccess)
      return VOSTI_ERR_CUDA;
    vosti_status st =
        vosti_kv_append(ctx, dk, dv, q_lens, start_pos, block_tables, block_table_stride, batch, stream);
    if (st == VOSTI_OK)
      st = vosti_paged_attention(ctx, dq, dout, q_lens, start_pos, seq_lens, block_tables, block_table_stride,
                                 batch, softmax_scale, stream);
    if (st != VOSTI_OK) {
      // Nothing of this step is reported as pending; what was enqueued is drained so that the
      // caller may free its buffers.
      cudaStreamSynchronize(ctx->in_stream);
      cudaStreamSynchronize(stream);
      return st;
    }
    // The output goes down on a third stream, under the kernels of the next step.
    if (cudaEventRecord(h.computed, stream) != cudaSuccess ||
        cudaStreamWaitEvent(ctx->out_stream, h.computed, 0) != cudaSuccess ||
        cudaMemcpyAsync(out_host, dout, qbytes, cudaMemcpyDeviceToHost, ctx->out_stream) != cudaSuccess)
      return VOSTI_ERR_CUDA;
  }
  if (cudaEventRecord(h.out_done, ctx->out_stream) != cudaSuccess) return VOSTI_ERR_CUDA;
  h.ticket = ctx->host_steps_issued;
  *ticket = ctx->host_steps_issued++;
  return VOSTI_OK;
}

vosti_status vosti_step_host(vosti_ctx* ctx, const void* q_host, void* out_host, const void* k_new_host,
                             const void* v_new_host, const int32_t* q_lens, const int32_t* start_pos,
                             const int32_t* seq_lens, const int32_t* block_tables,
                             int32_t block_table_stride, int32_t batch, float softmax_scale,
                             void* cuda_stream) {
  int64_t ticket = -1;
  const vosti_status st =
      vosti_step_host_async(ctx, q_host, out_host, k_new_host, v_new_host, q_lens, start_pos, seq_lens,
                            block_tables, block_table_stride, batch, softmax_scale, cuda_stream, &ticket);
  return st == VOSTI_OK ? vosti_step_host_wait(ctx, ticket) : st;
}

// ---- device-planned steps (graph capture) ------------------------------------------------------

size_t vosti_device_plan_bytes(const vosti_config* config) {
  if (!config || !geometry_ok(*config)) return 0;
  return device_plan_layout(config->max_batch, config->max_total_q, config->max_seq_len).total;
}

namespace {
// Premises every device-planned call shares; host-side, so they are reported at once.
vosti_status planned_call_ok(const vosti_ctx* ctx, const void* plan, const int32_t* block_tables_dev,
                             int32_t batch, int32_t max_q_len) {
  if (!ctx || !plan || batch < 0 || max_q_len < 1) return VOSTI_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(plan) % 16) return VOSTI_ERR_INVALID_ARG;
  if (batch > 0 && !block_tables_dev) return VOSTI_ERR_INVALID_ARG;
  const vosti_config& c = ctx->cfg;
  if (batch > c.max_batch) return VOSTI_ERR_OUT_OF_RANGE;
  if (int64_t{max_q_len} * (c.n_q_heads / c.n_kv_heads) > nc::kSplitRowsMax) return VOSTI_ERR_UNSUPPORTED_CONFIG;
  if (ctx->lim.part_rows_max >= (int64_t{1} << 31)) return VOSTI_ERR_WORKSPACE;  // the planner counts in 32 bits
  return VOSTI_OK;
}
}  // namespace

vosti_status vosti_plan_device(vosti_ctx* ctx, void* plan, const int32_t* q_lens_dev,
                               const int32_t* start_pos_dev, const int32_t* block_tables_dev,
                               int32_t block_table_stride, int32_t batch, int32_t max_q_len, int32_t window,
                               void* cuda_stream) {
  vosti_status st = planned_call_ok(ctx, plan, block_tables_dev, batch, max_q_len);
  if (st != VOSTI_OK) return st;
  if (block_table_stride < 0 || window < 0 || (batch > 0 && (!q_lens_dev || !start_pos_dev)))
    return VOSTI_ERR_INVALID_ARG;
  const vosti_config& c = ctx->cfg;
  const DevicePlanLayout L = device_plan_layout(c.max_batch, c.max_total_q, c.max_seq_len);
  uint8_t* base = static_cast<uint8_t*>(plan);
  DevicePlanArgs a{};
  a.q_lens = q_lens_dev;
  a.start_pos = start_pos_dev;
  a.block_tables = block_tables_dev;
  a.stride = block_table_stride;
  a.batch = batch;
  a.max_q_len = max_q_len;
  a.G = c.n_q_heads / c.n_kv_heads;
  a.Hkv = c.n_kv_heads;
  a.window = window;
  a.num_pages = c.num_pages;
  a.max_seq_len = c.max_seq_len;
  a.items_max = std::min(L.items_max, ctx->lim.items_max);
  a.toks_max = L.toks_max;
  a.part_rows_max = ctx->lim.part_rows_max;
  a.header = reinterpret_cast<DevicePlanHeader*>(base);
  a.reqs = reinterpret_cast<ReqMeta*>(base + L.off_reqs);
  a.items = reinterpret_cast<SplitItem*>(base + L.off_items);
  a.toks = reinterpret_cast<int2*>(base + L.off_toks);
  a.scratch = reinterpret_cast<DevicePlanScratch*>(base + L.off_scratch);
  a.status = reinterpret_cast<uint32_t*>(ctx->ws + ctx->lim.off_status);
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (launch_dependent(device_plan_kernel, 1, batch <= 256 ? 256 : kPlanThreads, 0, stream, a) != cudaSuccess)
    return VOSTI_ERR_CUDA;
  ++ctx->launches;
  return VOSTI_OK;
}

vosti_status vosti_kv_append_planned(vosti_ctx* ctx, const void* plan, const void* k_new, const void* v_new,
                                     const int32_t* block_tables_dev, int32_t batch, int32_t max_q_len,
                                     void* cuda_stream) {
  vosti_status st = planned_call_ok(ctx, plan, block_tables_dev, batch, max_q_len);
  if (st != VOSTI_OK) return st;
  if (batch == 0) return VOSTI_OK;
  if (!k_new || !v_new) return VOSTI_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(k_new) | reinterpret_cast<uintptr_t>(v_new)) % 16) return VOSTI_ERR_INVALID_ARG;
  const vosti_config& c = ctx->cfg;
  const DevicePlanLayout L = device_plan_layout(c.max_batch, c.max_total_q, c.max_seq_len);
  AppendPlannedParams p{};
  p.k_new = static_cast<const __nv_bfloat16*>(k_new);
  p.v_new = static_cast<const __nv_bfloat16*>(v_new);
  p.pool = static_cast<__nv_bfloat16*>(c.kv_pool);
  p.reqs = reinterpret_cast<const ReqMeta*>(static_cast<const uint8_t*>(plan) + L.off_reqs);
  p.block_tables = block_tables_dev;
  p.batch = batch;
  p.max_q_len = max_q_len;
  p.Hkv = c.n_kv_heads;
  p.num_pages = c.num_pages;
  p.status = reinterpret_cast<uint32_t*>(ctx->ws + ctx->lim.off_status);
  const int64_t warps = int64_t{batch} * max_q_len * c.n_kv_heads;
  const int grid = static_cast<int>((warps + 3) / 4);
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const cudaError_t e = c.head_dim == 128
                            ? launch_dependent(kv_append_planned_kernel<128>, grid, 128, 0, stream, p)
                            : launch_dependent(kv_append_planned_kernel<64>, grid, 128, 0, stream, p);
  if (e != cudaSuccess) return VOSTI_ERR_CUDA;
  ++ctx->launches;
  return VOSTI_OK;
}

extern "C++" {
namespace {
template <int D>
vosti_status launch_attention_planned(vosti_ctx* ctx, const AttnParams& p, int64_t workers_bound,
                                      cudaStream_t stream) {
  using Cfg = SplitKernelCfg<D>;
  // The item count is known to the device only: a full persistent grid, whose idle workers leave
  // at once.  The host's bound on it (every request at the longest context the configuration
  // allows) still picks the few-worker variants for small batches; a loose bound costs speed only.
  cudaError_t e;
  if (workers_bound <= 2 * ctx->sm_count)
    e = launch_dependent(attn_split_kernel<D, 2>, ctx->sm_count, 64, SplitKernelCfg<D, 2>::kSmemBytes, stream,
                         ctx->kv_map3, p);
  else if (workers_bound <= 4 * ctx->sm_count)
    e = launch_dependent(attn_split_kernel<D, 4>, ctx->sm_count, 128, SplitKernelCfg<D, 4>::kSmemBytes, stream,
                         ctx->kv_map3, p);
  else
    e = launch_dependent(attn_split_kernel<D>, ctx->sm_count, Cfg::kWarps * 32, Cfg::kSmemBytes, stream,
                         ctx->kv_map3, p);
  if (e != cudaSuccess) return VOSTI_ERR_CUDA;
  const int64_t warps = int64_t{p.n_split_tokens} * p.Hq;
  if (launch_dependent(combine_kernel<D>, static_cast<int>((warps + 3) / 4), 128, 0, stream, p) != cudaSuccess)
    return VOSTI_ERR_CUDA;
  ctx->launches += 2;
  return VOSTI_OK;
}
}  // namespace
}  // extern "C++"

vosti_status vosti_paged_attention_planned(vosti_ctx* ctx, const void* plan, const void* q, void* out, float* lse,
                                           const int32_t* block_tables_dev, int32_t batch, int32_t max_q_len,
                                           float softmax_scale, int32_t window, void* cuda_stream) {
  vosti_status st = planned_call_ok(ctx, plan, block_tables_dev, batch, max_q_len);
  if (st != VOSTI_OK) return st;
  if (window < 0) return VOSTI_ERR_INVALID_ARG;
  if (!(softmax_scale >= 0.0f) || !std::isfinite(softmax_scale)) return VOSTI_ERR_INVALID_ARG;
  if (batch == 0) return VOSTI_OK;
  if (!q || !out) return VOSTI_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(out)) % 16) return VOSTI_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(lse) % 4) return VOSTI_ERR_INVALID_ARG;
  const vosti_config& c = ctx->cfg;
  const DevicePlanLayout L = device_plan_layout(c.max_batch, c.max_total_q, c.max_seq_len);
  const uint8_t* base = static_cast<const uint8_t*>(plan);
  AttnParams p{};
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.out = static_cast<__nv_bfloat16*>(out);
  p.reqs = reinterpret_cast<const ReqMeta*>(base + L.off_reqs);
  p.items = nullptr;
  p.split_items = reinterpret_cast<const SplitItem*>(base + L.off_items);
  p.packed_rows = nullptr;
  p.ticket = reinterpret_cast<uint32_t*>(ctx->ws + ctx->lim.off_status + 64);
  p.done = reinterpret_cast<uint32_t*>(ctx->ws + ctx->lim.off_status + 128);
  p.bt_flat = block_tables_dev;
  p.split_tokens = reinterpret_cast<const int2*>(base + L.off_toks);
  p.ws_u = reinterpret_cast<float*>(ctx->ws + ctx->lim.off_part_u);
  p.ws_mz = reinterpret_cast<float2*>(ctx->ws + ctx->lim.off_part_mz);
  p.ws_uc = reinterpret_cast<float*>(ctx->ws + ctx->lim.off_uc);
  p.status = reinterpret_cast<uint32_t*>(ctx->ws + ctx->lim.off_status);
  p.n_workers = 0;
  p.n_split_tokens = static_cast<int32_t>(std::min<int64_t>(int64_t{batch} * max_q_len, L.toks_max));  // grid bound
  p.Hq = c.n_q_heads;
  p.Hkv = c.n_kv_heads;
  p.G = c.n_q_heads / c.n_kv_heads;
  p.c = static_cast<float>(static_cast<double>(softmax_scale) * 1.4426950408889634074);
  p.window = window;  // the one the plan was made with
  p.lse = lse;
  p.counts = reinterpret_cast<const int32_t*>(base);
  p.num_pages = static_cast<int32_t>(c.num_pages);
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const int64_t groups = (int64_t{max_q_len} * p.G + nc::kRowsPerGroup - 1) / nc::kRowsPerGroup;
  const int64_t workers_bound = int64_t{batch} * groups * ctx->lim.k_max * c.n_kv_heads;
  return c.head_dim == 128 ? launch_attention_planned<128>(ctx, p, workers_bound, stream)
                           : launch_attention_planned<64>(ctx, p, workers_bound, stream);
}

vosti_status vosti_poll_device_status(vosti_ctx* ctx, void* cuda_stream) {
  if (!ctx) return VOSTI_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  uint32_t word = 0;
  uint8_t* d = ctx->ws + ctx->lim.off_status;
  if (cudaMemcpyAsync(&word, d, sizeof word, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
      cudaMemsetAsync(d, 0, kAlign, stream) != cudaSuccess ||
      cudaStreamSynchronize(stream) != cudaSuccess)
    return VOSTI_ERR_CUDA;
  if (word & kStatusTimeout) return VOSTI_ERR_TIMEOUT;
  return (word & kStatusBadMetadata) ? VOSTI_ERR_OUT_OF_RANGE : VOSTI_OK;
}

vosti_status vosti_selftest_bounded_wait(vosti_ctx* ctx, uint32_t limit_us, void* cuda_stream) {
  if (!ctx || limit_us == 0 || limit_us > 100000) return VOSTI_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  bounded_wait_selftest_kernel<<<1, 32, 0, stream>>>(reinterpret_cast<uint32_t*>(ctx->ws + ctx->lim.off_status),
                                                   static_cast<uint64_t>(limit_us) * 1000ull);
  ++ctx->launches;
  return cudaGetLastError() == cudaSuccess ? VOSTI_OK : VOSTI_ERR_CUDA;
}

vosti_status vosti_selftest_mma(vosti_ctx* ctx, const void* a, const void* b, int32_t mode, float* d_tc,
                                float* d_warp, void* cuda_stream) {
  if (!ctx || !a || !b || !d_tc || !d_warp || (mode != 0 && mode != 1)) return VOSTI_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(b)) % 16) return VOSTI_ERR_INVALID_ARG;
  constexpr int kSmem = 128 * 128 + 64 * 128 + 64 + 1024;
  mma_selftest_kernel<<<1, 128, kSmem, static_cast<cudaStream_t>(cuda_stream)>>>(
      static_cast<const __nv_bfloat16*>(a), static_cast<const __nv_bfloat16*>(b), mode, d_tc, d_warp,
      reinterpret_cast<uint32_t*>(ctx->ws + ctx->lim.off_status));
  ++ctx->launches;
  return cudaGetLastError() == cudaSuccess ? VOSTI_OK : VOSTI_ERR_CUDA;
}

vosti_status vosti_profile_enable(vosti_ctx* ctx, int32_t mode) {
  if (!ctx || mode < 0 || mode > 3) return VOSTI_ERR_INVALID_ARG;
  ctx->profile_mode = mode;
  if (mode) ctx->ev_used = 0;
  return VOSTI_OK;
}

vosti_status vosti_profile_read(vosti_ctx* ctx, double* kernel_ms_sum, int64_t* kernels_timed) {
  if (!ctx) return VOSTI_ERR_INVALID_ARG;
  double sum = 0.0;
  for (size_t i = 0; i < ctx->ev_used; ++i) {
    float ms = 0.f;
    if (cudaEventSynchronize(ctx->ev_stop[i]) != cudaSuccess ||
        cudaEventElapsedTime(&ms, ctx->ev_start[i], ctx->ev_stop[i]) != cudaSuccess)
      return VOSTI_ERR_CUDA;
    sum += ms;
  }
  if (kernel_ms_sum) *kernel_ms_sum = sum;
  if (kernels_timed) *kernels_timed = static_cast<int64_t>(ctx->ev_used);
  return VOSTI_OK;
}

int64_t vosti_launch_count(const vosti_ctx* ctx) { return ctx ? ctx->launches : 0; }

vosti_status vosti_host_time(vosti_ctx* ctx, int64_t* nanoseconds, int64_t* calls, int32_t reset) {
  if (!ctx) return VOSTI_ERR_INVALID_ARG;
  if (nanoseconds) *nanoseconds = ctx->host_ns;
  if (calls) *calls = ctx->host_calls;
  if (reset) ctx->host_ns = ctx->host_calls = 0;
  return VOSTI_OK;
}

vosti_status vosti_last_schedule(const vosti_ctx* ctx, int64_t* split_items, int64_t* packed_items,
                                 int64_t* tile_items) {
  if (!ctx) return VOSTI_ERR_INVALID_ARG;
  if (split_items) *split_items = ctx->last_split_items;
  if (packed_items) *packed_items = ctx->last_packed_items;
  if (tile_items) *tile_items = ctx->last_tile_items;
  return VOSTI_OK;
}

}  // extern "C"
