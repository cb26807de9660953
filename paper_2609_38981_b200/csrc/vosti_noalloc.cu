// vosti_paged_attention_noalloc: split-parallel paged attention for callers that
// may not allocate memory.
//
// Who cannot allocate: a serving engine that has reserved all of the GPU's
// memory for its KV pool at start-up and hands the rest out through its own
// pool allocator (a cudaMalloc there fails, or fragments what the engine
// thinks it owns); a latency-critical decode loop, where cudaMalloc and
// cudaFree synchronise the whole device and stall every stream; and plug-ins
// that a host framework gives device pointers but no right to create memory of
// their own.  Such callers cannot build a vosti_ctx either, because
// vosti_create pins host memory and creates streams and events.
//
// This entry point therefore owns NO heap or device allocation.  Everything it
// needs beyond the caller's inputs and outputs lives in one file-scope device
// array, `g_noalloc_scratch` (16 MiB, resident on every GPU that loads the
// library until the process exits): scheduler words, the per-call metadata and
// the partial (m, z, U) rows of the KV splits.  It runs the same kernels as
// vosti_paged_attention (attn_split_kernel + combine_kernel), so its output is
// bit-identical to that entry point's.
//
// The array's name is a host-side stand-in, not a device address: the device
// address is fetched once per device with cudaGetSymbolAddress and that pointer
// is what the kernels receive.
//
// The per-call metadata (request records, work items, page ids) is planned on
// the host at call time and copied from a static host buffer with up to four
// cudaMemcpyAsync calls covering only what the call uses; the source is
// pageable, so the call also waits for earlier work on the stream.
//
// Failure detection: the kernels' bounded waits set the status word at the
// start of the array, as they do in a context's workspace.  The word is sticky
// -- calls do not clear it -- and vosti_noalloc_poll_status reads and clears it.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <mutex>

#include "attn_split.cuh"
#include "aux_kernels.cuh"

namespace vosti {
namespace {

constexpr size_t kScratchBytes = size_t{16} << 20;
constexpr int kMaxDevices = 64;
// Capacities (the documented maxima of the entry point).
constexpr int kMaxBatch = 64;
constexpr int kMaxTotalQ = 256;
constexpr int kMaxItems = 1024;    // split-parallel work items
constexpr int kMaxPageIds = 16384; // page-table entries carried by one call
// Layout of the scratch array.
constexpr size_t kOffWords = 0;                    // status word (sticky until polled), then ticket and done
constexpr size_t kOffTicket = 64;                  // ticket at +64, done at +128: zero at every kernel start
constexpr size_t kOffMeta = 1024;
constexpr size_t kMetaBytes = sizeof(ReqMeta) * kMaxBatch + sizeof(SplitItem) * kMaxItems +
                              sizeof(int32_t) * kMaxPageIds + sizeof(int2) * kMaxTotalQ;
constexpr size_t kOffPartMz = (kOffMeta + kMetaBytes + 1023) / 1024 * 1024;
constexpr int64_t kMaxPartRows = 28000;            // partial rows: (m, z) + U[128] floats each
constexpr size_t kOffPartU = (kOffPartMz + sizeof(float2) * kMaxPartRows + 1023) / 1024 * 1024;
static_assert(kOffPartU + sizeof(float) * kMaxPartRows * 128 <= kScratchBytes, "scratch layout exceeds the array");

}  // namespace
}  // namespace vosti

// The scratch itself.  File scope, static: one copy per loaded module per GPU.
static __device__ __align__(256) unsigned char g_noalloc_scratch[vosti::kScratchBytes];

namespace vosti {
namespace {

std::mutex g_mutex;
unsigned char* g_scratch_ptr[kMaxDevices] = {};   // device address of the array, per device
bool g_ready[kMaxDevices] = {};
alignas(16) unsigned char g_host_blob[kMetaBytes]; // staging for the metadata upload (guarded by g_mutex)

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

// Once per device, with that device current: resolve the array's device address
// and raise the kernels' dynamic shared-memory limit.
vosti_status setup_device(int device) {
  if (g_ready[device]) return VOSTI_OK;
  void* ptr = nullptr;
  if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) return VOSTI_ERR_CUDA;
  if (cudaFuncSetAttribute(attn_split_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           SplitKernelCfg<128>::kSmemBytes) != cudaSuccess ||
      cudaFuncSetAttribute(attn_split_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           SplitKernelCfg<64>::kSmemBytes) != cudaSuccess)
    return VOSTI_ERR_CUDA;
  g_scratch_ptr[device] = static_cast<unsigned char*>(ptr);
  g_ready[device] = true;
  return VOSTI_OK;
}

template <int D>
vosti_status launch(const CUtensorMap& map, const AttnParams& p, int sm_count, cudaStream_t stream) {
  using Cfg = SplitKernelCfg<D>;
  const int grid = std::min((p.n_workers + Cfg::kWarps - 1) / Cfg::kWarps, sm_count);
  attn_split_kernel<D><<<grid, Cfg::kWarps * 32, Cfg::kSmemBytes, stream>>>(map, p);
  const int warps = p.n_split_tokens * p.Hq;
  combine_kernel<D><<<(warps + 3) / 4, 128, 0, stream>>>(p);
  return cudaGetLastError() == cudaSuccess ? VOSTI_OK : VOSTI_ERR_CUDA;
}

}  // namespace
}  // namespace vosti

using namespace vosti;

extern "C" vosti_status vosti_paged_attention_noalloc(
    int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, int32_t page_size, const void* kv_pool,
    int64_t num_pages, const void* q, void* out, const int32_t* q_lens, const int32_t* start_pos,
    const int32_t* seq_lens, const int32_t* block_tables, int32_t block_table_stride, int32_t batch,
    float softmax_scale, void* cuda_stream) {
  // ---- geometry and arguments ------------------------------------------------------
  if ((head_dim != 64 && head_dim != 128) || page_size != nc::kPageSize || n_q_heads <= 0 || n_kv_heads <= 0 ||
      n_q_heads % n_kv_heads || num_pages <= 0 || num_pages * n_kv_heads >= (int64_t{1} << 26))
    return VOSTI_ERR_UNSUPPORTED_CONFIG;
  const int G = n_q_heads / n_kv_heads;
  if (G != 1 && G != 2 && G != 4 && G != 8 && G != 16) return VOSTI_ERR_UNSUPPORTED_CONFIG;
  if (batch < 0 || block_table_stride < 0) return VOSTI_ERR_INVALID_ARG;
  if (!(softmax_scale >= 0.0f) || !std::isfinite(softmax_scale)) return VOSTI_ERR_INVALID_ARG;
  if (batch == 0) return VOSTI_OK;
  if (!kv_pool || !q || !out || !q_lens || !start_pos || !seq_lens || !block_tables) return VOSTI_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(out)) % 16 ||
      reinterpret_cast<uintptr_t>(kv_pool) % 1024)
    return VOSTI_ERR_INVALID_ARG;
  if (batch > kMaxBatch) return VOSTI_ERR_WORKSPACE;  // beyond the static scratch's capacity

  std::lock_guard<std::mutex> lock(g_mutex);  // one metadata staging buffer, one scratch array
  int device = 0, sm_count = 0;
  if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) return VOSTI_ERR_CUDA;
  vosti_status st = setup_device(device);
  if (st != VOSTI_OK) return st;
  if (cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) return VOSTI_ERR_CUDA;
  unsigned char* scratch = g_scratch_ptr[device];

  // ---- plan: every request must be split-parallel; everything must fit the scratch -----
  unsigned char* blob = g_host_blob;
  ReqMeta* reqs = reinterpret_cast<ReqMeta*>(blob);
  SplitItem* items = reinterpret_cast<SplitItem*>(blob + sizeof(ReqMeta) * kMaxBatch);
  int32_t* bt_flat = reinterpret_cast<int32_t*>(blob + sizeof(ReqMeta) * kMaxBatch + sizeof(SplitItem) * kMaxItems);
  int2* toks = reinterpret_cast<int2*>(blob + sizeof(ReqMeta) * kMaxBatch + sizeof(SplitItem) * kMaxItems +
                                       sizeof(int32_t) * kMaxPageIds);
  int64_t row0 = 0, bt_used = 0, n_items = 0, part_rows = 0, n_tok = 0;
  for (int r = 0; r < batch; ++r) {
    const int64_t ql = q_lens[r], sp = start_pos[r], sl = seq_lens[r];
    if (ql < 0 || sp < 0 || sp + ql > sl || sl >= (int64_t{1} << 30)) return VOSTI_ERR_OUT_OF_RANGE;
    ReqMeta& m = reqs[r];
    m.q_row0 = static_cast<int32_t>(row0);
    m.q_len = static_cast<int32_t>(ql);
    m.start = static_cast<int32_t>(sp);
    m.n_pages = 0;
    m.bt_off = static_cast<int32_t>(bt_used);
    m.n_splits = 0;
    m.first_split = 0;
    m.pad = 0;
    m.part_base = part_rows;
    row0 += ql;
    if (ql == 0) continue;
    const int64_t rows = ql * G;
    if (rows > nc::kSplitRowsMax) return VOSTI_ERR_UNSUPPORTED_CONFIG;  // long queries need vosti_paged_attention
    const int64_t n_eff = sp + ql;
    const int64_t n_pages = (n_eff + page_size - 1) / page_size;
    if (n_pages > block_table_stride || (sl + page_size - 1) / page_size > block_table_stride)
      return VOSTI_ERR_OUT_OF_RANGE;
    const int64_t n_splits = (n_eff - 1) / nc::kSplitLen + 1;
    if (row0 > kMaxTotalQ || bt_used + n_pages > kMaxPageIds ||
        part_rows + int64_t{n_kv_heads} * n_splits * rows > kMaxPartRows)
      return VOSTI_ERR_WORKSPACE;
    const int32_t* row = block_tables + static_cast<size_t>(r) * block_table_stride;
    for (int64_t b = 0; b < n_pages; ++b) {
      if (row[b] < 0 || row[b] >= num_pages) return VOSTI_ERR_OUT_OF_RANGE;
      bt_flat[bt_used + b] = row[b];
    }
    m.n_pages = static_cast<int32_t>(n_pages);
    m.n_splits = static_cast<int32_t>(n_splits);
    const int groups = static_cast<int>((rows + nc::kRowsPerGroup - 1) / nc::kRowsPerGroup);
    for (int g = 0; g < groups; ++g) {
      const int64_t last_tok = std::min<int64_t>(ql - 1, (int64_t{g} * nc::kRowsPerGroup + 15) / G);
      const int k_g = static_cast<int>((sp + last_tok) / nc::kSplitLen + 1);
      if (n_items + k_g > kMaxItems) return VOSTI_ERR_WORKSPACE;
      for (int k = 0; k < k_g; ++k) {
        SplitItem& si = items[n_items++];
        si.q_row0 = m.q_row0; si.q_len = m.q_len; si.start = m.start; si.n_pages = m.n_pages;
        si.bt_index = m.bt_off + k * nc::kPagesPerSplit;
        si.split = k; si.row_group = g; si.n_splits = m.n_splits;
        si.part_base = m.part_base; si.req = r; si.first_split = 0;
      }
    }
    for (int i = 0; i < ql; ++i) toks[n_tok++] = make_int2(r, i);
    bt_used += n_pages;
    part_rows += int64_t{n_kv_heads} * n_splits * rows;
  }
  if (n_items == 0) return VOSTI_OK;

  // ---- tensor map of the caller's pool (host-side encode, no allocation) ----------------
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !fn)
    return VOSTI_ERR_CUDA;
  alignas(64) CUtensorMap map;  // the 3-D page map the split kernel gathers with: (64, rows, d/64)
  {
    const cuuint64_t dims[3] = {64, static_cast<cuuint64_t>(num_pages) * n_kv_heads * 2 * page_size,
                                static_cast<cuuint64_t>(head_dim / 64)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(head_dim) * 2, 128};
    const cuuint32_t box[3] = {64, static_cast<cuuint32_t>(page_size), static_cast<cuuint32_t>(head_dim / 64)};
    const cuuint32_t estr[3] = {1, 1, 1};
    if (reinterpret_cast<EncodeTiledFn>(fn)(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(kv_pool),
                                            dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return VOSTI_ERR_CUDA;
  }

  // ---- upload metadata, clear what must start at zero, launch ------------------------------
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  // The scheduler words (ticket, done) keep whatever the last call left; they must be zero at
  // kernel start.  The status word before them is left alone: it is sticky until polled.
  if (cudaMemsetAsync(scratch + kOffWords + kOffTicket, 0, 1024 - kOffTicket, stream) != cudaSuccess)
    return VOSTI_ERR_CUDA;
  // Only what this call uses goes up.  The source is pageable, so each copy returns once the
  // runtime has staged it (after earlier work on the stream): the static host buffer is then free.
  unsigned char* dmeta = scratch + kOffMeta;
  const size_t off_items = sizeof(ReqMeta) * kMaxBatch, off_bt = off_items + sizeof(SplitItem) * kMaxItems,
               off_toks = off_bt + sizeof(int32_t) * kMaxPageIds;
  if (cudaMemcpyAsync(dmeta, blob, sizeof(ReqMeta) * batch, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
      cudaMemcpyAsync(dmeta + off_items, blob + off_items, sizeof(SplitItem) * n_items, cudaMemcpyHostToDevice,
                      stream) != cudaSuccess ||
      cudaMemcpyAsync(dmeta + off_bt, blob + off_bt, sizeof(int32_t) * bt_used, cudaMemcpyHostToDevice, stream) !=
          cudaSuccess ||
      cudaMemcpyAsync(dmeta + off_toks, blob + off_toks, sizeof(int2) * n_tok, cudaMemcpyHostToDevice, stream) !=
          cudaSuccess)
    return VOSTI_ERR_CUDA;
  AttnParams p;
  p.beside_split = 0;
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.out = static_cast<__nv_bfloat16*>(out);
  p.reqs = reinterpret_cast<const ReqMeta*>(dmeta);
  p.items = nullptr;
  p.split_items = reinterpret_cast<const SplitItem*>(dmeta + off_items);
  p.ticket = reinterpret_cast<uint32_t*>(scratch + kOffWords + kOffTicket);
  p.done = reinterpret_cast<uint32_t*>(scratch + kOffWords + kOffTicket + 64);
  p.bt_flat = reinterpret_cast<const int32_t*>(dmeta + off_bt);
  p.split_tokens = reinterpret_cast<const int2*>(dmeta + off_toks);
  p.ws_u = reinterpret_cast<float*>(scratch + kOffPartU);
  p.ws_mz = reinterpret_cast<float2*>(scratch + kOffPartMz);
  p.ws_uc = nullptr;
  p.status = reinterpret_cast<uint32_t*>(scratch + kOffWords);
  p.n_workers = static_cast<int32_t>(n_items * n_kv_heads);
  p.n_split_tokens = static_cast<int32_t>(n_tok);
  p.Hq = n_q_heads;
  p.Hkv = n_kv_heads;
  p.G = G;
  p.c = static_cast<float>(static_cast<double>(softmax_scale) * 1.4426950408889634074);
  p.window = 0;
  p.lse = nullptr;
  p.counts = nullptr;
  p.num_pages = 0;
  p.tile_pack_items = nullptr;
  p.tile_rows = nullptr;
  p.packed_rows = nullptr;
  return head_dim == 128 ? launch<128>(map, p, sm_count, stream) : launch<64>(map, p, sm_count, stream);
}

// Shared by the two status calls: the current device's scratch address (set-up on first use).
static vosti_status noalloc_scratch_of_current_device(unsigned char** scratch) {
  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) return VOSTI_ERR_CUDA;
  const vosti_status st = setup_device(device);
  if (st == VOSTI_OK) *scratch = g_scratch_ptr[device];
  return st;
}

extern "C" vosti_status vosti_noalloc_poll_status(void* cuda_stream) {
  std::lock_guard<std::mutex> lock(g_mutex);
  unsigned char* scratch = nullptr;
  const vosti_status st = noalloc_scratch_of_current_device(&scratch);
  if (st != VOSTI_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  uint32_t word = 0;  // a stack word: the copy is staged by the runtime, nothing is allocated here
  if (cudaMemcpyAsync(&word, scratch + kOffWords, sizeof word, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
      cudaMemsetAsync(scratch + kOffWords, 0, sizeof word, stream) != cudaSuccess ||
      cudaStreamSynchronize(stream) != cudaSuccess)
    return VOSTI_ERR_CUDA;
  if (word & kStatusTimeout) return VOSTI_ERR_TIMEOUT;
  return (word & kStatusBadMetadata) ? VOSTI_ERR_OUT_OF_RANGE : VOSTI_OK;
}

extern "C" vosti_status vosti_noalloc_selftest_bounded_wait(uint32_t limit_us, void* cuda_stream) {
  if (limit_us == 0 || limit_us > 100000) return VOSTI_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_mutex);
  unsigned char* scratch = nullptr;
  const vosti_status st = noalloc_scratch_of_current_device(&scratch);
  if (st != VOSTI_OK) return st;
  bounded_wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      reinterpret_cast<uint32_t*>(scratch + kOffWords), static_cast<uint64_t>(limit_us) * 1000ull);
  return cudaGetLastError() == cudaSuccess ? VOSTI_OK : VOSTI_ERR_CUDA;
}
