// Per-call metadata that the host planner writes and the kernels read.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

#include "../../include/vosti.h"

namespace vosti {

// Bits of the device status word.
constexpr uint32_t kStatusTimeout = 1u;      // a bounded wait gave up
constexpr uint32_t kStatusBadMetadata = 2u;  // a device-planned step met lengths / page ids outside the premises

// One request of a call, as the kernels see it.
struct ReqMeta {
  int32_t q_row0;     // first packed row of the request
  int32_t q_len;      // query rows (tokens)
  int32_t start;      // logical position of row 0
  int32_t n_pages;    // used pages = ceil((start + q_len) / P)
  int32_t bt_off;     // offset of the request's page ids in the flat table
  int32_t n_splits;   // splits the request's rows touch: last split - first_split + 1
  int32_t first_split;  // first split any row of the request sees (0 without a sliding window)
  int32_t pad;
  int64_t part_base;  // first partial row of the request (split-parallel requests only)
};

// One split-parallel work item, self-contained so that a persistent warp needs
// a single record per ticket.  48 bytes.
struct SplitItem {
  int32_t q_row0, q_len, start, n_pages;
  int32_t bt_index;  // index in the flat table of the first page of this split
  int32_t split, row_group, n_splits;
  int64_t part_base;
  int32_t req;          // < 0: packed item (rows from packed_rows[16 * (-1 - req) ...], q_len = rows in use)
  int32_t first_split;  // of the request: partial slabs are indexed by split - first_split
};
static_assert(sizeof(SplitItem) == 48, "SplitItem is read as three 16-byte words");

// One row of a packed split item: rows of different requests whose block tables name the
// same physical pages for a whole split share one 16-row MMA tile, so the split is read
// once for all of them.  16 bytes; a packed item owns 16 consecutive entries.
struct PackedRow {
  int32_t q_row_g;     // packed query token row (low 24 bits) and head within the KV group (high 8 bits)
  int32_t p;           // logical position of the row
  int32_t slab_row;    // partial row for KV head 0: part_base + split * rows + row of the request
  int32_t kvh_stride;  // partial rows between consecutive KV heads of the request: n_splits * rows
};

struct AttnParams {
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  const ReqMeta* reqs;
  const vosti_work_item* items;    // sequential items
  const SplitItem* split_items;    // split-parallel items, longest first; req < 0: packed item -1 - req
  const PackedRow* packed_rows;    // 16 per packed item
  uint32_t* ticket;                // next split-parallel worker index (self-resetting)
  uint32_t* done;                  // warps that have left the persistent kernel
  const int32_t* bt_flat;
  const int2* split_tokens;  // (request, token) of every row the combine kernel finishes
  float* ws_u;               // partial U rows [rows][D]
  float2* ws_mz;             // partial (m, z) per row
  float* ws_uc;              // running fold of the tile kernel: per CTA 2 x [D/4][128] float4
  uint32_t* status;
  int32_t n_workers;         // items of this launch times n_kv_heads
  int32_t n_split_tokens;
  int32_t Hq, Hkv, G;
  float c;                   // sigma * log2(e), rounded once on the host
  int32_t window;            // sliding window w: key j visible iff p - w < j <= p; 0 = no window
  float* lse;                // optional [T][Hq] natural-log log-sum-exp output, or nullptr
  // Device-planned calls: {n_workers, n_split_tokens} written by the planning kernel earlier in
  // the stream (the two fields above are then only upper bounds for the grids); nullptr otherwise.
  const int32_t* counts;
  // Shared-split packing through the tile kernel: per packed tile {index of the split's first page id in
  // the flat table, split, rows in use, 0} and 128 row records; nullptr when there are none.
  const int4* tile_pack_items;
  const PackedRow* tile_rows;
  int32_t num_pages;         // device-planned calls: page ids are checked against it when an item is drawn
  // Tile kernel launched right behind a split-parallel kernel of the same call, whose results it does
  // not read: it does not wait for that kernel before it starts (the two run side by side) but before
  // it ends, so that the kernel after it, which waits for this one, has waited for both.
  int32_t beside_split;
};

struct AppendParams {
  static constexpr int kInlineSlots = 256;
  const __nv_bfloat16* k_new;
  const __nv_bfloat16* v_new;
  __nv_bfloat16* pool;
  const int32_t* slot;  // per token: page * P + slot; nullptr: use inline_slot
  int32_t n_tokens, Hkv;
  int32_t inline_slot[kInlineSlots];
};

}  // namespace vosti
