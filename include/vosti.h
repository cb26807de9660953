/*
 * vosti.h -- C ABI of libvosti: batch-invariant paged attention for NVIDIA
 * B200 (sm_100a).
 *
 * One attention operation over a prefix-sharing paged KV cache whose output
 * for a logical (request content, token position, query head) has the same
 * bits however it is run: alone or co-batched, any prefill chunk size,
 * multi-token (prefill / speculative) or single-token (decode) query, any
 * physical page placement, shared or private prefix pages.  This is the
 * kernel-level contract of the paper's Sec. "Kernel contracts" and App. A
 * ("Verifying Paged Attention"): equal logical inputs give bitwise-equal
 * selected outputs across batch, query length, row index and page table.
 *
 * Conventions
 *   - "device" pointers are CUDA device memory of the context's GPU, "host"
 *     pointers ordinary host memory.  bf16 = 16-bit brain float.
 *   - Packed rows: [T, H, d] with T = sum of q_lens, request-major,
 *     token-minor (the paper's packed rows).  Row i of request r stands at
 *     logical position p = start_pos[r] + i  (Sec. "The causal contract":
 *     p = k_len - q_len + i) and attends keys 0..p of that request.
 *   - Logical cache through the page table (App. A):
 *         K[j,:] = K_phys[ block_table[r][j / P], j mod P, : ]   (V alike)
 *   - Pool layout:  kv_pool[page][kv_head][0=K,1=V][slot 0..P-1][e 0..d-1]
 *     bf16, so one (page, kv_head, K|V) chunk is P*d*2 contiguous bytes.
 *   - Query head h reads KV head h / (n_q_heads / n_kv_heads).
 *   - Every call is asynchronous on the given CUDA stream (cudaStream_t
 *     passed as void*; NULL = the legacy default stream).  Host metadata
 *     arrays are copied before the call returns and may be reused at once.
 *   - A context must be driven from one stream at a time: calls that overlap
 *     on the GPU share the workspace and race.
 *   - Errors are returned as status codes; nothing aborts, nothing falls
 *     back to another implementation.  On any error no kernel was launched
 *     unless the status is VOSTI_ERR_CUDA / VOSTI_ERR_TIMEOUT.
 *
 * Numerics are frozen at build time (key tile 64, KV split length 512, the
 * fold and exponent rules): vosti_fingerprint() hashes them.  Outputs are
 * comparable bit for bit only under one fingerprint on one GPU model.
 */
#ifndef VOSTI_H_
#define VOSTI_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct vosti_ctx vosti_ctx;

typedef enum {
  VOSTI_OK = 0,
  VOSTI_ERR_INVALID_ARG = 1,        /* null pointer, negative size, bad scale */
  VOSTI_ERR_UNSUPPORTED_CONFIG = 2, /* geometry outside the frozen set */
  VOSTI_ERR_OUT_OF_RANGE = 3,       /* lengths / page ids violate the call premises */
  VOSTI_ERR_WORKSPACE = 4,          /* workspace too small or misaligned */
  VOSTI_ERR_CUDA = 5,               /* a CUDA runtime / driver call failed */
  VOSTI_ERR_TIMEOUT = 6             /* a bounded device-side wait gave up */
} vosti_status;

enum {
  VOSTI_FLAG_CHECK_WRITE_SLOTS = 1, /* kv_append verifies that write slots are pairwise disjoint */
  /* Shared-prefix row packing, a scheduling decision that cannot change a bit
   * (Sec. "Separate cache reuse from generation": requests that reuse a cached
   * prefix name the same physical pages).  Among the split-parallel requests of
   * a call (decode, speculative), rows of different requests whose block tables
   * hold the same 32 page ids for a whole 512-key split that lies wholly below
   * their positions are packed 16 to an MMA tile: the split is fetched and
   * multiplied once per 16 rows instead of once per request.  Every row still
   * receives its own partial (m, z, U) for that split, computed from the same
   * keys in the same order, and the fold is unchanged, so outputs are bitwise
   * those of the unpacked schedule (tested by comparing the two).  Applies when
   * window == 0.  When the groups of 48 rows or more hold at least 4096 rows x
   * splits between them, those groups are packed 128 rows to a tile of the
   * tensor-memory kernel instead (one more kernel launch per call, an eighth
   * of the reads of the shared pages); same partials, same bits. */
  VOSTI_FLAG_PACK_SHARED_SPLITS = 2,
  /* With PACK_SHARED_SPLITS: groups of 48 rows or more always go through the
   * tensor-memory kernel, however little they hold (tests; callers that know
   * their steps are bound by the GPU and not by the host). */
  VOSTI_FLAG_PACK_THROUGH_TILES = 4,
  /* A call that launches both the split-parallel kernel (decode and other short
   * queries) and the tensor-memory tile kernel (prefill chunks, packed tiles)
   * runs the two side by side on every SM: they read nothing of each other and
   * are bound by different units.  This flag runs them one after the other
   * instead (tests compare the two schedules bit for bit; measurements). */
  VOSTI_FLAG_NO_OVERLAP = 8
};

/* The fixed deployment configuration (Sec. "Fixed kernel choices": tile
 * parameters are bound at initialisation from model and deployment only; a
 * configuration outside the supported set is rejected, never auto-tuned).
 * Supported: head_dim in {64, 128}; page_size 16; n_q_heads a multiple of
 * n_kv_heads with ratio in {1, 2, 4, 8, 16}. */
typedef struct {
  int32_t n_q_heads, n_kv_heads, head_dim, page_size;
  int64_t num_pages;      /* pages in kv_pool */
  void* kv_pool;          /* device, caller-owned, 1024-byte aligned, layout above */
  int32_t max_batch;      /* largest `batch` of any call */
  int64_t max_total_q;    /* largest sum of q_lens of any call */
  int64_t max_seq_len;    /* largest seq_len of any request */
  void* workspace;        /* device, caller-owned, 1024-byte aligned */
  size_t workspace_bytes; /* >= vosti_workspace_bytes(config) */
  uint32_t flags;         /* VOSTI_FLAG_* */
} vosti_config;

/* One unit of scheduled work (App. A: the kernel's parallel loop over query
 * tiles and heads; the KV split is this library's addition).  Rows of a
 * request are numbered token*G + head_in_group; row group g holds rows
 * 16g..16g+15.  A split-parallel item is one row group and one KV split
 * (split_end = split_begin + 1); a sequential item is a tile of sixteen row
 * groups starting at row_group (256 rows) that walks splits 0..split_end-1 of
 * 512 keys each in order.  Every item is run once per KV head. */
typedef struct {
  int32_t req, row_group, split_begin, split_end;
} vosti_work_item;

/* Device workspace the configuration needs (host-only; reads no pointer
 * field).  Returns 0 if the geometry is unsupported. */
size_t vosti_workspace_bytes(const vosti_config* config);

/* Work planning (host-only, no GPU needed).  Writes up to `cap` items to
 * `items` (may be NULL with cap 0) and the total count to *n_items; *n_split
 * receives how many leading items are split-parallel (they emit one partial
 * (m, z, U) per split, folded later in split order), the rest walk their
 * splits in order and fold in place; *n_partial_rows the number of partial
 * rows.  The plan of a request is a pure function of its own
 * (q_len, start_pos) and the geometry: never of batch size, other requests,
 * page ids or table width (Sec. "Fixed kernel choices").  Only the order of
 * items (longest first) depends on the batch; results do not depend on it.
 * Premises checked: q_len >= 0, start_pos >= 0, start_pos + q_len <= seq_len
 * <= max_seq_len, batch <= max_batch, sum q_len <= max_total_q. */
vosti_status vosti_plan(const vosti_config* config, const int32_t* q_lens, const int32_t* start_pos,
                        const int32_t* seq_lens, int32_t batch, vosti_work_item* items, int64_t cap,
                        int64_t* n_items, int64_t* n_split, int64_t* n_partial_rows);

/* The same plan under a sliding window of `window` keys (0: none; < 0 is
 * INVALID_ARG): a row group only gets items for the splits that hold a key
 * some row of the group sees (App. A, masks: the window adds j > p - w), and
 * partial rows are counted from the first split the request's first row sees.
 * A sequential item reports in split_begin / split_end the splits it walks. */
vosti_status vosti_plan_ex(const vosti_config* config, const int32_t* q_lens, const int32_t* start_pos,
                           const int32_t* seq_lens, int32_t batch, int32_t window,
                           vosti_work_item* items, int64_t cap, int64_t* n_items, int64_t* n_split,
                           int64_t* n_partial_rows);

/* Create a context on the current CUDA device: checks the geometry, builds
 * the TMA tensor map of the pool, allocates host staging (the only memory
 * the library owns) and clears the device status word.  Synchronous. */
vosti_status vosti_create(vosti_ctx** out, const vosti_config* config);
vosti_status vosti_destroy(vosti_ctx* ctx);

/* KV write into page slots (Sec. "Separate cache reuse from generation": new
 * K/V values go to the request's private suffix slots; shared or registered
 * prefix pages stay immutable -- keeping write slots off shared pages is the
 * caller's premise).  Token i of request r is written to page
 * block_tables[r][(start_pos[r]+i) / P], slot (start_pos[r]+i) mod P, for
 * every KV head.  Bit-exact copy.
 *   k_new, v_new   device [T, n_kv_heads, d] bf16, 16-byte aligned
 *   q_lens, start_pos   host [batch]
 *   block_tables   host [batch, block_table_stride]; only entries that a
 *                  written position indexes are read
 * Errors: OUT_OF_RANGE if a position falls outside the table or a page id
 * outside the pool, or (with VOSTI_FLAG_CHECK_WRITE_SLOTS) two tokens share
 * a slot. */
vosti_status vosti_kv_append(vosti_ctx* ctx, const void* k_new, const void* v_new,
                             const int32_t* q_lens, const int32_t* start_pos,
                             const int32_t* block_tables, int32_t block_table_stride, int32_t batch,
                             void* cuda_stream);

/* Causal GQA attention over the paged cache (App. A, "A Simplified Tile IR":
 * tiled online softmax with fp32 state (m, z, U), base-two exponent,
 * weights cast to bf16 before the second product, identity step for rows
 * that see nothing of a tile, O = U * (z > 0 ? 1/z : 0)).  Reads only the
 * pool: the chunk's own tokens must have been appended first (that is how
 * prefill and decode see the same keys).
 *   q, out        device [T, n_q_heads, d] bf16, 16-byte aligned; every out row is overwritten
 *   q_lens, start_pos, seq_lens   host [batch]; q_len == 0 skips the request
 *   block_tables  host [batch, block_table_stride]; only the entries
 *                 0 .. ceil((start_pos+q_len)/P)-1 of a row are read
 *   softmax_scale natural-log scale sigma >= 0, finite (scores are sigma * q.k)
 * Keys j > p are never visible; slots at or beyond start_pos+q_len may hold
 * anything (they are zero-filled on chip), all other inputs must be finite
 * (the paper's unchecked finiteness premise).
 * Errors: OUT_OF_RANGE for violated premises (start_pos+q_len > seq_len,
 * seq_len > max_seq_len, table too short, page id outside the pool, batch or
 * total rows above the configured maxima). */
vosti_status vosti_paged_attention(vosti_ctx* ctx, const void* q, void* out, const int32_t* q_lens,
                                   const int32_t* start_pos, const int32_t* seq_lens,
                                   const int32_t* block_tables, int32_t block_table_stride,
                                   int32_t batch, float softmax_scale, void* cuda_stream);

/* vosti_paged_attention with the two options of App. A:
 *   window   sliding window w >= 0 (App. A, masks: a window adds j > p - w to
 *            the causal mask, so the row at p sees keys max(0, p-w+1) .. p);
 *            0 means no window and gives exactly vosti_paged_attention.  Key
 *            tiles and KV splits stay absolute (counted from key 0), so the
 *            bits of a row still depend only on its own (p, head), the keys it
 *            sees, sigma and w -- and with w > p they equal the unwindowed bits.
 *            Block-table entries of pages that lie wholly before the window of
 *            the request's first row, i.e. entries b < max(0, start_pos-w+1)/P,
 *            are not read: the caller may have released those pages.
 *   lse      device [T, n_q_heads] fp32, 4-byte aligned, or NULL: receives the
 *            auxiliary log-sum-exp of the scaled scores over the visible keys
 *            (App. A, after the output equation), natural logarithm:
 *            (m + log2 z) ln 2 from the same folded (m, z) the output uses, so
 *            it is batch-invariant bit for bit as well.
 * All other arguments, premises and errors as for vosti_paged_attention;
 * window < 0 is INVALID_ARG. */
vosti_status vosti_paged_attention_ex(vosti_ctx* ctx, const void* q, void* out, float* lse,
                                      const int32_t* q_lens, const int32_t* start_pos,
                                      const int32_t* seq_lens, const int32_t* block_tables,
                                      int32_t block_table_stride, int32_t batch, float softmax_scale,
                                      int32_t window, void* cuda_stream);

/* Context-parallel decode (the paper's discussion of multi-GPU determinism,
 * Sec. "Discussion": distributed KV must not change a request's bits).  The KV
 * pages of a long request are spread over `cp_world` GPUs by split: split k
 * (keys 512 k .. 512 k + 511) lives on rank k mod cp_world.  Each rank runs
 *   vosti_cp_partial   -- the partial (m, z, U) of the splits it owns, from its
 *                         own pool and block table (entries of other ranks'
 *                         splits are not read); the slabs of all other splits
 *                         are set to zero;
 *   an exchange        -- that gives every rank every split's partial rows in
 *                         the two workspace ranges this call reports: an
 *                         all-gather of the rows each rank owns (listed by
 *                         vosti_cp_segments; half the volume of the
 *                         alternative), or a sum over ranks of the whole
 *                         ranges (fp32 all-reduce: x + 0 = x; zeros may change
 *                         sign, which the output rule absorbs);
 *   vosti_cp_combine   -- the left fold over all splits and the output, on any
 *                         rank that wants the result.
 * The fold sees the same partials in the same order as a single-GPU call, so
 * outputs and log-sum-exp are bitwise those of vosti_paged_attention.  Only
 * split-parallel requests (q_len * group size <= 32: decode, speculative
 * queries) are accepted (UNSUPPORTED_CONFIG otherwise); no sliding window.
 * *u_offset / *u_bytes and *mz_offset / *mz_bytes are byte ranges inside the
 * context's workspace; q and the three length arrays must be the same on every
 * rank and in both calls. */
vosti_status vosti_cp_partial(vosti_ctx* ctx, const void* q, const int32_t* q_lens,
                              const int32_t* start_pos, const int32_t* seq_lens,
                              const int32_t* block_tables, int32_t block_table_stride, int32_t batch,
                              float softmax_scale, int32_t cp_rank, int32_t cp_world, size_t* u_offset,
                              size_t* u_bytes, size_t* mz_offset, size_t* mz_bytes, void* cuda_stream);
vosti_status vosti_cp_combine(vosti_ctx* ctx, void* out, float* lse, const int32_t* q_lens,
                              const int32_t* start_pos, const int32_t* seq_lens, int32_t batch,
                              void* cuda_stream);

/* The exchange plan of a context-parallel call (host-only, needs no GPU): the
 * partial rows that rank cp_rank of cp_world writes, as segments (first row,
 * number of rows) in ascending order; rows index both ranges vosti_cp_partial
 * reports ([row][head_dim] fp32 and [row] (m, z)).  The segments of all ranks
 * are disjoint and together cover rows 0 .. *n_partial_rows - 1.  Writes
 * min(*n_segments, cap) segments as pairs of int64; a first call with cap = 0
 * sizes the array.  Same premises and errors as vosti_plan; requests with long
 * queries give UNSUPPORTED_CONFIG. */
vosti_status vosti_cp_segments(const vosti_config* config, const int32_t* q_lens,
                               const int32_t* start_pos, const int32_t* seq_lens, int32_t batch,
                               int32_t cp_rank, int32_t cp_world, int64_t* segments, int64_t cap,
                               int64_t* n_segments, int64_t* n_partial_rows);

/* One serving step from HOST buffers: copies q, k_new, v_new to the device,
 * runs vosti_kv_append then vosti_paged_attention, copies the output back
 * and waits for it.  Same arithmetic, same kernels; exists so that a caller
 * (and the end-to-end benchmark) can drive the path without device tensors.
 *   q_host, out_host     host [T, n_q_heads, d] bf16 (pinned memory makes the copies asynchronous)
 *   k_new_host, v_new_host   host [T, n_kv_heads, d] bf16
 * Synchronous: returns after out_host is complete. */
vosti_status vosti_step_host(vosti_ctx* ctx, const void* q_host, void* out_host,
                             const void* k_new_host, const void* v_new_host, const int32_t* q_lens,
                             const int32_t* start_pos, const int32_t* seq_lens,
                             const int32_t* block_tables, int32_t block_table_stride, int32_t batch,
                             float softmax_scale, void* cuda_stream);

/* The same step without the wait, for callers that keep several steps in
 * flight: inputs go up on a stream of the context while the previous step's
 * kernels run on `cuda_stream`, and the output comes down on another while the
 * next step's kernels run.  Steps execute in the order issued (KV appended by
 * one is visible to the next); the kernels, the plan and therefore the bits
 * are those of vosti_step_host.  The int32 arrays are read before the call
 * returns; q_host, k_new_host, v_new_host must stay unchanged, and out_host is
 * not valid, until vosti_step_host_wait(ctx, *ticket) has returned.  Up to
 * VOSTI_HOST_STEPS_IN_FLIGHT steps may be pending; issuing one more first
 * waits for the oldest.  Host buffers should be pinned (pageable memory makes
 * the copies synchronous).  All steps of a context must use one cuda_stream. */
#define VOSTI_HOST_STEPS_IN_FLIGHT 3
vosti_status vosti_step_host_async(vosti_ctx* ctx, const void* q_host, void* out_host,
                                   const void* k_new_host, const void* v_new_host,
                                   const int32_t* q_lens, const int32_t* start_pos,
                                   const int32_t* seq_lens, const int32_t* block_tables,
                                   int32_t block_table_stride, int32_t batch, float softmax_scale,
                                   void* cuda_stream, int64_t* ticket);
/* Blocks until the step's out_host is complete.  A ticket already waited for
 * (explicitly, or because a later step reused its staging) returns at once;
 * INVALID_ARG for a ticket never issued. */
vosti_status vosti_step_host_wait(vosti_ctx* ctx, int64_t ticket);

/* Device-planned steps, for decode loops replayed from a CUDA graph.  (The
 * paper has no counterpart: this is the planning of the operation above moved
 * to the GPU, not a different computation.)
 *
 * vosti_paged_attention reads its lengths and block tables on the host, so a
 * captured graph would replay the metadata of the step it was captured on.
 * Here q_lens, start_pos and block_tables live in DEVICE memory and may change
 * between replays; a planning kernel turns them into the same work items the
 * host planner makes, and the append / attention / combine kernels read those.
 * None of the three calls below synchronises, allocates, creates events or
 * reads device memory on the host: all may be issued while a stream is being
 * captured, and the captured graph replayed with other metadata, Q, K/V rows
 * and output contents at the same addresses.  Output bits are those of
 * vosti_kv_append + vosti_paged_attention for the same logical requests.
 *
 * Only split-parallel requests: every q_len * (n_q_heads / n_kv_heads) <= 32
 * (decode, speculative queries); max_q_len bounds every q_len and must satisfy
 * the same limit (UNSUPPORTED_CONFIG otherwise).  Rows of q / k_new / v_new /
 * out are packed in request order (sum of q_lens rows), as in the host-planned
 * calls; seq_len of a request is start_pos + q_len.  `window` is the sliding
 * window of vosti_paged_attention_ex (0 = none), a host value fixed at
 * capture; the attention call must be given the window its plan was made
 * with.  Block-table entries wholly before the window of a request's first row
 * are not looked at (the caller may have given those pages back).
 *
 *   plan            device, vosti_device_plan_bytes(config) bytes, 16-byte
 *                   aligned; written by vosti_plan_device, read by the other
 *                   two; may be shared by contexts of equal configuration
 *                   limits (one plan per step, one context per layer)
 *   q_lens_dev, start_pos_dev   device [batch] int32
 *   block_tables_dev            device [batch][block_table_stride] int32
 *   batch, max_q_len, block_table_stride   host values, fixed at capture
 * Metadata cannot be checked on the host.  The planning kernel checks it:
 * a request with lengths outside the premises (negative, q_len > max_q_len,
 * start_pos + q_len > max_seq_len or beyond block_table_stride pages) is
 * treated as empty, a page id outside the pool is never written to (reads of
 * it return zeros), a batch that exceeds the workspace runs nothing; in each
 * case the device status word is set and the next vosti_poll_device_status
 * returns VOSTI_ERR_OUT_OF_RANGE.  Errors detectable from the host values are
 * returned by the call as usual. */
size_t vosti_device_plan_bytes(const vosti_config* config);
vosti_status vosti_plan_device(vosti_ctx* ctx, void* plan, const int32_t* q_lens_dev,
                               const int32_t* start_pos_dev, const int32_t* block_tables_dev,
                               int32_t block_table_stride, int32_t batch, int32_t max_q_len,
                               int32_t window, void* cuda_stream);
vosti_status vosti_kv_append_planned(vosti_ctx* ctx, const void* plan, const void* k_new,
                                     const void* v_new, const int32_t* block_tables_dev, int32_t batch,
                                     int32_t max_q_len, void* cuda_stream);
vosti_status vosti_paged_attention_planned(vosti_ctx* ctx, const void* plan, const void* q, void* out,
                                           float* lse, const int32_t* block_tables_dev, int32_t batch,
                                           int32_t max_q_len, float softmax_scale, int32_t window,
                                           void* cuda_stream);

/* Split-parallel paged attention for callers that must not allocate.  (The
 * paper has no counterpart: this is a packaging variant of the operation
 * above, not a different computation.)
 *
 * Some callers cannot call cudaMalloc or create a vosti_ctx (which pins host
 * memory and creates streams and events): a serving engine that reserved all
 * device memory for its KV pool at start-up and owns the rest through its own
 * allocator, a latency-critical decode loop that cannot afford the device-wide
 * synchronisation of cudaMalloc / cudaFree, a plug-in that receives device
 * pointers from its host framework but may not create memory of its own.
 * This entry point allocates nothing on host or device and needs no context.
 * Its scratch (status and scheduler words, the call's metadata, the partial
 * (m, z, U) rows) is a 16 MiB file-scope device array that every GPU loading
 * the library holds until the process exits.  It launches the same kernels
 * as vosti_paged_attention, so the output bits are the same.
 *
 *   kv_pool, q, out   device, as for vosti_paged_attention (pool 1024-byte aligned)
 *   q_lens, start_pos, seq_lens, block_tables   host, same meaning as above
 *   cuda_stream       a stream of the CURRENT device (the scratch used is the
 *                     current device's); pool, q and out live on that device
 * Limits (beyond them the call returns VOSTI_ERR_WORKSPACE and launches
 * nothing): batch <= 64, sum of q_lens <= 256, at most 16384 page-table
 * entries in use, at most 1024 (row group, split) items, at most 28000
 * partial rows (n_kv_heads * splits * q_len * G summed over requests).  Every
 * request must satisfy q_len * G <= 32 (decode / speculative queries);
 * longer queries return VOSTI_ERR_UNSUPPORTED_CONFIG.
 * The first call on a device resolves the scratch array's device address and
 * sets kernel attributes; make that first call before any stream capture.
 * The call plans on the host and copies its metadata (only the part in use)
 * from a pageable host buffer inside the library: it returns once that is
 * staged, which waits for earlier work on the stream; the kernels then run
 * asynchronously on the stream.
 * All calls share the one array: what must start at zero is cleared by every
 * call, and two calls that overlap on the GPU (different streams, or the same
 * library used from two threads without ordering) race on it.
 * Failure detection: a kernel that gives up on a bounded wait sets the status
 * word at the start of the array (its output is then undefined).  Calls do
 * not clear that word; vosti_noalloc_poll_status does. */
vosti_status vosti_paged_attention_noalloc(int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                                           int32_t page_size, const void* kv_pool, int64_t num_pages,
                                           const void* q, void* out, const int32_t* q_lens,
                                           const int32_t* start_pos, const int32_t* seq_lens,
                                           const int32_t* block_tables, int32_t block_table_stride,
                                           int32_t batch, float softmax_scale, void* cuda_stream);

/* The status word of the allocation-free entry point, on the current device:
 * waits for the stream, reads the word, clears it, and returns VOSTI_OK or
 * VOSTI_ERR_TIMEOUT (a kernel of some vosti_paged_attention_noalloc call
 * since the last poll gave up on a bounded wait).  Allocates nothing and
 * needs no context.  (No counterpart in the paper.) */
vosti_status vosti_noalloc_poll_status(void* cuda_stream);

/* Failure-detection self-test of that path (no GPU fault involved): one warp
 * waits limit_us microseconds (1..100000) on a barrier nothing completes,
 * gives up, sets the static status word and returns normally; the next
 * vosti_noalloc_poll_status reports VOSTI_ERR_TIMEOUT and clears it. */
vosti_status vosti_noalloc_selftest_bounded_wait(uint32_t limit_us, void* cuda_stream);

/* Waits for the stream and reads the device status word: VOSTI_OK,
 * VOSTI_ERR_TIMEOUT if a kernel gave up on a bounded wait (its output is
 * then undefined), or VOSTI_ERR_OUT_OF_RANGE if a device-planned step met
 * metadata outside the premises.  The word is cleared by the read. */
vosti_status vosti_poll_device_status(vosti_ctx* ctx, void* cuda_stream);

/* Failure-detection self-test (no GPU fault involved): launches one warp that
 * waits, with the bounded wait every kernel of the library uses, on a barrier
 * that nothing completes.  After limit_us microseconds (1..100000) the warp
 * gives up, sets the device status word and returns normally; the next
 * vosti_poll_device_status then reports VOSTI_ERR_TIMEOUT and clears it, and
 * the context stays usable. */
vosti_status vosti_selftest_bounded_wait(vosti_ctx* ctx, uint32_t limit_us, void* cuda_stream);

/* Self-test of the hardware premises of the numerical contract (the paper's
 * trusted tile-operation rules, Sec. "Value-Aware Regional Analysis", and the
 * dot rule of App. A "Backward Regional Dependencies"): computes one small
 * product twice -- with tcgen05.mma and with mma.sync.m16n8k16, both in
 * chunks of 16 ascending from a zero accumulator -- and writes both results.
 *   mode 0 (score form): D[128][64] = A[128][64] . B[64][64]^T
 *   mode 1 (value form): D[128][64] = W[128][64] . V[64][64], W from tensor memory
 *   a, b     device bf16, row-major, 16-byte aligned
 *   d_tc, d_warp   device fp32 [128][64]: the tcgen05 and the warp-MMA result
 * The caller compares bits (the two kernels of the library agree bit for bit
 * only if these do), permutes rows of a to check that an output row depends on
 * its own operand row alone, and zeroes weights to check that a zero weight
 * contributes exactly nothing.  A bounded wait inside reports through the
 * device status word. */
vosti_status vosti_selftest_mma(vosti_ctx* ctx, const void* a, const void* b, int32_t mode, float* d_tc,
                                float* d_warp, void* cuda_stream);

/* Timing of one kernel of the path with CUDA events recorded on the caller's
 * stream around each of its launches.  mode: 0 stops recording; 1 times the
 * split-parallel attention kernel (the decode hot loop, a3-a7), 2 the
 * sequential attention kernel (long queries), 3 the cross-split combine.
 * A non-zero mode starts a fresh record.  vosti_profile_read waits for the
 * recorded events and returns the summed kernel time in milliseconds and the
 * number of launches timed. */
vosti_status vosti_profile_enable(vosti_ctx* ctx, int32_t mode);
vosti_status vosti_profile_read(vosti_ctx* ctx, double* kernel_ms_sum, int64_t* kernels_timed);

/* Kernels launched through this context since creation. */
int64_t vosti_launch_count(const vosti_ctx* ctx);

/* Host time (steady clock, nanoseconds) spent inside vosti_kv_append and the
 * host-planned attention entry points of this context -- validation, planning,
 * metadata upload, launches -- and the number of such calls, since creation
 * or the last call with reset != 0.  Measures the library's own host cost
 * without the binding's.  Either pointer may be NULL. */
vosti_status vosti_host_time(vosti_ctx* ctx, int64_t* nanoseconds, int64_t* calls, int32_t reset);

/* The schedule of the last attention call of this context: split-parallel work
 * items (16-row packed ones included), how many of them are packed items
 * (shared-split packing, VOSTI_FLAG_PACK_SHARED_SPLITS), and tile items: the
 * 256-row items of long queries plus the 128-row packed tiles that large
 * sharing groups are routed to.  Any pointer may be NULL.  Host-side
 * bookkeeping only. */
vosti_status vosti_last_schedule(const vosti_ctx* ctx, int64_t* split_items, int64_t* packed_items,
                                 int64_t* tile_items);

/* Hash of the frozen numerics: the paper's deployment identity W (Sec. "A
 * System-Level Formulation": outputs are compared under one fixed deployment
 * configuration).  It is computed from the list vosti_contract returns -- the
 * library version, key tile, split length, rows per group, the split-parallel
 * row limit, page size, and one id per rule that decides bits (exponent,
 * reference maximum and its step, row-sum order, fold, reciprocal, zero sign,
 * MMA chunk order, log-sum-exp) -- plus, with a context, its head_dim and
 * page_size.  Two builds with equal fingerprints give equal bits on the same
 * GPU model.  ctx may be NULL. */
uint64_t vosti_fingerprint(const vosti_ctx* ctx);

/* The words the fingerprint is made of, in hashing order; returns their
 * number (at most 32) and writes min(number, cap) of them.  Host-only. */
int32_t vosti_contract(uint32_t* words, int32_t cap);

/* Frozen constants: key tile B_N, split length L_S, rows per row group. */
void vosti_constants(int32_t* key_tile, int32_t* split_len, int32_t* rows_per_group);

const char* vosti_status_string(vosti_status status);

#ifdef __cplusplus
}
#endif
#endif /* VOSTI_H_ */
