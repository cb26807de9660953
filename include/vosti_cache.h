/* vosti_cache.h -- host-side prefix-cache manager for the paged KV pool.
 *
 * It hands out the block tables that vosti_kv_append / vosti_paged_attention
 * consume, following Sec. "Engine Implementation":
 *   * "Exact prefix matching": a cached page is reusable only for the token
 *     prefix that produced it.  A rolling hash finds candidate pages; a
 *     candidate is accepted only if its exact token block, its depth in the
 *     prefix and its physical parent page all agree, so a hash collision can
 *     never justify reuse.  Under memory pressure only unreferenced leaves of
 *     the parent chain are evicted, so a parent's page id cannot be recycled
 *     while a retained child still names it.
 *   * "Separate cache reuse from generation": pages whose KV values a step
 *     produces become reusable only at the next step boundary
 *     (vosti_cache_step_boundary); hits are resolved against what earlier
 *     steps published.  Registered pages are immutable; a request writes only
 *     to its private suffix pages.
 * and maintaining the bookkeeping half of Sec. "Engine Invariants" (layout
 * consistency, sharing and write isolation); the KV-value half -- every
 * initialised live or retained entry equals what a cold run on its causal
 * prefix computes -- follows when the caller writes position p of a request
 * only after vosti_cache_admit / _append placed it in a private page, and
 * reports it with vosti_cache_computed afterwards.
 *
 * Everything here is host memory and plain integers: no CUDA call, no device
 * pointer.  Not thread-safe: one scheduler thread drives one cache.
 * Only whole pages are shared; the tail page of a request is always private.
 * All functions return VOSTI_OK or an error and leave the cache unchanged on
 * error.
 */
#ifndef VOSTI_CACHE_H_
#define VOSTI_CACHE_H_

#include <stdint.h>

#include "vosti.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct vosti_cache vosti_cache;

/* A manager for pages 0 .. num_pages-1 of `page_size` tokens each. */
vosti_status vosti_cache_create(vosti_cache** out, int64_t num_pages, int32_t page_size);
vosti_status vosti_cache_destroy(vosti_cache* cache);

/* Admit a request with its prompt `tokens[0 .. n_tokens)` (host, n_tokens >= 1)
 * under a caller-chosen id not in use.  Resolves prefix hits page by page from
 * the front (stopping at the first miss, and always leaving at least the last
 * token to compute), takes a reference on every hit page, and allocates private
 * pages for the rest of the prompt, evicting unreferenced leaves if the free
 * list runs dry.  *n_cached receives the number of leading tokens whose KV
 * values are already in the pool: the caller prefills positions
 * n_cached .. n_tokens-1.
 * Errors: INVALID_ARG (bad pointers, id in use), OUT_OF_RANGE (not enough free
 * or evictable pages; nothing was changed). */
vosti_status vosti_cache_admit(vosti_cache* cache, int64_t request_id, const int32_t* tokens,
                               int64_t n_tokens, int64_t* n_cached);

/* Append `n` generated tokens to a live request's history (decode), allocating
 * a private page whenever the history crosses a page boundary.
 * Errors: INVALID_ARG (unknown id), OUT_OF_RANGE (no page to be had). */
vosti_status vosti_cache_append(vosti_cache* cache, int64_t request_id, const int32_t* tokens, int64_t n);

/* Report that the KV values of positions < upto of the request are now in the
 * pool (upto may only grow, and not beyond the history).  Private pages that
 * are thereby complete are queued for registration; they become reusable at
 * the next step boundary. */
vosti_status vosti_cache_computed(vosti_cache* cache, int64_t request_id, int64_t upto);

/* End of an engine step: publishes the pages queued since the last boundary
 * (exact tokens, depth, physical parent, rolling hash).  A page whose prefix is
 * already published under another physical page stays private to its request. */
vosti_status vosti_cache_step_boundary(vosti_cache* cache);

/* The request is over: its references are dropped.  Registered pages stay
 * resident (retained, reusable, evictable once they are unreferenced leaves);
 * private pages go back to the free list. */
vosti_status vosti_cache_finish(vosti_cache* cache, int64_t request_id);

/* The request's block table: page ids in logical order for its whole history.
 * Writes min(*n_pages, cap) entries. */
vosti_status vosti_cache_block_table(const vosti_cache* cache, int64_t request_id, int32_t* pages,
                                     int64_t cap, int64_t* n_pages);

/* Counters; any pointer may be NULL.  free + retained + live == num_pages;
 * `retained` = registered pages with no live reference, `live` = pages held by
 * some live request (shared ones counted once). */
vosti_status vosti_cache_stats(const vosti_cache* cache, int64_t* free_pages, int64_t* retained_pages,
                               int64_t* live_pages, int64_t* hit_pages, int64_t* evicted_pages);

/* Full consistency check of the bookkeeping (layout, reference and child
 * counts, parent chains of registered pages, the hash index, disjointness of
 * private pages and the free list).  VOSTI_OK, or INVALID_ARG with *what (if
 * not NULL) set to a static string naming the violated condition. */
vosti_status vosti_cache_check(const vosti_cache* cache, const char** what);

/* Provenance of a registered page (for tests and tools): its depth, physical
 * parent (-1 at depth 0), live references and registered children.  Returns
 * OUT_OF_RANGE if the page is not registered. */
vosti_status vosti_cache_page_info(const vosti_cache* cache, int32_t page, int32_t* depth,
                                   int32_t* parent, int32_t* refs, int32_t* children);

/* Test hook: AND every prefix hash with `mask` (0 makes all prefixes collide), so
 * that tests can show that a collision never leads to reuse.  Only on an empty
 * cache (nothing registered yet); INVALID_ARG otherwise. */
vosti_status vosti_cache_debug_set_hash_mask(vosti_cache* cache, uint64_t mask);

#ifdef __cplusplus
}
#endif
#endif /* VOSTI_CACHE_H_ */
