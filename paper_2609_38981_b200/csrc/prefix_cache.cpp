// Host-side prefix-cache manager (include/vosti_cache.h): exact prefix matching
// over a parent chain of registered pages, reference counts, eviction of
// unreferenced leaves only, and publication of new pages at step boundaries
// (Sec. "Engine Implementation", Sec. "Engine Invariants").  Plain C++, no CUDA.
#include <algorithm>
#include <cstdint>
#include <cstring>
#include <new>
#include <set>
#include <unordered_map>
#include <utility>
#include <vector>

#include "../../include/vosti_cache.h"

namespace {

enum PageState : uint8_t { kFree = 0, kPrivate = 1, kPending = 2, kRegistered = 3 };

struct Page {
  PageState state = kFree;
  int32_t parent = -1;    // registered: physical parent page (-1 at depth 0)
  int32_t depth = -1;     // registered: block index in the prefix
  int32_t refs = 0;       // registered: live requests holding it
  int32_t children = 0;   // registered: registered pages naming it as parent
  uint64_t hash = 0;      // registered: rolling hash of the prefix up to and including this block
  int64_t tick = 0;       // when it last became unreferenced (eviction order: oldest first)
  int64_t owner = -1;     // private / pending: the owning request
};

struct Request {
  std::vector<int32_t> tokens;
  std::vector<int32_t> table;
  int64_t computed = 0;       // positions whose KV values are in the pool
  int64_t cached_blocks = 0;  // leading blocks held as registered pages (a reference each)
  int64_t queued_blocks = 0;  // blocks below this are registered or queued for registration
  uint64_t chain_hash = 0;    // rolling hash of blocks [0, cached_blocks)
};

struct Pending {
  int64_t request;
  int64_t block;
  int32_t page;
};

constexpr uint64_t kHashSeed = 0xcbf29ce484222325ull;

// Rolling hash: extends the hash of a prefix by one block of tokens.
uint64_t extend_hash(uint64_t h, const int32_t* tokens, int n) {
  for (int i = 0; i < n; ++i) {
    h ^= static_cast<uint64_t>(static_cast<uint32_t>(tokens[i])) + 0x9E3779B97F4A7C15ull + (h << 6) + (h >> 2);
    h *= 0x100000001b3ull;
  }
  return h;
}

}  // namespace

struct vosti_cache {
  int64_t num_pages = 0;
  int32_t P = 0;
  uint64_t hash_mask = ~0ull;  // tests narrow it to force collisions
  std::vector<Page> pages;
  std::vector<int32_t> page_tokens;  // [num_pages][P], valid for registered pages
  std::vector<int32_t> free_list;
  std::unordered_multimap<uint64_t, int32_t> index;  // hash -> registered pages
  std::set<std::pair<int64_t, int32_t>> leaves;      // (tick, page): registered, unreferenced, childless
  std::unordered_map<int64_t, Request> requests;
  std::vector<Pending> pending;
  int64_t clock = 0;
  int64_t retained = 0;  // registered pages with refs == 0
  int64_t hit_pages = 0, evicted_pages = 0;

  // Rolling hash of a prefix extended by one block (narrowed by the test mask, so that
  // different prefixes can be made to collide on purpose).
  uint64_t ext(uint64_t h, const int32_t* block) const { return extend_hash(h, block, P) & hash_mask; }

  void unref(int32_t pg) {
    Page& p = pages[pg];
    if (--p.refs == 0) {
      p.tick = ++clock;
      ++retained;
      if (p.children == 0) leaves.insert({p.tick, pg});
    }
  }
  void ref(int32_t pg) {
    Page& p = pages[pg];
    if (p.refs++ == 0) {
      --retained;
      if (p.children == 0) leaves.erase({p.tick, pg});
    }
  }
  // Evicts the oldest unreferenced leaf.  Its parent may become a leaf in turn.
  bool evict_one() {
    if (leaves.empty()) return false;
    const int32_t pg = leaves.begin()->second;
    leaves.erase(leaves.begin());
    Page& p = pages[pg];
    auto range = index.equal_range(p.hash);
    for (auto it = range.first; it != range.second; ++it)
      if (it->second == pg) {
        index.erase(it);
        break;
      }
    if (p.parent >= 0) {
      Page& par = pages[p.parent];
      if (--par.children == 0 && par.refs == 0) leaves.insert({par.tick, p.parent});
    }
    p = Page{};
    --retained;
    ++evicted_pages;
    free_list.push_back(pg);
    return true;
  }
  // One private page for `owner`; the caller has checked that enough pages can be had.
  int32_t take_page(int64_t owner) {
    if (free_list.empty() && !evict_one()) return -1;
    const int32_t pg = free_list.back();
    free_list.pop_back();
    Page& p = pages[pg];
    p = Page{};
    p.state = kPrivate;
    p.owner = owner;
    return pg;
  }
  void release_private(int32_t pg) {
    pages[pg] = Page{};
    free_list.push_back(pg);
  }
  // A registered page holding exactly this block at this depth under this parent, or -1.
  int32_t find(uint64_t h, const int32_t* block, int64_t depth, int32_t parent) const {
    auto range = index.equal_range(h);
    for (auto it = range.first; it != range.second; ++it) {
      const Page& p = pages[it->second];
      if (p.state == kRegistered && p.depth == depth && p.parent == parent && p.hash == h &&
          std::memcmp(&page_tokens[static_cast<size_t>(it->second) * P], block, sizeof(int32_t) * P) == 0)
        return it->second;
    }
    return -1;
  }
};

extern "C" {

vosti_status vosti_cache_create(vosti_cache** out, int64_t num_pages, int32_t page_size) {
  if (!out) return VOSTI_ERR_INVALID_ARG;
  *out = nullptr;
  if (num_pages <= 0 || num_pages > INT32_MAX || page_size <= 0) return VOSTI_ERR_INVALID_ARG;
  vosti_cache* c = new (std::nothrow) vosti_cache();
  if (!c) return VOSTI_ERR_INVALID_ARG;
  c->num_pages = num_pages;
  c->P = page_size;
  c->pages.resize(static_cast<size_t>(num_pages));
  c->page_tokens.resize(static_cast<size_t>(num_pages) * page_size);
  c->free_list.resize(static_cast<size_t>(num_pages));
  for (int64_t i = 0; i < num_pages; ++i) c->free_list[i] = static_cast<int32_t>(num_pages - 1 - i);  // page 0 first
  *out = c;
  return VOSTI_OK;
}

vosti_status vosti_cache_destroy(vosti_cache* cache) {
  delete cache;
  return VOSTI_OK;
}

vosti_status vosti_cache_debug_set_hash_mask(vosti_cache* cache, uint64_t mask) {
  if (!cache || !cache->index.empty()) return VOSTI_ERR_INVALID_ARG;
  cache->hash_mask = mask;
  return VOSTI_OK;
}

vosti_status vosti_cache_admit(vosti_cache* c, int64_t request_id, const int32_t* tokens, int64_t n_tokens,
                               int64_t* n_cached) {
  if (!c || !tokens || n_tokens < 1 || !n_cached || c->requests.count(request_id)) return VOSTI_ERR_INVALID_ARG;
  const int P = c->P;
  const int64_t n_pages = (n_tokens + P - 1) / P;
  const int64_t max_hits = (n_tokens - 1) / P;  // at least the last token is left to compute
  // 1. resolve hits against what earlier steps published
  std::vector<int32_t> table;
  table.reserve(static_cast<size_t>(n_pages));
  uint64_t h = kHashSeed;
  int32_t prev = -1;
  for (int64_t b = 0; b < max_hits; ++b) {
    const uint64_t hb = c->ext(h, tokens + b * P);
    const int32_t pg = c->find(hb, tokens + b * P, b, prev);
    if (pg < 0) break;
    table.push_back(pg);
    prev = pg;
    h = hb;
  }
  const int64_t hits = static_cast<int64_t>(table.size());
  // 2. can the rest be allocated?  Every unreferenced registered page is evictable, leaf by
  //    leaf (a request holds all the ancestors of a page it holds), except the hits themselves.
  int64_t hits_retained = 0;
  for (int32_t pg : table) hits_retained += c->pages[pg].refs == 0 ? 1 : 0;
  const int64_t need = n_pages - hits;
  if (need > static_cast<int64_t>(c->free_list.size()) + c->retained - hits_retained) return VOSTI_ERR_OUT_OF_RANGE;
  // 3. commit
  for (int32_t pg : table) c->ref(pg);
  for (int64_t b = hits; b < n_pages; ++b) table.push_back(c->take_page(request_id));
  Request& r = c->requests[request_id];
  r.tokens.assign(tokens, tokens + n_tokens);
  r.table = std::move(table);
  r.computed = hits * P;
  r.cached_blocks = r.queued_blocks = hits;
  r.chain_hash = h;
  c->hit_pages += hits;
  *n_cached = hits * P;
  return VOSTI_OK;
}

vosti_status vosti_cache_append(vosti_cache* c, int64_t request_id, const int32_t* tokens, int64_t n) {
  if (!c || n < 0 || (n > 0 && !tokens)) return VOSTI_ERR_INVALID_ARG;
  auto it = c->requests.find(request_id);
  if (it == c->requests.end()) return VOSTI_ERR_INVALID_ARG;
  Request& r = it->second;
  const int P = c->P;
  const int64_t total = static_cast<int64_t>(r.tokens.size()) + n;
  const int64_t need = (total + P - 1) / P - static_cast<int64_t>(r.table.size());
  if (need > static_cast<int64_t>(c->free_list.size()) + c->retained) return VOSTI_ERR_OUT_OF_RANGE;
  r.tokens.insert(r.tokens.end(), tokens, tokens + n);
  for (int64_t i = 0; i < need; ++i) r.table.push_back(c->take_page(request_id));
  return VOSTI_OK;
}

vosti_status vosti_cache_computed(vosti_cache* c, int64_t request_id, int64_t upto) {
  if (!c) return VOSTI_ERR_INVALID_ARG;
  auto it = c->requests.find(request_id);
  if (it == c->requests.end()) return VOSTI_ERR_INVALID_ARG;
  Request& r = it->second;
  if (upto < r.computed || upto > static_cast<int64_t>(r.tokens.size())) return VOSTI_ERR_OUT_OF_RANGE;
  r.computed = upto;
  const int64_t complete = upto / c->P;
  for (int64_t b = r.queued_blocks; b < complete; ++b) {
    const int32_t pg = r.table[static_cast<size_t>(b)];
    c->pages[pg].state = kPending;
    c->pending.push_back({request_id, b, pg});
  }
  r.queued_blocks = std::max(r.queued_blocks, complete);
  return VOSTI_OK;
}

vosti_status vosti_cache_step_boundary(vosti_cache* c) {
  if (!c) return VOSTI_ERR_INVALID_ARG;
  const int P = c->P;
  for (const Pending& pe : c->pending) {
    auto it = c->requests.find(pe.request);
    if (it == c->requests.end()) continue;  // finished meanwhile: its pages were released
    Request& r = it->second;
    Page& p = c->pages[pe.page];
    if (pe.block >= static_cast<int64_t>(r.table.size()) || r.table[static_cast<size_t>(pe.block)] != pe.page ||
        p.state != kPending || p.owner != pe.request)
      continue;
    p.state = kPrivate;
    // Published pages form a chain of physical parents: a block can only follow a registered one.
    if (pe.block != r.cached_blocks) continue;
    const int32_t parent = pe.block == 0 ? -1 : r.table[static_cast<size_t>(pe.block - 1)];
    const int32_t* block = r.tokens.data() + pe.block * P;
    const uint64_t h = c->ext(r.chain_hash, block);
    if (c->find(h, block, pe.block, parent) >= 0) continue;  // this prefix is published already: stay private
    std::memcpy(&c->page_tokens[static_cast<size_t>(pe.page) * P], block, sizeof(int32_t) * P);
    p.state = kRegistered;
    p.parent = parent;
    p.depth = static_cast<int32_t>(pe.block);
    p.refs = 1;  // the producing request
    p.children = 0;
    p.hash = h;
    p.owner = -1;
    if (parent >= 0) ++c->pages[parent].children;  // the parent is held by this request: not a leaf candidate
    c->index.insert({h, pe.page});
    r.cached_blocks = pe.block + 1;
    r.chain_hash = h;
  }
  c->pending.clear();
  return VOSTI_OK;
}

vosti_status vosti_cache_finish(vosti_cache* c, int64_t request_id) {
  if (!c) return VOSTI_ERR_INVALID_ARG;
  auto it = c->requests.find(request_id);
  if (it == c->requests.end()) return VOSTI_ERR_INVALID_ARG;
  Request& r = it->second;
  // children before parents, so that a chain left without references lists its deepest page first
  for (int64_t b = static_cast<int64_t>(r.table.size()) - 1; b >= 0; --b) {
    const int32_t pg = r.table[static_cast<size_t>(b)];
    if (b < r.cached_blocks) c->unref(pg);
    else c->release_private(pg);
  }
  c->requests.erase(it);
  return VOSTI_OK;
}

vosti_status vosti_cache_block_table(const vosti_cache* c, int64_t request_id, int32_t* pages, int64_t cap,
                                     int64_t* n_pages) {
  if (!c || cap < 0 || (cap > 0 && !pages)) return VOSTI_ERR_INVALID_ARG;
  auto it = c->requests.find(request_id);
  if (it == c->requests.end()) return VOSTI_ERR_INVALID_ARG;
  const std::vector<int32_t>& t = it->second.table;
  const int64_t n = static_cast<int64_t>(t.size());
  for (int64_t i = 0; i < std::min(n, cap); ++i) pages[i] = t[static_cast<size_t>(i)];
  if (n_pages) *n_pages = n;
  return VOSTI_OK;
}

vosti_status vosti_cache_stats(const vosti_cache* c, int64_t* free_pages, int64_t* retained_pages,
                               int64_t* live_pages, int64_t* hit_pages, int64_t* evicted_pages) {
  if (!c) return VOSTI_ERR_INVALID_ARG;
  const int64_t nfree = static_cast<int64_t>(c->free_list.size());
  if (free_pages) *free_pages = nfree;
  if (retained_pages) *retained_pages = c->retained;
  if (live_pages) *live_pages = c->num_pages - nfree - c->retained;
  if (hit_pages) *hit_pages = c->hit_pages;
  if (evicted_pages) *evicted_pages = c->evicted_pages;
  return VOSTI_OK;
}

vosti_status vosti_cache_page_info(const vosti_cache* c, int32_t page, int32_t* depth, int32_t* parent,
                                   int32_t* refs, int32_t* children) {
  if (!c || page < 0 || page >= c->num_pages) return VOSTI_ERR_INVALID_ARG;
  const Page& p = c->pages[page];
  if (p.state != kRegistered) return VOSTI_ERR_OUT_OF_RANGE;
  if (depth) *depth = p.depth;
  if (parent) *parent = p.parent;
  if (refs) *refs = p.refs;
  if (children) *children = p.children;
  return VOSTI_OK;
}

vosti_status vosti_cache_check(const vosti_cache* c, const char** what) {
  if (!c) return VOSTI_ERR_INVALID_ARG;
  auto fail = [&](const char* msg) {
    if (what) *what = msg;
    return VOSTI_ERR_INVALID_ARG;
  };
  if (what) *what = "";
  const int P = c->P;
  const size_t N = static_cast<size_t>(c->num_pages);
  // free list: free pages, each once
  std::vector<int32_t> seen(N, 0);
  for (int32_t pg : c->free_list) {
    if (pg < 0 || pg >= c->num_pages) return fail("free list entry out of range");
    if (c->pages[pg].state != kFree) return fail("page on the free list is not free");
    if (seen[pg]++) return fail("page twice on the free list");
  }
  size_t n_free = 0, n_retained = 0;
  for (size_t i = 0; i < N; ++i) n_free += c->pages[i].state == kFree ? 1 : 0;
  if (n_free != c->free_list.size()) return fail("a free page is missing from the free list");
  // requests: layout, provenance of the cached prefix, ownership of the private suffix
  std::vector<int32_t> refs(N, 0), uses(N, 0);
  for (const auto& kv : c->requests) {
    const Request& r = kv.second;
    const int64_t n = static_cast<int64_t>(r.tokens.size());
    if (static_cast<int64_t>(r.table.size()) != (n + P - 1) / P) return fail("block table length does not match the history");
    if (r.computed < 0 || r.computed > n) return fail("initialised length outside the history");
    if (r.cached_blocks > r.queued_blocks || r.queued_blocks > r.computed / P)
      return fail("registered blocks beyond the initialised prefix");
    uint64_t h = kHashSeed;
    for (int64_t b = 0; b < static_cast<int64_t>(r.table.size()); ++b) {
      const int32_t pg = r.table[static_cast<size_t>(b)];
      if (pg < 0 || pg >= c->num_pages) return fail("block table entry out of range");
      const Page& p = c->pages[pg];
      ++uses[pg];
      if (b < r.cached_blocks) {
        h = c->ext(h, r.tokens.data() + b * P);
        if (p.state != kRegistered) return fail("cached block is not a registered page");
        if (p.depth != b) return fail("registered page at the wrong depth of a request");
        if (p.parent != (b ? r.table[static_cast<size_t>(b - 1)] : -1)) return fail("registered page under the wrong parent");
        if (p.hash != h) return fail("registered page with the wrong prefix hash");
        if (std::memcmp(&c->page_tokens[static_cast<size_t>(pg) * P], r.tokens.data() + b * P, sizeof(int32_t) * P))
          return fail("registered page holds other tokens than the request's block");
        ++refs[pg];
      } else {
        if (p.state != kPrivate && p.state != kPending) return fail("suffix page is neither private nor pending");
        if (p.owner != kv.first) return fail("suffix page owned by another request");
      }
    }
    if (r.chain_hash != h) return fail("request's chain hash is stale");
  }
  // pages: counts, parent chains, write isolation
  std::vector<int32_t> children(N, 0);
  for (size_t i = 0; i < N; ++i) {
    const Page& p = c->pages[i];
    if (p.state == kPrivate || p.state == kPending) {
      if (uses[i] != 1) return fail("private page not in exactly one block table");
      if (!c->requests.count(p.owner)) return fail("private page of a request that is gone");
    } else if (p.state == kRegistered) {
      if (p.refs != refs[i]) return fail("reference count differs from the live requests holding the page");
      if (p.refs == 0) ++n_retained;
      if (p.depth < 0) return fail("registered page without depth");
      if ((p.depth == 0) != (p.parent < 0)) return fail("parent link inconsistent with depth");
      if (p.parent >= 0) {
        const Page& par = c->pages[p.parent];
        if (par.state != kRegistered) return fail("parent of a registered page is not registered");
        if (par.depth != p.depth - 1) return fail("parent at the wrong depth");
        if (par.refs < p.refs) return fail("a page has more holders than its parent");
        ++children[p.parent];
      }
      size_t in_index = 0;
      auto range = c->index.equal_range(p.hash);
      for (auto it = range.first; it != range.second; ++it) in_index += it->second == static_cast<int32_t>(i) ? 1 : 0;
      if (in_index != 1) return fail("registered page not exactly once in the hash index");
    } else if (uses[i] != 0) {
      return fail("free page in a block table");
    }
  }
  size_t n_leaves = 0;
  for (size_t i = 0; i < N; ++i) {
    const Page& p = c->pages[i];
    if (p.state != kRegistered) continue;
    if (p.children != children[i]) return fail("child count differs from the registered children");
    // the prefix hash of a registered page follows from its parent's and its own tokens
    const uint64_t hp = p.parent >= 0 ? c->pages[p.parent].hash : kHashSeed;
    if (c->ext(hp, &c->page_tokens[i * P]) != p.hash) return fail("stored hash does not follow from the parent chain");
    if (p.refs == 0 && p.children == 0) {
      ++n_leaves;
      if (!c->leaves.count({p.tick, static_cast<int32_t>(i)})) return fail("unreferenced leaf missing from the eviction set");
    }
  }
  if (n_leaves != c->leaves.size()) return fail("eviction set holds a page that is not an unreferenced leaf");
  if (static_cast<int64_t>(n_retained) != c->retained) return fail("retained count is stale");
  if (c->index.size() != N - n_free - [&] {
        size_t priv = 0;
        for (size_t i = 0; i < N; ++i) priv += (c->pages[i].state == kPrivate || c->pages[i].state == kPending) ? 1 : 0;
        return priv;
      }())
    return fail("hash index size differs from the number of registered pages");
  return VOSTI_OK;
}

}  // extern "C"
