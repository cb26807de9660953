"""Prefix-cache manager (include/vosti_cache.h), host only.

Pins: the life cycle drawn in the paper's KV-cache figure (share, retain, evict
a leaf, reuse + recompute) with its reference counts; exact matching under
forced hash collisions; publication only at step boundaries; eviction of
unreferenced leaves only; and a randomised run that checks, after every
operation, the manager's own consistency check plus the KV-value invariant of
Sec. "Engine Invariants" against a shadow pool in which the value stored for
position p is a digest of the causal prefix tokens[0..p]."""
import os
import re
import ctypes
import hashlib

import numpy as np
import pytest

from paper_2609_38981_b200 import build as vbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def pc():
    vbuild.build()
    from paper_2609_38981_b200 import cache
    return cache


def test_library_exports_every_declared_symbol(pc):
    text = open(os.path.join(ROOT, "include", "vosti_cache.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = sorted(set(re.findall(r"\b(vosti_cache_[a-z_]+)\s*\(", text)))
    assert len(names) == 12
    from paper_2609_38981_b200 import binding
    lib = ctypes.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(pc.EXPORTS) == names


def prefill(c, rid, n):
    """The caller's side of a step: KV for all n positions written."""
    c.computed(rid, n)


A, B, C_ = 1, 2, 3
a, b, c_, d, e, f, x, y = range(100, 108)


def test_figure_share_retain_evict_reuse(pc):
    """Pages of two tokens.  A = [a b c d x], B = [a b e f y] (the fifth token keeps the
    last full page reusable: only whole pages strictly before the last token are hits)."""
    c = pc.PrefixCache(num_pages=5, page_size=2)
    # A runs alone first: cold
    assert c.admit(A, [a, b, c_, d, x]) == 0
    ta = c.block_table(A)
    assert len(ta) == 3 and len(set(ta)) == 3
    prefill(c, A, 5)
    assert c.page_info(ta[0]) is None          # not published before the step boundary
    c.step_boundary()
    assert c.page_info(ta[0]) == (0, -1, 1, 1) and c.page_info(ta[1]) == (1, ta[0], 1, 0)
    assert c.page_info(ta[2]) is None          # the partial tail page stays private
    # 1 Share: B arrives, reuses [a b], computes its own branch
    assert c.admit(B, [a, b, e, f, y]) == 2
    tb = c.block_table(B)
    assert tb[0] == ta[0] and tb[1] != ta[1]
    assert c.page_info(ta[0]) == (0, -1, 2, 1)  # refs = 2
    prefill(c, B, 5)
    c.step_boundary()
    assert c.page_info(ta[0]) == (0, -1, 2, 2) and c.page_info(tb[1]) == (1, ta[0], 1, 0)
    assert c.check() == ""
    # 2 Retain: both finish; the three registered pages stay with refs = 0
    c.finish(A)
    c.finish(B)
    assert [c.page_info(p)[2] for p in (ta[0], ta[1], tb[1])] == [0, 0, 0]
    assert c.stats()["retained"] == 3 and c.stats()["free"] == 2 and c.check() == ""
    # 3 Evict: memory pressure takes a leaf, never the parent of a retained child.
    #   A five-page request needs 5 pages: 2 free + 3 evictions would empty the cache, so ask for 3.
    assert c.admit(9, [1, 2, 3, 4, 5, 6]) == 0       # 3 pages: 2 free + 1 eviction
    s = c.stats()
    assert s["evicted_pages"] == 1 and s["retained"] == 2
    assert c.page_info(ta[1]) is None                # A's leaf [c d] went first (oldest unreferenced leaf)
    assert c.page_info(ta[0]) == (0, -1, 0, 1)       # the parent survives with one retained child
    assert c.page_info(tb[1]) == (1, ta[0], 0, 0)
    c.finish(9)
    assert c.check() == ""
    # 4 Reuse + recompute: C = [a b c d z] hits [a b] only and recomputes [c d] in a fresh page
    assert c.admit(C_, [a, b, c_, d, 77]) == 2
    tc = c.block_table(C_)
    assert tc[0] == ta[0] and c.page_info(ta[0])[2] == 1
    prefill(c, C_, 5)
    c.step_boundary()
    assert c.page_info(tc[1]) == (1, ta[0], 1, 0) and c.page_info(tb[1]) == (1, ta[0], 0, 0)
    assert c.check() == ""
    c.close()


def test_same_step_pages_are_not_reusable(pc):
    c = pc.PrefixCache(16, 2)
    c.admit(1, [1, 2, 3, 4, 5])
    prefill(c, 1, 5)
    assert c.admit(2, [1, 2, 3, 4, 5]) == 0       # same step: nothing published yet
    c.step_boundary()
    assert c.admit(3, [1, 2, 3, 4, 5]) == 4       # next step: two whole pages, last token left to compute
    assert c.admit(4, [1, 2, 3, 4]) == 2          # a prompt ending on a page edge keeps its last page to compute
    # request 2 computed the same prefix in private pages: publishing finds it already there
    prefill(c, 2, 5)
    c.step_boundary()
    t1, t2 = c.block_table(1), c.block_table(2)
    assert c.page_info(t2[0]) is None and c.page_info(t1[0])[2] == 3
    assert c.check() == ""


def test_hash_collisions_never_justify_reuse(pc):
    c = pc.PrefixCache(64, 2)
    c.debug_set_hash_mask(0)                        # every prefix hashes to 0
    c.admit(1, [1, 2, 3, 4, 9])
    prefill(c, 1, 5)
    c.step_boundary()
    assert c.admit(2, [5, 6, 3, 4, 9]) == 0         # other first block
    assert c.admit(3, [1, 2, 7, 8, 9]) == 2         # same first block, other second
    assert c.admit(4, [3, 4, 1, 2, 9]) == 0         # the same blocks at other depths
    assert c.admit(5, [1, 2, 3, 4, 9]) == 4
    for r in (2, 3, 4, 5):
        prefill(c, r, 5)
    c.step_boundary()
    # [3 4] exists under two different parents now ([1 2] and [5 6]); a request is matched
    # through the parent it actually has
    assert c.admit(6, [5, 6, 3, 4, 1]) == 4
    assert c.block_table(6)[:2] == c.block_table(2)[:2]
    assert c.check() == ""


def test_only_unreferenced_leaves_are_evicted_and_failure_changes_nothing(pc):
    c = pc.PrefixCache(8, 2)
    c.admit(1, list(range(10, 19)))                 # 9 tokens: 5 pages
    prefill(c, 1, 9)
    c.step_boundary()
    chain = c.block_table(1)[:4]
    c.finish(1)
    assert c.stats() == {"free": 4, "retained": 4, "live": 0, "hit_pages": 0, "evicted_pages": 0}
    # a live request holds the first two pages of the chain
    assert c.admit(2, list(range(10, 14)) + [1]) == 4
    before = (c.stats(), [c.page_info(p) for p in chain])
    # 3 pages held by request 2, 2 retained (evictable), 3 free -> at most 5 more pages
    with pytest.raises(Exception):
        c.admit(3, list(range(50, 62)))             # 6 pages: refused
    assert (c.stats(), [c.page_info(p) for p in chain]) == before and c.check() == ""
    assert c.admit(3, list(range(50, 60))) == 0     # 5 pages: evicts the two unreferenced pages, deepest first
    assert c.page_info(chain[3]) is None and c.page_info(chain[2]) is None
    assert c.page_info(chain[1]) == (1, chain[0], 1, 0) and c.page_info(chain[0]) == (0, -1, 1, 1)
    assert c.stats()["free"] == 0 and c.check() == ""
    with pytest.raises(Exception):
        c.append(2, [5, 6])                         # would need a page: none to be had
    assert c.check() == ""


def digest(tokens) -> bytes:
    return hashlib.blake2b(np.asarray(tokens, dtype=np.int32).tobytes(), digest_size=8).digest()


@pytest.mark.parametrize("seed,mask", [(0, ~0 & (2 ** 64 - 1)), (1, ~0 & (2 ** 64 - 1)), (2, 0x3)])
def test_randomised_lifecycle_keeps_the_kv_value_invariant(pc, seed, mask):
    """Random admissions (from a small family of prompts that share prefixes), chunked
    prefill, decode, step boundaries and completions in a pool small enough to evict all the
    time.  The shadow pool models E.kv: a slot holds the digest of the causal prefix whose KV
    value was written there.  After every operation: the manager's check passes; every
    initialised position of every live request reads its own prefix digest through its block
    table (cached positions were never written by this request: they must have been produced
    by an identical prefix); and no two live requests can write the same slot."""
    rng = np.random.default_rng(seed)
    P, N = 4, 28
    c = pc.PrefixCache(N, P)
    c.debug_set_hash_mask(mask)
    shadow = {}                                      # (page, slot) -> digest
    stems = [rng.integers(0, 50, size=40).tolist() for _ in range(3)]
    live = {}                                        # id -> dict(tokens, done)
    next_id = 0

    def verify():
        assert c.check() == ""
        writable = {}
        for rid, r in live.items():
            tb = c.block_table(rid)
            assert len(tb) == -(-len(r["tokens"]) // P)
            for p in range(r["done"]):
                assert shadow.get((tb[p // P], p % P)) == digest(r["tokens"][:p + 1]), (rid, p)
            for p in range(r["done"], len(r["tokens"])):
                key = (tb[p // P], p % P)
                assert key not in writable, "two requests may write the same slot"
                writable[key] = rid
        s = c.stats()
        assert s["free"] + s["retained"] + s["live"] == N

    for _ in range(2000):
        op = rng.integers(0, 6)
        if op == 0 and len(live) < 5:                # admit
            stem = stems[rng.integers(0, 3)]
            n = int(rng.integers(1, 36))
            toks = stem[:n]
            if rng.random() < 0.5 and n > 2:         # branch off somewhere
                k = int(rng.integers(1, n))
                toks = toks[:k] + rng.integers(50, 60, size=n - k).tolist()
            try:
                cached = c.admit(next_id, toks)
            except Exception:
                verify()
                continue
            assert cached % P == 0 and cached < len(toks)
            live[next_id] = dict(tokens=list(toks), done=cached)
            next_id += 1
        elif op == 1 and live:                       # a prefill chunk (or the decode token's KV): write, then report
            rid = list(live)[rng.integers(0, len(live))]
            r = live[rid]
            if r["done"] == len(r["tokens"]):
                continue                             # nothing to compute: decode appends come from op 4
            upto = min(len(r["tokens"]), r["done"] + int(rng.integers(1, 9)))
            tb = c.block_table(rid)
            for p in range(r["done"], upto):
                shadow[(tb[p // P], p % P)] = digest(r["tokens"][:p + 1])
            c.computed(rid, upto)
            r["done"] = upto
        elif op == 2:
            c.step_boundary()
        elif op == 3 and live and rng.random() < 0.5:  # finish
            rid = list(live)[rng.integers(0, len(live))]
            c.finish(rid)
            del live[rid]
        elif op == 4 and live:                       # decode with a known token
            rid = list(live)[rng.integers(0, len(live))]
            r = live[rid]
            if r["done"] == len(r["tokens"]):
                t = int(rng.integers(0, 60))
                try:
                    c.append(rid, [t])
                except Exception:
                    verify()
                    continue
                r["tokens"].append(t)
        verify()
    st = c.stats()
    assert st["hit_pages"] > 0 and st["evicted_pages"] > 0   # the run really shared and really evicted
    c.close()
