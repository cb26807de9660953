"""Host-side checks that need no GPU: the C-ABI library loads, exports every
symbol the header declares, and its host-only entry points (planning,
workspace sizing, constants, status strings) behave as documented."""
import os
import re
import ctypes

import numpy as np
import pytest

from paper_2609_38981_b200 import build as vbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def vb():
    vbuild.build()
    from paper_2609_38981_b200 import binding
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "vosti.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(vosti_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(vb):
    names = declared_functions()
    assert len(names) >= 16
    lib = ctypes.CDLL(vb.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in vosti.h but not exported"
    assert sorted(vb.EXPORTS) == names


def test_the_attention_library_does_not_contain_the_linear_layer(vb):
    """Multi-GPU runs carry only the attention library: it must stand on its own."""
    lib = ctypes.CDLL(vb.LIB_PATH)
    assert not hasattr(lib, "vosti_linear") and not hasattr(lib, "vosti_rmsnorm")
    assert not any("linear" in name or "rmsnorm" in name for name in vb.EXPORTS)


def test_linear_header_symbols_and_tile_shape(vb):
    """The linear layer's tile shape is a host-side function of (N, K) alone."""
    from paper_2609_38981_b200 import linear as vl
    text = open(os.path.join(ROOT, "include", "vosti_linear.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = sorted(set(re.findall(r"\b(vosti_[a-z_]+)\s*\(", text)))
    lib = ctypes.CDLL(vl.LIB_PATH)          # the linear layer is a library of its own
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(vl.EXPORTS) == names
    assert vl.vosti_linear_tile_shape(4096, 4096) == (128, 256, 64)
    assert vl.vosti_linear_tile_shape(28672, 4096) == (128, 256, 64)
    assert vl.vosti_linear_tile_shape(128, 64) == (128, 128, 64)
    assert vl.vosti_linear_segments(4096, 4096) == 4 and vl.vosti_linear_segments(6144, 4096) == 4
    assert vl.vosti_linear_workspace_bytes(3, 128, 64) == 3 * 128 * 4 and vl.vosti_linear_workspace_bytes(3, 100, 64) == 0
    for N, K in ((0, 64), (100, 64), (128, 32), (128, 0)):
        with pytest.raises(vb.VostiError) as e:
            vl.vosti_linear_tile_shape(N, K)
        assert e.value.status == vb.VOSTI_ERR_UNSUPPORTED_CONFIG


def test_constants_and_fingerprint(vb):
    c = vb.vosti_constants()
    assert c == {"key_tile": 64, "split_len": 512, "rows_per_group": 16}
    assert vb.vosti_fingerprint() == vb.vosti_fingerprint() != 0
    assert vb.vosti_status_string(0) == "ok" and "range" in vb.vosti_status_string(3)


def cfg(vb, hq=32, hkv=8, d=128, P=16, pages=1000, mb=64, mq=4096, ms=8192):
    return vb.make_config(hq, hkv, d, P, pages, mb, mq, ms)


def test_unsupported_geometry_is_rejected_not_tuned(vb):
    assert vb.vosti_workspace_bytes(cfg(vb)) > 0
    for bad in (dict(d=96), dict(P=32), dict(hq=30), dict(hq=24, hkv=8), dict(pages=0)):
        assert vb.vosti_workspace_bytes(cfg(vb, **bad)) == 0
        with pytest.raises(vb.VostiError) as e:
            vb.vosti_plan(cfg(vb, **bad), [1], [0], [1])
        assert e.value.status == vb.VOSTI_ERR_UNSUPPORTED_CONFIG


def test_plan_premises(vb):
    c = cfg(vb)
    for q, s, n in (([2], [5], [6]), ([-1], [0], [4]), ([1], [-1], [4]), ([1], [0], [9000]),
                    ([4097], [0], [4097])):
        with pytest.raises(vb.VostiError) as e:
            vb.vosti_plan(c, q, s, n)
        assert e.value.status == vb.VOSTI_ERR_OUT_OF_RANGE
    items, n_split, n_part = vb.vosti_plan(c, [0, 0], [0, 3], [0, 3])
    assert len(items) == 0 and n_split == 0 and n_part == 0


def plan_of_request(vb, c, q, s):
    items, n_split, n_part = vb.vosti_plan(c, [q], [s], [s + q])
    return sorted(map(tuple, items[:, 1:])), n_split, n_part


def test_plan_is_a_pure_function_of_the_request(vb):
    """Co-batching, batch order and seq_len slack must not change which
    (row group, split range) items a request gets."""
    c = cfg(vb)
    rng = np.random.default_rng(0)
    reqs = [(1, 511), (1, 512), (1, 4095), (3, 1000), (8, 2047), (9, 100), (512, 0), (512, 7000),
            (128, 512), (1, 0)]
    alone = {r: plan_of_request(vb, c, *r) for r in reqs}
    for _ in range(5):
        order = rng.permutation(len(reqs))
        q = [reqs[i][0] for i in order]
        s = [reqs[i][1] for i in order]
        n = [a + b + int(rng.integers(0, 50)) for a, b in zip(q, s)]
        items, n_split, n_part = vb.vosti_plan(c, q, s, n)
        for slot, i in enumerate(order):
            mine = sorted(tuple(it[1:]) for it in items if it[0] == slot)
            assert mine == alone[reqs[i]][0]
        assert n_split == sum(a[1] for a in alone.values())
        assert n_part == sum(a[2] for a in alone.values())


def test_plan_shapes(vb):
    c = cfg(vb)          # G = 4, rows per group 16, split 512, split-parallel up to 32 rows
    # decode at p = 1300: splits 0,1,2, one row group, split-parallel
    items, n_split, n_part = plan_of_request(vb, c, 1, 1300)
    assert items == [(0, 0, 1), (0, 1, 2), (0, 2, 3)] and n_split == 3
    assert n_part == 8 * 3 * 4                      # kv heads x splits x rows
    # 8 tokens x G=4 = 32 rows: two row groups, still split-parallel
    items, n_split, _ = plan_of_request(vb, c, 8, 508)   # positions 508..515
    assert items == [(0, 0, 1), (1, 0, 1), (1, 1, 2)] and n_split == 3
    # 9 tokens: 36 rows > 32 -> one tile item that walks all its splits in order
    items, n_split, n_part = plan_of_request(vb, c, 9, 1020)
    assert n_split == 0 and n_part == 0
    assert items == [(0, 0, 3)]
    # 100 tokens x G=4 = 400 rows: two 256-row tiles starting at row groups 0 and 16
    items, n_split, _ = plan_of_request(vb, c, 100, 500)
    assert n_split == 0 and items == [(0, 0, 2), (16, 0, 2)]
    # boundaries: position exactly at a split edge
    assert plan_of_request(vb, c, 1, 511)[0] == [(0, 0, 1)]
    assert plan_of_request(vb, c, 1, 512)[0] == [(0, 0, 1), (0, 1, 2)]


def test_plan_under_a_sliding_window(vb):
    """Items only for the splits that hold a key some row of the group sees; the first
    visible key of a row at p is max(0, p - w + 1)."""
    c = cfg(vb)          # G = 4, 8 kv heads

    def plan_w(q, s, w):
        items, n_split, n_part = vb.vosti_plan_ex(c, [q], [s], [s + q], w)
        return list(map(tuple, items[:, 1:])), n_split, n_part

    # window 0 and a window longer than the context: the unwindowed plan
    for q, s in ((1, 1300), (8, 508), (9, 1020), (100, 500)):
        base = vb.vosti_plan(c, [q], [s], [s + q])
        for w in (0, s + q, 10 ** 6):
            got = vb.vosti_plan_ex(c, [q], [s], [s + q], w)
            assert (got[0] == base[0]).all() and got[1:] == base[1:]
    # decode at p = 1300, w = 100: keys 1201..1300, all in split 2
    assert plan_w(1, 1300, 100) == ([(0, 2, 3)], 1, 8 * 1 * 4)
    # p = 1030, w = 100: keys 931..1030 -> tiles 14, 15 of split 1 and tile 16 of split 2 (longest first)
    assert plan_w(1, 1030, 100) == ([(0, 1, 2), (0, 2, 3)], 2, 8 * 2 * 4)
    # w = 1: only the key at p
    assert plan_w(1, 1024, 1) == ([(0, 2, 3)], 1, 8 * 4)
    assert plan_w(1, 1023, 1) == ([(0, 1, 2)], 1, 8 * 4)
    # 8 tokens at 508..515, w = 4: group 0 (tokens 0..3, keys 505..511) split 0 only;
    # group 1 (tokens 4..7, keys 509..515) splits 0 and 1; partial rows from split 0
    items, n_split, n_part = plan_w(8, 508, 4)
    assert sorted(items) == [(0, 0, 1), (1, 0, 1), (1, 1, 2)] and n_part == 8 * 2 * 32
    # the same tokens at 1020..1027, w = 4: the request's first split is 1, so two splits of partial rows
    items, n_split, n_part = plan_w(8, 1020, 4)
    assert sorted(items) == [(0, 1, 2), (1, 1, 2), (1, 2, 3)] and n_part == 8 * 2 * 32
    # a tile item reports the splits it walks: 100 tokens at 2000, w = 600 -> rows 0..255 are tokens
    # 0..63 (keys 1401..2063: splits 2..4), rows 256..399 tokens 64..99 (keys 1465..2099: splits 2..4)
    items, n_split, n_part = plan_w(100, 2000, 600)
    assert n_split == 0 and n_part == 0 and items == [(0, 2, 5), (16, 2, 5)]
    with pytest.raises(vb.VostiError) as e:
        vb.vosti_plan_ex(c, [1], [0], [1], -1)
    assert e.value.status == vb.VOSTI_ERR_INVALID_ARG


def test_items_are_ordered_longest_first(vb):
    c = cfg(vb)
    items, n_split, _ = vb.vosti_plan(c, [1, 1, 1], [100, 4000, 700], [101, 4001, 701])
    # tiles walked per split-parallel item
    def tiles(it):
        p = [100, 4000, 700][it[0]]
        return min(it[3] * 8, p // 64 + 1) - it[2] * 8
    t = [tiles(it) for it in items[:n_split]]
    assert t == sorted(t, reverse=True)


# The contract words of the committed library and the fingerprint they hash to.  A change of any
# rule id, frozen size or the lazy-maximum step changes the fingerprint; this test then fails
# until the version word (first) is raised as well and the pair below is updated together --
# which is the point: bits may only change under a new version.
PINNED_CONTRACT = [2, 64, 512, 16, 32, 16, 1, 2, 0x41000000, 3, 1, 1, 1, 1, 1]
PINNED_FINGERPRINT = 0x0BE65E7990228BE9


def test_fingerprint_is_derived_from_the_contract_words(vb):
    words = vb.vosti_contract()
    # FNV-1a over the words, eight bytes each (the library's own rule, restated)
    h = 1469598103934665603
    for w in words:
        for i in range(8):
            h ^= (w >> (8 * i)) & 0xFF
            h = (h * 1099511628211) % (1 << 64)
    assert vb.vosti_fingerprint() == h
    if words != PINNED_CONTRACT:
        assert words[0] != PINNED_CONTRACT[0], \
            "a rule or frozen size of the numerical contract changed without a new version"
        raise AssertionError("contract changed under a new version: update PINNED_CONTRACT / PINNED_FINGERPRINT")
    assert vb.vosti_fingerprint() == PINNED_FINGERPRINT
    c = vb.vosti_constants()
    assert (c["key_tile"], c["split_len"], c["rows_per_group"]) == tuple(words[1:4])


PINNED_LINEAR_CONTRACT = [1, 128, 256, 128, 64, 148, 16, 1, 1]
PINNED_LINEAR_FINGERPRINT = 0xB054C1B6905B3D79


def test_linear_fingerprint_is_derived_from_its_contract_words(vb):
    """The linear layer's identity: tile sizes, the segment rule's constants (the wave of 148 units
    is a frozen number), one id per reduction rule.  Same discipline as the attention library."""
    from paper_2609_38981_b200 import linear as vl
    words = vl.vosti_linear_contract()
    h = 1469598103934665603
    for w in words:
        for i in range(8):
            h ^= (w >> (8 * i)) & 0xFF
            h = (h * 1099511628211) % (1 << 64)
    assert vl.vosti_linear_fingerprint() == h
    if words != PINNED_LINEAR_CONTRACT:
        assert words[0] != PINNED_LINEAR_CONTRACT[0], "a linear-layer rule changed without a new version"
        raise AssertionError("linear contract changed under a new version: update the pinned pair")
    assert h == PINNED_LINEAR_FINGERPRINT
    # the segment rule is what the words say: floor(148 / column tiles), segments of >= 16 blocks
    assert vl.vosti_linear_segments(4096, 4096) == min(148 // (4096 // 256), 4096 // 64 // 16)
    assert vl.vosti_linear_segments(28672, 4096) == 1
    assert vl.vosti_linear_segments(4096, 14336) == min(148 // 16, 14336 // 64 // 16)
