"""Shared-prefix row packing (VOSTI_FLAG_PACK_SHARED_SPLITS): rows of different
requests that name the same physical pages for a whole 512-key split are packed
16 to an MMA tile of the split-parallel kernel, or -- from 48 rows on -- 128 to
a tile of the tensor-memory kernel.  It is a scheduling decision: outputs (and
the log-sum-exp) must be bit for bit those of the unpacked schedule, whatever
mix of requests shares which prefix, and packing must really have happened."""
import numpy as np
import pytest
import torch

from paper_2609_38981_b200 import binding as vb
from paper_2609_38981_b200 import inputs

pytestmark = pytest.mark.gpu

GEOS = {
    "d64_g2": inputs.TINY,
    "d128_g4": inputs.Geometry(8, 2, 128, 16),
    "d128_g8": inputs.Geometry(8, 1, 128, 16),
}
NUM_PAGES = 2048
# packing, with groups of 48 rows or more always routed through the tile kernel
TILES = vb.VOSTI_FLAG_PACK_SHARED_SPLITS | vb.VOSTI_FLAG_PACK_THROUGH_TILES


def family(geo, seed, prefix, suffixes, first_index):
    """Requests that share one `prefix`-token prefix (its whole pages stored once)
    and continue privately for `suffixes[i]` tokens."""
    common = inputs.make_request(geo, seed, 900_000 + first_index, prefix)
    reqs = []
    for i, s in enumerate(suffixes):
        own = inputs.make_request(geo, seed, first_index + i, s)
        reqs.append(inputs.RequestContent(n=prefix + s, q0=0, k=torch.cat([common.k, own.k]),
                                          v=torch.cat([common.v, own.v]),
                                          q=torch.cat([common.q, own.q])))
    return reqs


def build(geo, seed=99):
    """Two families with different prefixes (1100 and 2100 tokens: 2 and 4 complete
    shared splits) and a loner."""
    gen = inputs.generator(seed)
    fam_a = family(geo, seed, 1100, (5, 40, 130, 600, 9, 77), 0)
    fam_b = family(geo, seed, 2100, (3, 300, 17, 64, 512), 100)
    loner = [inputs.make_request(geo, seed, 500, 1500)]
    reqs = fam_a + fam_b + loner
    P = geo.page_size
    need = [inputs.pages_needed(r.n, P) for r in reqs]
    ids = inputs.draw_pages(gen, NUM_PAGES, sum(need))
    at, tables = 0, []
    shared_a = shared_b = None
    for i, (r, c) in enumerate(zip(reqs, need)):
        tb = ids[at:at + c]
        at += c
        if i < len(fam_a):
            shared_a = shared_a or tb[:1100 // P]
            tb = shared_a + tb[1100 // P:]
        elif i < len(fam_a) + len(fam_b):
            shared_b = shared_b or tb[:2100 // P]
            tb = shared_b + tb[2100 // P:]
        tables.append(tb)
    return reqs, tables


def run(geo, reqs, tables, flags, calls, want_lse=True):
    """Upload everything, then run `calls` (lists of (request, start, q_len)) with attend only."""
    from paper_2609_38981_b200.harness import DeviceCache, bf16_bits
    cache = DeviceCache(geo, NUM_PAGES, max_batch=128, max_total_q=4096, max_seq_len=4096, flags=flags)
    # shared pages are written once per family member with identical content: harmless
    cache.upload(reqs, tables)
    scale = geo.head_dim ** -0.5
    outs, lses, packed = [], [], []
    for call in calls:
        idx = [i for i, _, _ in call]
        bt = inputs.block_table_array([tables[i] for i in idx])
        q = torch.cat([reqs[i].q_rows(s, n) for i, s, n in call])
        o, l = cache.attend_ex(q, [n for _, _, n in call], [s for _, s, _ in call],
                               [reqs[i].n for i in idx], bt, scale, want_lse=want_lse)
        outs.append(bf16_bits(o))
        lses.append(l.cpu().view(torch.int32))
        packed.append(vb.vosti_last_schedule(cache.ctx))
    cache.close()
    return outs, lses, packed


@pytest.fixture(scope="module", params=list(GEOS))
def env(request):
    geo = GEOS[request.param]
    reqs, tables = build(geo)
    return dict(geo=geo, reqs=reqs, tables=tables)


def decode_calls(reqs, q_len):
    last = [(i, r.n - q_len, q_len) for i, r in enumerate(reqs)]
    return [last, last[::-1], last[:6], last[3:9]]


@pytest.mark.parametrize("q_len", (1, 2, 4, 8))
def test_packed_schedule_gives_the_same_bits(env, q_len):
    import gpu_util as gu
    geo, reqs, tables = env["geo"], env["reqs"], env["tables"]
    if q_len * geo.group > 32:
        pytest.skip("not a split-parallel request in this geometry")
    calls = decode_calls(reqs, q_len)
    plain, plain_lse, sched0 = run(geo, reqs, tables, 0, calls)
    packed, packed_lse, sched1 = run(geo, reqs, tables, TILES, calls)
    for c in range(len(calls)):
        gu.assert_same_bits(packed[c], plain[c], f"call {c}")
        gu.assert_same_bits(packed_lse[c], plain_lse[c], f"call {c}, log-sum-exp")
        assert sched0[c][1] == 0
        # packed 16 to a tile of the split-parallel kernel, or (48 rows and more) 128 to a packed tile
        assert (sched1[c][1] > 0 or sched1[c][2] > 0) and sched1[c][0] < sched0[c][0], (sched0[c], sched1[c])
    # and both agree with the oracle
    from oracle import oracle
    scale = geo.head_dim ** -0.5
    at = 0
    for i, s, n in calls[0]:
        r = reqs[i]
        ref = oracle.attention_dense(inputs.bits(r.q[s:s + n]), inputs.bits(r.k), inputs.bits(r.v), s, scale)
        gu.assert_parity(packed[0][at:at + n], ref, f"request {i}")
        at += n


def test_expected_number_of_packed_items(env):
    """Family A: 6 requests x 2 complete splits, family B: 5 x 4; with q_len = 1 a request
    brings G rows, so a family's split needs ceil(members * G / 16) packed items."""
    geo, reqs, tables = env["geo"], env["reqs"], env["tables"]
    calls = [[(i, r.n - 1, 1) for i, r in enumerate(reqs)]]
    _, _, sched = run(geo, reqs, tables, TILES, calls)
    G = geo.group
    small = tiles = 0
    for members, splits in ((6, 2), (5, 4)):
        rows = members * G
        if rows >= 48:                      # a large group: 128 rows to a packed tile of the tile kernel
            tiles += splits * -(-rows // 128)
        else:
            small += splits * -(-rows // 16)
    assert sched[0][1] == small and sched[0][2] == tiles, (sched[0], small, tiles)
    # without the flag that forces them, so few shared rows never pay for the tile kernel's launch
    _, _, sched = run(geo, reqs, tables, vb.VOSTI_FLAG_PACK_SHARED_SPLITS, calls)
    assert sched[0][2] == 0 and sched[0][1] == 2 * -(-6 * G // 16) + 4 * -(-5 * G // 16), sched[0]


def test_a_lone_request_and_a_windowed_call_are_not_packed(env):
    from paper_2609_38981_b200.harness import DeviceCache
    geo, reqs, tables = env["geo"], env["reqs"], env["tables"]
    _, _, sched = run(geo, reqs, tables, vb.VOSTI_FLAG_PACK_SHARED_SPLITS, [[(0, reqs[0].n - 1, 1)]])
    assert sched[0][1] == 0
    cache = DeviceCache(geo, NUM_PAGES, max_batch=32, max_total_q=4096, max_seq_len=4096,
                        flags=vb.VOSTI_FLAG_PACK_SHARED_SPLITS)
    cache.upload(reqs, tables)
    idx = list(range(len(reqs)))
    bt = inputs.block_table_array(tables)
    q = torch.cat([r.q_rows(r.n - 1, 1) for r in reqs])
    cache.attend_ex(q, [1] * len(idx), [r.n - 1 for r in reqs], [r.n for r in reqs], bt,
                    geo.head_dim ** -0.5, window=700)
    assert vb.vosti_last_schedule(cache.ctx)[1] == 0
    cache.close()


def test_prefix_sharing_workload_full_size():
    """The benchmark's prefix-sharing batch (128 requests, 2048-token common prefix):
    the unpacked schedule and both packed ones give the same bits."""
    from paper_2609_38981_b200.harness import DeviceCache, bf16_bits
    import gpu_util as gu
    w = inputs.prefix_sharing()
    geo = w.geo
    outs, sched = [], []
    for flags in (0, vb.VOSTI_FLAG_PACK_SHARED_SPLITS, TILES | vb.VOSTI_FLAG_NO_OVERLAP):
        cache = DeviceCache(geo, w.num_pages, max_batch=w.batch, max_total_q=4096,
                            max_seq_len=max(w.seq_lens) + 16, flags=flags)
        cache.upload(w.requests[:1], w.tables[:1], upto=[2048])
        for r, t, s in zip(w.requests, w.tables, w.start_pos):
            cache.append(r.k[2048:s + 1], r.v[2048:s + 1], [s + 1 - 2048], [2048], inputs.block_table_array([t]))
        bt = inputs.block_table_array(w.tables)
        out, _ = cache.attend_ex(w.packed_q(), w.q_lens, w.start_pos, w.seq_lens, bt, geo.head_dim ** -0.5)
        outs.append(bf16_bits(out))
        sched.append(vb.vosti_last_schedule(cache.ctx))
        cache.close()
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])
    # 512 rows share each of the 4 prefix splits: 2048 rows x splits, the amount from which the tile
    # kernel's launch pays, so each split fills 4 packed tiles of 128 rows; the tile kernel runs beside
    # the split-parallel kernel of the private suffixes, or (third run) after it
    for sc in sched[1:]:
        assert sc[1] == 0 and sc[2] == 4 * (128 * geo.group // 128), sched
    gu.sampled_parity(w, outs[2], 64)


@pytest.mark.parametrize("members,q_len", [(40, 1), (23, 2), (70, 1)])
def test_large_groups_go_through_packed_tiles(env, members, q_len):
    """Dozens of requests on one 1100-token prefix (2 complete splits): their rows fill packed
    tiles of 128 (the last one ragged), computed by the tensor-memory kernel in its
    partial-output mode; bits and log-sum-exp equal the unpacked schedule's."""
    import gpu_util as gu
    geo = env["geo"]
    if q_len * geo.group > 32:
        pytest.skip("not a split-parallel request in this geometry")
    rng = np.random.default_rng(members)
    suffixes = [int(x) for x in rng.integers(q_len, 400, size=members)]
    reqs = family(geo, 7, 1100, suffixes, 0)
    P = geo.page_size
    gen = inputs.generator(members)
    need = [inputs.pages_needed(r.n, P) for r in reqs]
    ids = inputs.draw_pages(gen, NUM_PAGES, 1100 // P + sum(c - 1100 // P for c in need))
    shared, at, tables = ids[:1100 // P], 1100 // P, []
    for c in need:
        tables.append(shared + ids[at:at + c - 1100 // P])
        at += c - 1100 // P
    last = [(i, r.n - q_len, q_len) for i, r in enumerate(reqs)]
    calls = [last, last[::-1], last[: members // 2]]
    plain, plain_lse, sched0 = run(geo, reqs, tables, 0, calls)
    packed, packed_lse, sched1 = run(geo, reqs, tables, TILES, calls)
    for c, call in enumerate(calls):
        gu.assert_same_bits(packed[c], plain[c], f"call {c}")
        gu.assert_same_bits(packed_lse[c], plain_lse[c], f"call {c}, log-sum-exp")
        rows = len(call) * q_len * geo.group
        if rows >= 48:
            assert sched1[c][2] == 2 * -(-rows // 128) and sched1[c][1] == 0, (sched1[c], rows)
        else:
            assert sched1[c][1] == 2 * -(-rows // 16) and sched1[c][2] == 0, (sched1[c], rows)
