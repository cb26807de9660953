"""Contexts that span several KV splits (split length 512) and sit on tile /
split / page boundaries: the split-parallel path (partials + left fold in the
combine kernel) must agree bit for bit with the sequential path (fold in
registers), and both with the fp64 oracle within tolerance."""
import numpy as np
import pytest
import torch

from paper_2609_38981_b200 import inputs

pytestmark = pytest.mark.gpu

GEOS = {
    "d64_g2": inputs.TINY,
    "d128_g4": inputs.Geometry(8, 2, 128, 16),
    "d128_g8": inputs.Geometry(8, 1, 128, 16),
    "d64_g1": inputs.Geometry(2, 2, 64, 16),
    "d128_g16": inputs.Geometry(16, 1, 128, 16),
    "d64_g8": inputs.Geometry(8, 1, 64, 16),
    "d128_g1": inputs.Geometry(2, 2, 128, 16),
}
# around split edges (512 k), tile edges (64 k), page edges (16 k), and the degenerate 1
CONTEXTS = (1, 16, 511, 512, 513, 1023, 1024, 1025, 1600)
NUM_PAGES = 640


@pytest.fixture(scope="module", params=list(GEOS))
def env(request):
    from paper_2609_38981_b200.harness import DeviceCache
    import gpu_util as gu
    geo = GEOS[request.param]
    scale = geo.head_dim ** -0.5
    reqs = [inputs.make_request(geo, 4242, i, n) for i, n in enumerate(CONTEXTS)]
    gen = inputs.generator(4242)
    tables = inputs._assign_private_pages(gen, geo, NUM_PAGES, CONTEXTS)

    def cache(fill="zeros"):
        return DeviceCache(geo, NUM_PAGES, max_batch=16, max_total_q=8192, max_seq_len=2048,
                           pool_fill=fill)

    c = cache()
    canon = {}
    for i, r in enumerate(reqs):          # canonical: alone, one full-length call
        canon.update({i: gu.run_schedule(c, reqs, tables, [[(i, 0, r.n)]], scale)[i]})
    c.close()
    return dict(geo=geo, scale=scale, reqs=reqs, tables=tables, cache=cache, canon=canon, gu=gu)


def check(env, outs, what, rows=None):
    for i in outs:
        lo, hi = (0, env["reqs"][i].n) if rows is None else rows(i)
        env["gu"].assert_same_bits(outs[i][lo:hi], env["canon"][i][lo:hi], f"{what}, request {i}")


def test_parity_with_oracle(env):
    ref = env["gu"].oracle_rows(env["reqs"], env["scale"])
    for i in env["canon"]:
        env["gu"].assert_parity(env["canon"][i], ref[i], f"request {i}")


def test_cobatched_prefill(env):
    c = env["cache"]()
    outs = env["gu"].run_schedule(c, env["reqs"], env["tables"],
                                  [[(i, 0, r.n) for i, r in enumerate(env["reqs"])]], env["scale"])
    check(env, outs, "co-batched")
    c.close()


@pytest.mark.parametrize("chunk", [3, 64, 128, 500])
def test_chunked_prefill(env, chunk):
    gu, reqs = env["gu"], env["reqs"]
    c = env["cache"]("random")
    per = {i: gu.chunked(r.n, chunk) for i, r in enumerate(reqs)}
    steps = max(len(v) for v in per.values())
    sched = [[(i, *per[i][s]) for i in per if s < len(per[i])] for s in range(steps)]
    outs = gu.run_schedule(c, reqs, env["tables"], sched, env["scale"])
    check(env, outs, f"chunk {chunk}")
    c.close()


@pytest.mark.parametrize("ql", [1, 2, 4])
def test_decode_and_speculative_tail(env, ql):
    """The last 8 positions by split-parallel calls of q_len 1, 2 or 4 after a
    sequential prefill of the rest."""
    gu, reqs = env["gu"], env["reqs"]
    c = env["cache"]("nan")
    tail = {i: min(8, r.n) for i, r in enumerate(reqs)}
    sched = [[(i, 0, r.n - tail[i]) for i, r in enumerate(reqs) if r.n > tail[i]]]
    for w in range(8 // ql):
        sched.append([(i, r.n - tail[i] + w * ql, ql) for i, r in enumerate(reqs)
                      if w * ql + ql <= tail[i]])
    sched = [s for s in sched if s]
    outs = gu.run_schedule(c, reqs, env["tables"], sched, env["scale"])
    check(env, outs, f"tail q_len {ql}", rows=lambda i: (0, reqs[i].n - tail[i] % ql))
    c.close()


def test_decode_every_position_across_a_split_edge(env):
    """Single-token decode at positions 500..530 of the longest request."""
    gu, reqs = env["gu"], env["reqs"]
    i = len(reqs) - 1
    c = env["cache"]()
    c.upload(reqs, env["tables"])
    sched = [[(i, p, 1)] for p in range(500, 531)]
    outs = gu.run_schedule(c, reqs, env["tables"], sched, env["scale"], append=False,
                           seq_lens_override={i: reqs[i].n})
    gu.assert_same_bits(outs[i][500:531], env["canon"][i][500:531], "decode across split edge")
    c.close()


def test_companion_with_a_much_longer_context(env):
    """A decode next to a 1600-token stranger and next to nothing: same bits."""
    gu, reqs = env["gu"], env["reqs"]
    c = env["cache"]()
    c.upload(reqs, env["tables"])
    long_i = len(reqs) - 1
    for i in (0, 1, 2, 4):
        p = reqs[i].n - 1
        outs = gu.run_schedule(c, reqs, env["tables"], [[(long_i, 1599, 1), (i, p, 1)]],
                               env["scale"], append=False,
                               seq_lens_override={i: reqs[i].n, long_i: 1600})
        gu.assert_same_bits(outs[i][p:p + 1], env["canon"][i][p:p + 1], f"request {i} with stranger")
    c.close()
