"""Tiny invariance case on the GPU (4 query heads, 2 KV heads, head_dim 64,
contexts 37 / 100 / 250): parity with the fp64 oracle and bit-exact agreement
of every execution variation with the canonical run (each request alone, one
full-length call, identity page placement, zeroed pool)."""
import numpy as np
import pytest
import torch

from paper_2609_38981_b200 import inputs

pytestmark = pytest.mark.gpu

GEO = inputs.TINY
CONTEXTS = (37, 100, 250)
SCALE = GEO.head_dim ** -0.5
NUM_PAGES = 256


@pytest.fixture(scope="module")
def env():
    from paper_2609_38981_b200.harness import DeviceCache
    import gpu_util as gu
    reqs = inputs.tiny_requests(GEO, CONTEXTS)
    ident, at = [], 0
    for n in CONTEXTS:
        c = inputs.pages_needed(n, GEO.page_size)
        ident.append(list(range(at, at + c)))
        at += c

    def cache(fill="zeros", **kw):
        return DeviceCache(GEO, NUM_PAGES, max_batch=8, max_total_q=1024, max_seq_len=1024,
                           pool_fill=fill, **kw)

    canon = {}
    for i, r in enumerate(reqs):
        c = cache()
        canon[i] = gu.run_schedule(c, reqs, ident, [[(i, 0, r.n)]], SCALE)[i]
        c.close()
    return dict(reqs=reqs, ident=ident, cache=cache, canon=canon, gu=gu)


def check_all(env, outs, what):
    for i in outs:
        env["gu"].assert_same_bits(outs[i], env["canon"][i], f"{what}, request {i}")


def test_canonical_run_matches_oracle(env):
    ref = env["gu"].oracle_rows(env["reqs"], SCALE)
    for i in range(3):
        assert (env["canon"][i] != 0x7FC2).all() and (env["canon"][i] != 0x7FC1).all()
        env["gu"].assert_parity(env["canon"][i], ref[i], f"request {i}")


def test_kv_append_is_bit_exact_against_oracle(env):
    from oracle import oracle
    reqs, gu = env["reqs"], env["gu"]
    gen = inputs.generator(99)
    tables = inputs._assign_private_pages(gen, GEO, NUM_PAGES, CONTEXTS)
    c = env["cache"](fill="random")
    host_pool = inputs.bits(c.pool.cpu()).copy()
    bt = inputs.block_table_array(tables, stride=20)
    for starts, lens in (([0, 0, 0], [20, 1, 250]), ([20, 1, 0], [17, 99, 0])):
        k = torch.cat([r.k[s:s + l] for r, s, l in zip(reqs, starts, lens)])
        v = torch.cat([r.v[s:s + l] for r, s, l in zip(reqs, starts, lens)])
        c.append(k, v, lens, starts, bt)
        oracle.kv_append(host_pool, inputs.bits(k), inputs.bits(v), lens, starts, bt)
    assert np.array_equal(inputs.bits(c.pool.cpu()), host_pool)
    c.close()


@pytest.mark.parametrize("order", [(0, 1, 2), (2, 0, 1)])
def test_cobatched_full_prefill(env, order):
    c = env["cache"]()
    outs = env["gu"].run_schedule(c, env["reqs"], env["ident"],
                                  [[(i, 0, env["reqs"][i].n) for i in order]], SCALE)
    check_all(env, outs, f"co-batched order {order}")
    c.close()


@pytest.mark.parametrize("chunk", [1, 7, 32])
@pytest.mark.parametrize("together", [False, True])
def test_chunked_prefill(env, chunk, together):
    gu, reqs = env["gu"], env["reqs"]
    c = env["cache"]()
    per = {i: gu.chunked(r.n, chunk) for i, r in enumerate(reqs)}
    if together:
        steps = max(len(v) for v in per.values())
        sched = [[(i, *per[i][s]) for i in per if s < len(per[i])] for s in range(steps)]
    else:
        sched = [[(i, s, q)] for i in per for s, q in per[i]]
    outs = gu.run_schedule(c, reqs, env["ident"], sched, SCALE)
    check_all(env, outs, f"chunk {chunk} together={together}")
    c.close()


def test_mixed_chunk_schedule(env):
    gu, reqs = env["gu"], env["reqs"]
    c = env["cache"]()
    sched = [[(2, 0, 7), (0, 0, 30)], [(2, 7, 32), (1, 0, 64)], [(2, 39, 1), (1, 64, 1), (0, 30, 7)],
             [(2, 40, 88), (1, 65, 35)], [(2, 128, 122)]]
    outs = gu.run_schedule(c, reqs, env["ident"], sched, SCALE)
    check_all(env, outs, "mixed schedule")
    c.close()


def test_decode_of_last_tokens_equals_prefill(env):
    gu, reqs = env["gu"], env["reqs"]
    c = env["cache"]()
    sched = [[(i, 0, r.n - 8) for i, r in enumerate(reqs)]]
    sched += [[(i, r.n - 8 + t, 1) for i, r in enumerate(reqs)] for t in range(8)]
    outs = gu.run_schedule(c, reqs, env["ident"], sched, SCALE)
    check_all(env, outs, "prefill then 8 decode steps")
    c.close()


def test_speculative_windows_equal_decode(env):
    gu, reqs = env["gu"], env["reqs"]
    for ql in (2, 3, 4):
        c = env["cache"]()
        sched = [[(i, 0, r.n - 12) for i, r in enumerate(reqs)]]
        sched += [[(i, r.n - 12 + w * ql, ql) for i, r in enumerate(reqs)] for w in range(12 // ql)]
        outs = gu.run_schedule(c, reqs, env["ident"], sched, SCALE)
        check_all(env, outs, f"speculative q_len {ql}")
        c.close()


@pytest.mark.parametrize("placement", ["perm0", "perm1", "reversed", "interleaved"])
def test_page_placement(env, placement):
    gu, reqs = env["gu"], env["reqs"]
    need = [inputs.pages_needed(n, GEO.page_size) for n in CONTEXTS]
    if placement.startswith("perm"):
        tables = inputs._assign_private_pages(inputs.generator(7 + int(placement[-1])), GEO,
                                              NUM_PAGES, CONTEXTS)
    elif placement == "reversed":
        ids = list(range(NUM_PAGES - 1, NUM_PAGES - 1 - sum(need), -1))
        tables = [ids[sum(need[:i]):sum(need[:i + 1])] for i in range(3)]
    else:
        tables = [[3 * b + i for b in range(need[i])] for i in range(3)]
    c = env["cache"]()
    outs = gu.run_schedule(c, reqs, tables, [[(i, 0, r.n) for i, r in enumerate(reqs)]], SCALE)
    check_all(env, outs, placement)
    c.close()


@pytest.mark.parametrize("fill", [-1, 10 ** 6, "random"])
def test_wider_page_tables_with_unused_garbage(env, fill):
    gu, reqs = env["gu"], env["reqs"]
    c = env["cache"]()
    if fill == "random":
        fill = int(np.random.default_rng(0).integers(0, NUM_PAGES))
    outs = gu.run_schedule(c, reqs, env["ident"], [[(i, 0, r.n) for i, r in enumerate(reqs)]],
                           SCALE, stride=64, fill=fill)
    check_all(env, outs, f"stride 64 fill {fill}")
    c.close()


@pytest.mark.parametrize("fill", ["random", "nan"])
def test_pool_garbage_beyond_the_sequence(env, fill):
    gu, reqs = env["gu"], env["reqs"]
    c = env["cache"](fill=fill)
    sched = [[(i, *gu.chunked(r.n, 50)[w]) for i, r in enumerate(reqs)
              if w < len(gu.chunked(r.n, 50))] for w in range(5)]
    outs = gu.run_schedule(c, reqs, env["ident"], sched, SCALE)
    check_all(env, outs, f"pool fill {fill}")
    c.close()


def test_seq_len_longer_than_the_rows_attended(env):
    """Rows at positions [s, s+q) of a fully cached request: later keys exist
    but are masked."""
    gu, reqs = env["gu"], env["reqs"]
    c = env["cache"]()
    c.upload(reqs, env["ident"])
    sched = [[(0, 5, 20), (1, 0, 64), (2, 100, 3)], [(2, 249, 1), (1, 99, 1), (0, 0, 1)]]
    outs = gu.run_schedule(c, reqs, env["ident"], sched, SCALE, append=False,
                           seq_lens_override={0: 37, 1: 100, 2: 250})
    for i, lo, hi in ((0, 5, 25), (1, 0, 64), (2, 100, 103), (2, 249, 250), (1, 99, 100), (0, 0, 1)):
        gu.assert_same_bits(outs[i][lo:hi], env["canon"][i][lo:hi], f"request {i} rows {lo}:{hi}")
    c.close()


def test_repeated_calls_give_identical_bits(env):
    gu, reqs = env["gu"], env["reqs"]
    c = env["cache"]()
    c.upload(reqs, env["ident"])
    bt = inputs.block_table_array(env["ident"])
    q = torch.cat([r.q for r in reqs])
    first = None
    for it in range(20):
        stream = torch.cuda.Stream() if it % 2 else None
        if stream is not None:
            stream.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(stream):
                out = c.attend(q, list(CONTEXTS), [0, 0, 0], list(CONTEXTS), bt, SCALE)
            torch.cuda.current_stream().wait_stream(stream)
        else:
            out = c.attend(q, list(CONTEXTS), [0, 0, 0], list(CONTEXTS), bt, SCALE)
        bits_ = gu.bf16_bits(out)
        first = bits_ if first is None else first
        assert torch.equal(bits_, first)
    c.close()


def test_zero_scale_and_negative_zero_values(env):
    """sigma = 0 gives prefix means; a value column of -0.0 must come out as
    +0.0 in every variation (sign of an exact zero is canonical)."""
    gu = env["gu"]
    r = inputs.make_request(GEO, 5, 0, 70)
    r.v[:, :, 3] = -0.0
    tables = [list(range(5))]
    c = env["cache"]()
    full = gu.run_schedule(c, [r], tables, [[(0, 0, 70)]], 0.0)[0]
    c.close()
    c = env["cache"](fill="random")
    dec = gu.run_schedule(c, [r], tables, [[(0, s, 1)] for s in range(70)], 0.0)[0]
    c.close()
    gu.assert_same_bits(dec, full, "decode vs prefill at scale 0")
    assert (full[:, :, 3] == 0).all()
    means = torch.cumsum(r.v.to(torch.float64), 0) / torch.arange(1, 71)[:, None, None]
    want = means[:, [0, 0, 1, 1], :].numpy()
    gu.assert_parity(full, want, "prefix mean")


def test_rejected_calls_launch_nothing(env):
    from paper_2609_38981_b200 import binding as vb
    c = env["cache"]()
    q = torch.zeros(4, GEO.n_q_heads, GEO.head_dim, dtype=torch.bfloat16, device="cuda")
    out = torch.empty_like(q)
    before = vb.vosti_launch_count(c.ctx)
    bad = [
        dict(q_lens=[4], start=[0], seq=[3], bt=[[0]]),                  # start+q > seq
        dict(q_lens=[4], start=[30], seq=[34], bt=[[0, 1]]),             # table too short
        dict(q_lens=[4], start=[0], seq=[4], bt=[[NUM_PAGES]]),          # page id outside pool
        dict(q_lens=[4], start=[0], seq=[4], bt=[[-1]]),
        dict(q_lens=[4], start=[0], seq=[2000], bt=[[0] * 125]),         # seq_len > max_seq_len
    ]
    for b in bad:
        with pytest.raises(vb.VostiError) as e:
            vb.vosti_paged_attention(c.ctx, q, out, b["q_lens"], b["start"], b["seq"],
                                     np.array(b["bt"], np.int32), SCALE)
        assert e.value.status == vb.VOSTI_ERR_OUT_OF_RANGE
    with pytest.raises(vb.VostiError) as e:
        vb.vosti_paged_attention(c.ctx, q, out, [4], [0], [4], np.array([[0]], np.int32), -1.0)
    assert e.value.status == vb.VOSTI_ERR_INVALID_ARG
    k = torch.zeros(4, GEO.n_kv_heads, GEO.head_dim, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(vb.VostiError):
        vb.vosti_kv_append(c.ctx, k, k, [4], [14], np.array([[0]], np.int32))   # crosses the table
    assert vb.vosti_launch_count(c.ctx) == before
    assert vb.vosti_poll_device_status(c.ctx) == vb.VOSTI_OK
    c.close()


def test_write_slot_check(env):
    from paper_2609_38981_b200 import binding as vb
    c = env["cache"](flags=vb.VOSTI_FLAG_CHECK_WRITE_SLOTS)
    k = torch.zeros(2, GEO.n_kv_heads, GEO.head_dim, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(vb.VostiError) as e:     # two requests writing the same slot of page 0
        vb.vosti_kv_append(c.ctx, k, k, [1, 1], [3, 3], np.array([[0], [0]], np.int32))
    assert e.value.status == vb.VOSTI_ERR_OUT_OF_RANGE
    vb.vosti_kv_append(c.ctx, k, k, [1, 1], [3, 4], np.array([[0], [0]], np.int32))
    c.close()
