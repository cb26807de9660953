"""The allocation-free entry point (vosti_paged_attention_noalloc).

It serves callers that may not allocate -- an engine that has handed all device
memory to its own pool allocator, a decode loop that cannot afford the
device-wide synchronisation of cudaMalloc, a plug-in that is given device
pointers but may create none -- by keeping its scratch in a fixed device array
inside the library.  It must give exactly the bits of vosti_paged_attention, on
every call, although all calls reuse that one array.

This file sorts after every other test file so that a run which stops at the
first failure (pytest -x) has already exercised the rest of the library when it
gets here: the entry point is an addition beside the hot path, and a fault in
it should not hide the state of the path itself."""
import numpy as np
import pytest
import torch

from paper_2609_38981_b200 import inputs

pytestmark = pytest.mark.gpu


def _setup(geo=None, contexts=(1, 300, 512, 513, 1100, 1601), pages=700, max_seq_len=2048, seed=91):
    from paper_2609_38981_b200.harness import DeviceCache
    geo = geo or inputs.Geometry(8, 2, 128, 16)
    reqs = [inputs.make_request(geo, seed, i, n) for i, n in enumerate(contexts)]
    tables = inputs._assign_private_pages(inputs.generator(seed), geo, pages, contexts)
    cache = DeviceCache(geo, pages, max_batch=max(8, len(contexts)), max_total_q=4096,
                        max_seq_len=max_seq_len, pool_fill="random")
    cache.upload(reqs, tables)
    return geo, contexts, reqs, tables, cache


def _noalloc(vb, geo, cache, q, q_lens, starts, contexts, bt, scale):
    out = torch.empty_like(q)
    out.view(torch.int16).fill_(0x7FC1)
    vb.vosti_paged_attention_noalloc(geo.n_q_heads, geo.n_kv_heads, geo.head_dim, geo.page_size,
                                     cache.pool, q, out, q_lens, starts, list(contexts), bt, scale)
    torch.cuda.synchronize()
    return out


@pytest.mark.parametrize("geo", [inputs.Geometry(8, 2, 128, 16), inputs.Geometry(4, 2, 64, 16),
                                 inputs.Geometry(16, 2, 128, 16), inputs.Geometry(2, 2, 64, 16)],
                         ids=["d128_G4", "d64_G2", "d128_G8", "d64_G1"])
def test_noalloc_matches_the_context_entry_point_twice_in_a_row(geo):
    from paper_2609_38981_b200 import binding as vb
    from paper_2609_38981_b200.harness import bf16_bits
    import gpu_util as gu
    geo, contexts, reqs, tables, cache = _setup(geo)
    scale = geo.head_dim ** -0.5
    bt = inputs.block_table_array(tables, stride=128, fill=-1)
    max_q = 32 // geo.group
    # call A: single-token decode of every request; call B: speculative windows of 2..4 tokens
    calls = [
        ([1] * len(reqs), [n - 1 for n in contexts]),
        ([min(n, 1 + i % 4, max_q) for i, n in enumerate(contexts)], None),
    ]
    for q_lens, starts in calls:
        starts = [n - ql for n, ql in zip(contexts, q_lens)] if starts is None else starts
        q = torch.cat([r.q_rows(s, ql) for r, s, ql in zip(reqs, starts, q_lens)]).to(cache.device)
        ref = bf16_bits(cache.attend(q, q_lens, starts, list(contexts), bt, scale))
        for rep in range(2):        # two calls in a row share the static scratch
            out = _noalloc(vb, geo, cache, q, q_lens, starts, contexts, bt, scale)
            assert torch.equal(bf16_bits(out), ref), f"noalloc differs from the context path (rep {rep})"
        # and against the fp64 oracle directly (not only against the other GPU entry point)
        ref64 = np.concatenate([rows[s:s + ql] for rows, s, ql in zip(gu.oracle_rows(reqs, scale), starts, q_lens)])
        gu.assert_parity(bf16_bits(out), ref64, "noalloc vs oracle")
    assert vb.vosti_noalloc_poll_status() == vb.VOSTI_OK
    cache.close()


def test_noalloc_at_its_query_row_limit():
    """Exactly 256 query tokens in one call (the documented maximum) must run and match."""
    from paper_2609_38981_b200 import binding as vb
    from paper_2609_38981_b200.harness import bf16_bits
    contexts = tuple(20 + 3 * i for i in range(64))
    geo, contexts, reqs, tables, cache = _setup(contexts=contexts, pages=900, seed=92)
    scale = geo.head_dim ** -0.5
    bt = inputs.block_table_array(tables)
    q_lens = [4] * 64
    starts = [n - 4 for n in contexts]
    q = torch.cat([r.q_rows(s, 4) for r, s in zip(reqs, starts)]).to(cache.device)
    assert q.shape[0] == 256
    ref = bf16_bits(cache.attend(q, q_lens, starts, list(contexts), bt, scale))
    out = _noalloc(vb, geo, cache, q, q_lens, starts, contexts, bt, scale)
    assert torch.equal(bf16_bits(out), ref)
    cache.close()


def test_noalloc_rejects_what_its_scratch_cannot_hold():
    """One case per documented limit; every one returns before anything is launched."""
    from paper_2609_38981_b200 import binding as vb
    geo, contexts, reqs, tables, cache = _setup()
    bt = inputs.block_table_array(tables, stride=128)
    q = torch.zeros(300, geo.n_q_heads, geo.head_dim, dtype=torch.bfloat16, device=cache.device)
    out = torch.empty_like(q)
    args = (geo.n_q_heads, geo.n_kv_heads, geo.head_dim, geo.page_size, cache.pool, q, out)

    def status_of(q_lens, starts, seqs, table):
        with pytest.raises(vb.VostiError) as e:
            vb.vosti_paged_attention_noalloc(*args, q_lens, starts, seqs, table, 0.1)
        return e.value.status

    # a long query: not a split-parallel request
    assert status_of([200], [0], [200], bt[:1]) == vb.VOSTI_ERR_UNSUPPORTED_CONFIG
    # more requests than the metadata area holds
    assert status_of([1] * 65, [0] * 65, [1] * 65, np.zeros((65, 1), np.int32)) == vb.VOSTI_ERR_WORKSPACE
    # more than 256 query tokens: 33 requests of 8 tokens
    assert status_of([8] * 33, [0] * 33, [8] * 33, np.zeros((33, 1), np.int32)) == vb.VOSTI_ERR_WORKSPACE
    # more than 16384 page ids in use: 5 requests of 3300 pages each (pool ids all valid: page 0)
    wide = np.zeros((5, 3300), np.int32)
    assert status_of([1] * 5, [3300 * 16 - 1] * 5, [3300 * 16] * 5, wide) == vb.VOSTI_ERR_WORKSPACE
    # more than 1024 (row group, split) items: 12 requests x 2 row groups x 50 splits
    n = 50 * 512
    assert status_of([8] * 12, [n - 8] * 12, [n] * 12, np.zeros((12, n // 16), np.int32)) == vb.VOSTI_ERR_WORKSPACE
    # more than 28000 partial rows: 16 requests x 2 KV heads x 30 splits x 32 rows
    n = 30 * 512
    assert status_of([8] * 16, [n - 8] * 16, [n] * 16, np.zeros((16, n // 16), np.int32)) == vb.VOSTI_ERR_WORKSPACE
    # page id outside the pool
    assert status_of([1], [0], [1], np.array([[700]], np.int32)) == vb.VOSTI_ERR_OUT_OF_RANGE
    cache.close()


def test_noalloc_status_word_is_readable_and_sticky():
    """A bounded wait that runs out on this path is reported by the context-free poll, survives
    a later call (calls do not clear the word) and is cleared by the poll that reports it."""
    from paper_2609_38981_b200 import binding as vb
    from paper_2609_38981_b200.harness import bf16_bits
    geo, contexts, reqs, tables, cache = _setup()
    scale = geo.head_dim ** -0.5
    bt = inputs.block_table_array(tables, stride=128)
    assert vb.vosti_noalloc_poll_status() == vb.VOSTI_OK
    vb.vosti_noalloc_selftest_bounded_wait(2000)          # 2 ms: nothing faults, the warp gives up
    q_lens, starts = [1] * len(reqs), [n - 1 for n in contexts]
    q = torch.cat([r.q_rows(s, 1) for r, s in zip(reqs, starts)]).to(cache.device)
    ref = bf16_bits(cache.attend(q, q_lens, starts, list(contexts), bt, scale))
    out = _noalloc(vb, geo, cache, q, q_lens, starts, contexts, bt, scale)
    assert torch.equal(bf16_bits(out), ref)
    assert vb.vosti_noalloc_poll_status() == vb.VOSTI_ERR_TIMEOUT
    assert vb.vosti_noalloc_poll_status() == vb.VOSTI_OK
    cache.close()
