"""The allocation-free entry point (vosti_paged_attention_noalloc).

It serves callers that may not allocate -- code under stream capture, loops
whose memory is handed out by an outside allocator, plug-ins without the right
to create device memory -- by keeping its scratch in a fixed device array inside
the library.  It must give exactly the bits of vosti_paged_attention, on every
call, although all calls reuse that one array.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from paper_2609_38981_b200 import inputs

pytestmark = pytest.mark.gpu


def _setup():
    from paper_2609_38981_b200.harness import DeviceCache
    geo = inputs.Geometry(8, 2, 128, 16)
    contexts = (1, 300, 512, 513, 1100, 1601)
    reqs = [inputs.make_request(geo, 91, i, n) for i, n in enumerate(contexts)]
    tables = inputs._assign_private_pages(inputs.generator(91), geo, 700, contexts)
    cache = DeviceCache(geo, 700, max_batch=8, max_total_q=4096, max_seq_len=2048, pool_fill="random")
    cache.upload(reqs, tables)
    return geo, contexts, reqs, tables, cache


def test_noalloc_matches_the_context_entry_point_twice_in_a_row():
    from paper_2609_38981_b200 import binding as vb
    from paper_2609_38981_b200.harness import bf16_bits
    geo, contexts, reqs, tables, cache = _setup()
    scale = geo.head_dim ** -0.5
    bt = inputs.block_table_array(tables, stride=128, fill=-1)
    # call A: single-token decode of every request; call B: speculative windows of 2..4 tokens
    calls = [
        ([1] * len(reqs), [n - 1 for n in contexts]),
        ([min(n, 1 + i % 4) for i, n in enumerate(contexts)], None),
    ]
    for q_lens, starts in calls:
        starts = [n - ql for n, ql in zip(contexts, q_lens)] if starts is None else starts
        q = torch.cat([r.q_rows(s, ql) for r, s, ql in zip(reqs, starts, q_lens)]).to(cache.device)
        ref = bf16_bits(cache.attend(q, q_lens, starts, list(contexts), bt, scale))
        for rep in range(2):        # two calls in a row share the static scratch
            out = torch.empty_like(q)
            out.view(torch.int16).fill_(0x7FC1)
            vb.vosti_paged_attention_noalloc(geo.n_q_heads, geo.n_kv_heads, geo.head_dim,
                                             geo.page_size, cache.pool, q, out, q_lens, starts,
                                             list(contexts), bt, scale)
            torch.cuda.synchronize()
            assert torch.equal(bf16_bits(out), ref), f"noalloc differs from the context path (rep {rep})"
    cache.close()


def test_noalloc_rejects_what_its_scratch_cannot_hold():
    from paper_2609_38981_b200 import binding as vb
    geo, contexts, reqs, tables, cache = _setup()
    bt = inputs.block_table_array(tables, stride=128)
    q = torch.zeros(300, geo.n_q_heads, geo.head_dim, dtype=torch.bfloat16, device=cache.device)
    out = torch.empty_like(q)
    args = (geo.n_q_heads, geo.n_kv_heads, geo.head_dim, geo.page_size, cache.pool, q, out)
    with pytest.raises(vb.VostiError) as e:        # a long query: not a split-parallel request
        vb.vosti_paged_attention_noalloc(*args, [200], [0], [200], bt[:1], 0.1)
    assert e.value.status == vb.VOSTI_ERR_UNSUPPORTED_CONFIG
    with pytest.raises(vb.VostiError) as e:        # more requests than the metadata area holds
        vb.vosti_paged_attention_noalloc(*args, [1] * 65, [0] * 65, [1] * 65,
                                         np.zeros((65, 1), np.int32), 0.1)
    assert e.value.status == vb.VOSTI_ERR_WORKSPACE
    with pytest.raises(vb.VostiError) as e:        # page id outside the pool
        vb.vosti_paged_attention_noalloc(*args, [1], [0], [1], np.array([[700]], np.int32), 0.1)
    assert e.value.status == vb.VOSTI_ERR_OUT_OF_RANGE
    cache.close()
