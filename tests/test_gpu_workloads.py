"""The serving-shaped workloads at full size, driven the way the benchmark drives
them: parity against the oracle (every output row of the decode-shaped batches, 512
sampled rows of the prefill batch) and bitwise self-invariance against the same
requests run in other ways."""
import numpy as np
import pytest
import torch

from paper_2609_38981_b200 import inputs

pytestmark = pytest.mark.gpu


def make_cache(w, max_total_q=8192, fill="zeros", flags=0):
    from paper_2609_38981_b200.harness import DeviceCache
    return DeviceCache(w.geo, w.num_pages, max_batch=max(w.batch, 8), max_total_q=max_total_q,
                       max_seq_len=max(w.seq_lens), pool_fill=fill, flags=flags)


def run_step(cache, w):
    """The benchmark's step: append the batch's new tokens, then attend."""
    from paper_2609_38981_b200.harness import bf16_bits
    bt = inputs.block_table_array(w.tables)
    kn, vn = w.packed_new_kv()
    cache.append(kn, vn, w.q_lens, w.start_pos, bt)
    return bf16_bits(cache.attend(w.packed_q(), w.q_lens, w.start_pos, w.seq_lens, bt,
                                  w.geo.head_dim ** -0.5))


def rows_of(w):
    return np.concatenate([[0], np.cumsum(w.q_lens)])


def test_decode_heavy_full_size():
    import gpu_util as gu
    from paper_2609_38981_b200 import binding as vb
    w = inputs.decode_heavy()
    assert w.batch == 64 and w.num_pages == 200_000 and w.kv_bytes() > 500e6
    cache = make_cache(w)
    cache.upload(w.requests, w.tables, upto=w.start_pos)
    out = run_step(cache, w)
    assert vb.vosti_poll_device_status(cache.ctx) == vb.VOSTI_OK
    gu.full_parity(w, out)                   # all 2,048 (request, head) rows
    # each of a few requests alone, and next to one other request: same bits as in the batch of 64
    bt = inputs.block_table_array(w.tables)
    scale = w.geo.head_dim ** -0.5
    for r in (0, 17, 63):
        q = w.requests[r].q_rows(w.start_pos[r], 1)
        alone = gu.bf16_bits(cache.attend(q, [1], [w.start_pos[r]], [w.seq_lens[r]], bt[r:r + 1], scale))
        assert torch.equal(alone[0], out[r])
        pair = [5, r]
        q2 = torch.cat([w.requests[i].q_rows(w.start_pos[i], 1) for i in pair])
        two = gu.bf16_bits(cache.attend(q2, [1, 1], [w.start_pos[i] for i in pair],
                                        [w.seq_lens[i] for i in pair], bt[pair], scale))
        assert torch.equal(two[1], out[r])
    cache.close()
    # another physical placement of the same logical batch
    w2 = inputs.decode_heavy()
    perm = inputs.draw_pages(inputs.generator(4711), w2.num_pages, sum(len(t) for t in w2.tables))
    at = 0
    for t in w2.tables:
        t[:] = perm[at:at + len(t)]
        at += len(t)
    cache = make_cache(w2, fill="random")
    cache.upload(w2.requests, w2.tables, upto=w2.start_pos)
    out2 = run_step(cache, w2)
    assert torch.equal(out2, out)
    cache.close()


def test_prefix_sharing_equals_private_copies():
    import gpu_util as gu
    shared = inputs.prefix_sharing(shared=True)
    private = inputs.prefix_sharing(shared=False)
    assert shared.batch == 128 and shared.notes["shared_pages"] == 128
    assert all(a[:128] == shared.tables[0][:128] for a in shared.tables)       # stored once
    outs = []
    for w in (shared, private):
        cache = make_cache(w)
        # the common prefix is uploaded through the first request only when shared
        if w is shared:
            cache.upload(w.requests[:1], w.tables[:1], upto=[2048])
            for r, t, s in zip(w.requests, w.tables, w.start_pos):
                k, v = r.k[2048:s], r.v[2048:s]
                cache.append(k, v, [s - 2048], [2048], inputs.block_table_array([t]))
        else:
            cache.upload(w.requests, w.tables, upto=w.start_pos)
        outs.append(run_step(cache, w))
        cache.close()
    assert torch.equal(outs[0], outs[1])
    gu.full_parity(shared, outs[0])          # all 4,096 rows


def test_long_context_speculative_equals_token_by_token_decode():
    import gpu_util as gu
    w = inputs.long_context_speculative()
    assert w.geo.n_q_heads == 64 and max(w.seq_lens) > 100_000
    cache = make_cache(w)
    cache.upload(w.requests, w.tables, upto=w.start_pos)
    out = run_step(cache, w)
    gu.full_parity(w, out)                   # every speculative row, contexts up to 131,072 keys
    # token-by-token: the pool already holds every token; decode positions one at a time
    bt = inputs.block_table_array(w.tables)
    scale = w.geo.head_dim ** -0.5
    row0 = rows_of(w)
    for step in range(max(w.q_lens)):
        idx = [r for r in range(w.batch) if step < w.q_lens[r]]
        q = torch.cat([w.requests[r].q_rows(w.start_pos[r] + step, 1) for r in idx])
        one = gu.bf16_bits(cache.attend(q, [1] * len(idx), [w.start_pos[r] + step for r in idx],
                                        [w.seq_lens[r] for r in idx], bt[idx], scale))
        for j, r in enumerate(idx):
            assert torch.equal(one[j], out[row0[r] + step]), (r, step)
    cache.close()


def test_mixed_chunked_prefill_equals_requests_alone_with_chunk_128():
    import gpu_util as gu
    w = inputs.mixed_chunked_prefill()
    n_pre, chunk = w.notes["n_prefill"], w.notes["chunk"]
    assert n_pre == 8 and chunk == 512 and w.batch == 64
    cache = make_cache(w)
    cache.upload(w.requests, w.tables, upto=w.start_pos)
    out = run_step(cache, w)                       # one call: 8 x 512-token chunks + 56 decodes
    gu.sampled_parity(w, out, 512)           # (the full batch is 0.3 TFLOP in fp64: sampled)
    bt = inputs.block_table_array(w.tables)
    scale = w.geo.head_dim ** -0.5
    row0 = rows_of(w)
    for r in range(n_pre):                         # alone, four chunks of 128
        for c0 in range(0, chunk, 128):
            s = w.start_pos[r] + c0
            q = w.requests[r].q_rows(s, 128)
            part = gu.bf16_bits(cache.attend(q, [128], [s], [w.seq_lens[r]], bt[r:r + 1], scale))
            assert torch.equal(part, out[row0[r] + c0:row0[r] + c0 + 128]), (r, c0)
    for r in (n_pre, n_pre + 20, w.batch - 1):     # decodes alone
        q = w.requests[r].q_rows(w.start_pos[r], 1)
        alone = gu.bf16_bits(cache.attend(q, [1], [w.start_pos[r]], [w.seq_lens[r]], bt[r:r + 1], scale))
        assert torch.equal(alone[0], out[row0[r]])
    cache.close()
    # The call above ran its two attention kernels side by side (the decodes' split-parallel kernel in
    # its narrow form beside the chunks' tile kernel); one after the other they give the same bits.
    from paper_2609_38981_b200 import binding as vb
    cache = make_cache(w, flags=vb.VOSTI_FLAG_NO_OVERLAP)
    cache.upload(w.requests, w.tables, upto=w.start_pos)
    assert torch.equal(run_step(cache, w), out)
    cache.close()
