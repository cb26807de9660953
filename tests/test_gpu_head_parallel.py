"""KV-head sharding on one GPU: W ranks as W contexts, each over a pool that holds only its own
KV heads; every rank's output head slice must be, bit for bit, the corresponding heads of the
single-context call (no reduction is split, so nothing may differ), for prefill chunks and for
decode."""
import numpy as np
import pytest
import torch

from paper_2609_38981_b200 import head_parallel as hp
from paper_2609_38981_b200 import inputs

pytestmark = pytest.mark.gpu

GEO = inputs.Geometry(16, 4, 128, 16)
CONTEXTS = (40, 513, 1100)
NUM_PAGES = 256


@pytest.mark.parametrize("world", (2, 4))
def test_head_sharded_ranks_give_the_single_gpu_bits(world):
    import gpu_util as gu
    from paper_2609_38981_b200.harness import DeviceCache, bf16_bits
    scale = GEO.head_dim ** -0.5
    reqs = [inputs.make_request(GEO, 77, i, n) for i, n in enumerate(CONTEXTS)]
    tables = inputs._assign_private_pages(inputs.generator(77), GEO, NUM_PAGES, CONTEXTS)
    bt = inputs.block_table_array(tables)
    calls = [([n - 5 for n in CONTEXTS], [0] * 3), ([5] * 3, [n - 5 for n in CONTEXTS])]   # prefill, then a 5-token step
    full = DeviceCache(GEO, NUM_PAGES, max_batch=4, max_total_q=4096, max_seq_len=2048)
    want = []
    for qls, sts in calls:
        k = torch.cat([r.k[s:s + q] for r, s, q in zip(reqs, sts, qls)])
        v = torch.cat([r.v[s:s + q] for r, s, q in zip(reqs, sts, qls)])
        q = torch.cat([r.q_rows(s, n) for r, s, n in zip(reqs, sts, qls)])
        full.append(k, v, qls, sts, bt)
        want.append(bf16_bits(full.attend(q, qls, sts, [s + n for s, n in zip(sts, qls)], bt, scale)))
    full.close()
    ref = np.concatenate([rows[-5:] for rows in gu.oracle_rows(reqs, scale)])
    got_last = torch.cat([want[1][sum([5] * i):sum([5] * i) + 5] for i in range(3)])
    gu.assert_parity(got_last, ref, "single-context call vs oracle")
    lgeo = hp.local_geometry(GEO, world)
    assert lgeo.group == GEO.group
    for rank in range(world):
        c = DeviceCache(lgeo, NUM_PAGES, max_batch=4, max_total_q=4096, max_seq_len=2048, pool_fill="nan")
        for (qls, sts), w_bits in zip(calls, want):
            k = hp.head_slice(torch.cat([r.k[s:s + q] for r, s, q in zip(reqs, sts, qls)]), rank, world)
            v = hp.head_slice(torch.cat([r.v[s:s + q] for r, s, q in zip(reqs, sts, qls)]), rank, world)
            q = hp.head_slice(torch.cat([r.q_rows(s, n) for r, s, n in zip(reqs, sts, qls)]), rank, world)
            c.append(k, v, qls, sts, bt)
            got = bf16_bits(c.attend(q, qls, sts, [s + n for s, n in zip(sts, qls)], bt, scale))
            hl = lgeo.n_q_heads
            assert torch.equal(got, w_bits[:, rank * hl:(rank + 1) * hl].contiguous()), (world, rank)
        c.close()


def test_gather_heads_with_one_rank_is_the_identity():
    x = torch.randn(7, 4, 64).bfloat16()
    assert hp.gather_heads(x, 1) is x
