"""Context-parallel decode (vosti_cp_partial / vosti_cp_combine) on one GPU: the
ranks are separate contexts with separate pools, run one after the other; each
pool holds only the pages of the splits its rank owns (split k on rank k mod W),
everything else is non-finite garbage behind block-table entries of -1.  The
exchange is emulated with the exchange plan the real ranks use
(context_parallel.exchange_plan: every rank's owned rows are copied to every
other rank's arrays, as the all-gather does), and, as a second route, with the
elementwise sum an all-reduce would compute.  Outputs and log-sum-exp must be
bitwise those of the single-GPU call, which is itself checked against the fp64
oracle."""
import numpy as np
import pytest
import torch

from paper_2609_38981_b200 import binding as vb
from paper_2609_38981_b200 import context_parallel as cp
from paper_2609_38981_b200 import inputs

pytestmark = pytest.mark.gpu

GEOS = {"d128_g4": inputs.Geometry(8, 2, 128, 16), "d64_g2": inputs.TINY, "d128_g8": inputs.Geometry(8, 1, 128, 16)}
CONTEXTS = (1, 300, 512, 513, 1500, 2300, 4000)
NUM_PAGES = 1024


def owned_only(tables, rank, world):
    """The block tables a rank would hold: -1 for pages of splits it does not own."""
    out = []
    for tb in tables:
        out.append([pg if (b // 32) % world == rank else -1 for b, pg in enumerate(tb)])
    return out


@pytest.mark.parametrize("geo_name", list(GEOS))
@pytest.mark.parametrize("world", (1, 2, 3, 4))
@pytest.mark.parametrize("q_len", (1, 4))
def test_context_parallel_equals_single_gpu(geo_name, world, q_len):
    from paper_2609_38981_b200.harness import DeviceCache, bf16_bits
    geo = GEOS[geo_name]
    if q_len * geo.group > 32:
        pytest.skip("not a split-parallel request in this geometry")
    scale = geo.head_dim ** -0.5
    reqs = [inputs.make_request(geo, 2024, i, n + q_len - 1) for i, n in enumerate(CONTEXTS)]
    tables = inputs._assign_private_pages(inputs.generator(2024), geo, NUM_PAGES, [r.n for r in reqs])
    qls = [q_len] * len(reqs)
    starts = [r.n - q_len for r in reqs]
    seqs = [r.n for r in reqs]
    q = torch.cat([r.q_rows(s, q_len) for r, s in zip(reqs, starts)])
    # single GPU
    ref = DeviceCache(geo, NUM_PAGES, max_batch=8, max_total_q=4096, max_seq_len=4200)
    ref.upload(reqs, tables)
    want, want_lse = ref.attend_ex(q, qls, starts, seqs, inputs.block_table_array(tables), scale, want_lse=True)
    want, want_lse = bf16_bits(want), want_lse.cpu().view(torch.int32)
    import gpu_util as gu
    ref64 = np.concatenate([rows[s:s + q_len] for rows, s in zip(gu.oracle_rows(reqs, scale), starts)])
    gu.assert_parity(want, ref64, "single-GPU call vs oracle")
    full_pool = ref.pool.clone()
    plan = cp.exchange_plan(ref.ctx.cfg, qls, starts, seqs, world)
    ref.close()
    # W ranks, one after the other
    ranks, sums = [], None
    for rank in range(world):
        c = DeviceCache(geo, NUM_PAGES, max_batch=8, max_total_q=4096, max_seq_len=4200, pool_fill="nan")
        mine = owned_only(tables, rank, world)
        for tb in mine:                       # copy the owned pages' content from the full pool
            ids = torch.tensor([p for p in tb if p >= 0], dtype=torch.long, device=c.pool.device)
            if len(ids):
                c.pool[ids] = full_pool[ids]
        u, mz = vb.vosti_cp_partial(c.ctx, q.to(c.device).contiguous(), qls, starts, seqs,
                                    inputs.block_table_array(mine, fill=-1), scale, rank, world)
        torch.cuda.synchronize()
        sums = (u.clone(), mz.clone()) if sums is None else (sums[0] + u, sums[1] + mz)
        ranks.append((c, u, mz))
    # route 1, the all-gather of owned rows: rank r's rows, as the exchange plan lists them, are
    # copied into every other rank's arrays (the rest of those arrays is poisoned first, so a row
    # the plan forgot would show); every rank folds and must give the single-GPU bits
    D = geo.head_dim
    own = [(u.view(-1, D).clone(), mz.view(-1, 2).clone()) for _, u, mz in ranks]
    assert plan.n_rows == own[0][0].shape[0]
    for me, (c, u, mz) in enumerate(ranks):
        u.fill_(float("nan"))
        mz.fill_(float("nan"))
        for r in range(world):
            idx = torch.from_numpy(plan.rows_of[r]).to(c.device)
            u.view(-1, D).index_copy_(0, idx, own[r][0].index_select(0, idx))
            mz.view(-1, 2).index_copy_(0, idx, own[r][1].index_select(0, idx))
        out = torch.empty_like(q, device=c.device)
        lse = torch.empty(q.shape[:2], dtype=torch.float32, device=c.device)
        vb.vosti_cp_combine(c.ctx, out, lse, qls, starts, seqs)
        assert torch.equal(bf16_bits(out), want), (geo_name, world, q_len, "all-gather", me)
        assert torch.equal(lse.cpu().view(torch.int32), want_lse)
    # route 2, the all-reduce: every rank receives the elementwise sum and folds
    for c, u, mz in ranks:
        u.copy_(sums[0])
        mz.copy_(sums[1])
        out = torch.empty_like(q, device=c.device)
        lse = torch.empty(q.shape[:2], dtype=torch.float32, device=c.device)
        vb.vosti_cp_combine(c.ctx, out, lse, qls, starts, seqs)
        assert torch.equal(bf16_bits(out), want), (geo_name, world, q_len)
        assert torch.equal(lse.cpu().view(torch.int32), want_lse)
        c.close()


def test_rank_level_call_with_one_rank_equals_the_plain_call():
    """cp_paged_attention, the function real ranks call, with a world of one (no process group)."""
    from paper_2609_38981_b200.harness import DeviceCache, bf16_bits
    geo = GEOS["d128_g4"]
    scale = geo.head_dim ** -0.5
    reqs = [inputs.make_request(geo, 2025, i, n) for i, n in enumerate(CONTEXTS)]
    tables = inputs._assign_private_pages(inputs.generator(2025), geo, NUM_PAGES, [r.n for r in reqs])
    qls, starts, seqs = [1] * len(reqs), [r.n - 1 for r in reqs], [r.n for r in reqs]
    q = torch.cat([r.q_rows(s, 1) for r, s in zip(reqs, starts)])
    c = DeviceCache(geo, NUM_PAGES, max_batch=8, max_total_q=4096, max_seq_len=4200)
    c.upload(reqs, tables)
    bt = inputs.block_table_array(tables)
    want = bf16_bits(c.attend(q, qls, starts, seqs, bt, scale))
    qd = q.to(c.device).contiguous()
    out = torch.empty_like(qd)
    cp.cp_paged_attention(c.ctx, qd, out, None, qls, starts, seqs, bt, scale, rank=0, world=1)
    assert torch.equal(bf16_bits(out), want)
    c.close()


def test_prefill_chunks_are_refused():
    from paper_2609_38981_b200.harness import DeviceCache
    geo = GEOS["d128_g4"]
    c = DeviceCache(geo, 64, max_batch=4, max_total_q=256, max_seq_len=512)
    r = inputs.make_request(geo, 1, 0, 100)
    bt = inputs.block_table_array([list(range(7))])
    with pytest.raises(vb.VostiError) as e:
        vb.vosti_cp_partial(c.ctx, r.q_rows(0, 100).to(c.device).contiguous(), [100], [0], [100], bt,
                            0.1, 0, 2)
    assert e.value.status == vb.VOSTI_ERR_UNSUPPORTED_CONFIG
    with pytest.raises(vb.VostiError):
        vb.vosti_cp_partial(c.ctx, r.q_rows(99, 1).to(c.device).contiguous(), [1], [99], [100], bt, 0.1, 2, 2)
    c.close()
