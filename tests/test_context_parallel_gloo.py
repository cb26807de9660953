"""The exchange step of context-parallel decode on CPU, as two and three gloo
ranks, through the very function the GPU path uses
(paper_2609_38981_b200.context_parallel.exchange_partials) and the library's own
layout rule (vosti_cp_segments, host-only): every rank fills the partial rows of
the splits it owns (split k on rank k mod W), leaves the rest as poison, and after
the all-gather of owned rows every rank must hold every row bit for bit.  Values
include negative maxima, tiny normalisers and negative zeros."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_38981_b200 import binding as vb
from paper_2609_38981_b200 import context_parallel as cp

GEO = dict(n_q_heads=8, n_kv_heads=2, head_dim=128, page_size=16)
# decode and speculative requests: contexts around split boundaries, an empty request, q_len up to 4
Q_LENS = [1, 4, 1, 0, 2, 1, 3]
STARTS = [0, 508, 511, 0, 1023, 2999, 5000]
SEQS = [s + q for s, q in zip(STARTS, Q_LENS)]


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _cfg():
    return vb.make_config(num_pages=4096, max_batch=16, max_total_q=64, max_seq_len=8192, **GEO)


def full_partials(n_rows, d):
    rng = np.random.default_rng(5)
    u = rng.standard_normal((n_rows, d)).astype(np.float32) * 37.0
    mz = np.stack([rng.standard_normal(n_rows).astype(np.float32) * 20.0 - 30.0,       # maxima, mostly negative
                   np.exp(rng.uniform(-80, 8, size=n_rows)).astype(np.float32)], -1)   # normalisers, some tiny
    u[3, :4] = -0.0
    u[7, 5] = 0.0
    return u, mz


def test_segments_of_all_ranks_partition_the_partial_rows():
    cfg = _cfg()
    G = GEO["n_q_heads"] // GEO["n_kv_heads"]
    want_rows = sum(GEO["n_kv_heads"] * ((s + q - 1) // 512 + 1) * q * G for s, q in zip(STARTS, Q_LENS) if q)
    for world in (1, 2, 3, 5):
        plan = cp.exchange_plan(cfg, Q_LENS, STARTS, SEQS, world)
        assert plan.n_rows == want_rows
        allrows = np.concatenate(plan.rows_of)
        assert len(allrows) == want_rows and np.array_equal(np.sort(allrows), np.arange(want_rows))
        assert plan.pad_rows == max(plan.counts)
    # the owner of a row is its split modulo the world: request 6 (start 5000, 3 tokens) has 10 splits
    seg, _ = vb.vosti_cp_segments(cfg, Q_LENS, STARTS, SEQS, 1, 3)
    base = sum(GEO["n_kv_heads"] * ((s + q - 1) // 512 + 1) * q * G for s, q in zip(STARTS[:6], Q_LENS[:6]) if q)
    rows = 3 * G
    mine = [(base + (h * 10 + k) * rows, rows) for h in range(2) for k in (1, 4, 7)]
    assert [tuple(x) for x in seg if x[0] >= base] == mine


def _rank_main(rank, world, port, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    plan = cp.exchange_plan(_cfg(), Q_LENS, STARTS, SEQS, world)
    d = GEO["head_dim"]
    u_all, mz_all = full_partials(plan.n_rows, d)
    u = torch.full((plan.n_rows, d), float("nan"))
    mz = torch.full((plan.n_rows, 2), float("nan"))
    mine = torch.from_numpy(plan.rows_of[rank])
    u[mine] = torch.from_numpy(u_all)[mine]
    mz[mine] = torch.from_numpy(mz_all)[mine]
    sent = cp.exchange_partials(u, mz, plan, rank)
    ret[rank] = (u.numpy().view(np.uint32).copy(), mz.numpy().view(np.uint32).copy(), sent)
    dist.barrier()
    dist.destroy_process_group()


def _check(world):
    port = _free_port()
    with mp.Manager() as mgr:
        ret = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, ret), nprocs=world, join=True)
        plan = cp.exchange_plan(_cfg(), Q_LENS, STARTS, SEQS, world)
        u, mz = full_partials(plan.n_rows, GEO["head_dim"])
        for rank in range(world):
            got_u, got_mz, sent = ret[rank]
            assert np.array_equal(got_u, u.view(np.uint32)), f"rank {rank}: U partials changed in the exchange"
            assert np.array_equal(got_mz, mz.view(np.uint32)), f"rank {rank}: (m, z) changed in the exchange"
            assert sent == plan.pad_rows * (GEO["head_dim"] + 2) * 4


def test_two_ranks():
    _check(2)


def test_three_ranks():
    _check(3)
