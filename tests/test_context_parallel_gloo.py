"""The exchange step of context-parallel decode on CPU, as two and three gloo
ranks: every rank holds the partial (m, z, U) slabs of the splits it owns
(split k on rank k mod W) and zeros elsewhere; an all-reduce (sum, fp32) must
hand every rank the union of the slabs bit for bit -- the property the
single-GPU equality of the fold rests on.  Values include negative maxima,
denormal-sized normalisers and negative zeros (whose sign may turn positive:
the attention output rule adds +0 for exactly that reason)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


N_SPLITS, ROWS, D = 11, 6, 16


def full_partials():
    rng = np.random.default_rng(5)
    u = rng.standard_normal((N_SPLITS, ROWS, D)).astype(np.float32) * 37.0
    mz = np.stack([rng.standard_normal((N_SPLITS, ROWS)).astype(np.float32) * 20.0 - 30.0,       # maxima, mostly negative
                   np.exp(rng.uniform(-80, 8, size=(N_SPLITS, ROWS))).astype(np.float32)], -1)  # normalisers, some tiny
    u[3, 2, :4] = -0.0
    u[7, 0, 5] = 0.0
    return u, mz


def _rank_main(rank, world, port, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    u, mz = full_partials()
    mine = np.array([k % world == rank for k in range(N_SPLITS)])
    tu = torch.from_numpy(np.where(mine[:, None, None], u, np.float32(0.0)).copy())
    tmz = torch.from_numpy(np.where(mine[:, None, None], mz, np.float32(0.0)).copy())
    dist.all_reduce(tu, op=dist.ReduceOp.SUM)
    dist.all_reduce(tmz, op=dist.ReduceOp.SUM)
    ret[rank] = (tu.numpy().view(np.uint32).copy(), tmz.numpy().view(np.uint32).copy())
    dist.barrier()
    dist.destroy_process_group()


def _check(world):
    port = _free_port()
    with mp.Manager() as mgr:
        ret = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, ret), nprocs=world, join=True)
        u, mz = full_partials()
        want_u, want_mz = (u + np.float32(0.0)).view(np.uint32), mz.view(np.uint32)   # -0 may have become +0
        for rank in range(world):
            got_u, got_mz = ret[rank]
            assert np.array_equal(got_u, want_u), f"rank {rank}: U partials changed in the exchange"
            assert np.array_equal(got_mz, want_mz), f"rank {rank}: (m, z) changed in the exchange"
        # everything except the sign of zeros is the original bit pattern
        assert np.array_equal(want_u[u != 0], u.view(np.uint32)[u != 0])


def test_two_ranks():
    _check(2)


def test_three_ranks():
    _check(3)
