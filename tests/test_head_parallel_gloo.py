"""The exchange of KV-head sharding on CPU as two and four gloo ranks: the all-gather of output
head slices must assemble the single-GPU layout [T, Hq, d] (heads in rank order) on every rank."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_38981_b200 import head_parallel as hp

T, HQ, D = 11, 8, 16


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def full_output():
    return (torch.arange(T * HQ * D, dtype=torch.float32).reshape(T, HQ, D) * 0.25 - 100.0).to(torch.bfloat16)


def _rank_main(rank, world, port, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = hp.head_slice(full_output(), rank, world)
    got = hp.gather_heads(mine, world)
    ret[rank] = bool(torch.equal(got.view(torch.int16), full_output().view(torch.int16)))
    dist.barrier()
    dist.destroy_process_group()


def _check(world):
    port = _free_port()
    with mp.Manager() as mgr:
        ret = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, ret), nprocs=world, join=True)
        assert all(ret[r] for r in range(world))


def test_two_ranks():
    _check(2)


def test_four_ranks():
    _check(4)
