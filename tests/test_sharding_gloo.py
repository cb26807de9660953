"""The N > 1 path on CPU: ranks take their own seeded batch (no data-path
collective), and the only exchange is the max / sum of scalars after the timed
region, through the function bench.py uses for it.  Run as two gloo ranks."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_38981_b200 import inputs


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    w = bench.make_workload("decode_heavy", rank, pool_pages=12000)
    # every rank owns a different batch of the same shape (weak scaling)
    sig = torch.tensor([float(sum(w.seq_lens)), float(w.kv_bytes()), float(w.total_q)], dtype=torch.float64)
    gathered = [torch.zeros_like(sig) for _ in range(world)]
    dist.all_gather(gathered, sig)
    # the reductions bench.py itself runs after its timed region (same function, gloo instead of NCCL)
    elapsed = bench.reduce_over_ranks(dist, [1.0 + rank, 2.0 + rank], "max")      # stand-in timings
    total = bench.reduce_over_ranks(dist, sig[1:].tolist(), "sum")
    if rank == 0:
        ret["gathered"] = [g.tolist() for g in gathered]
        ret["elapsed"] = elapsed
        ret["total"] = total
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_take_disjoint_batches_and_reduce_scalars():
    world = 2
    port = _free_port()
    with mp.Manager() as mgr:
        ret = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, ret), nprocs=world, join=True)
        g = ret["gathered"]
        assert g[0] != g[1], "ranks must draw different batches"
        assert all(x[2] == 64 for x in g)                      # same shape: 64 query tokens each
        assert ret["elapsed"] == [2.0, 3.0]                    # max over ranks
        assert ret["total"] == [g[0][1] + g[1][1], 128.0]      # bytes and tokens summed over ranks
