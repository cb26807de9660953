"""Context-parallel decode as real ranks: the KV splits of every request are
spread over the ranks of a ``torch.distributed`` process group (split k on rank
k mod W), each rank computes the partial (m, z, U) rows of the splits it owns,
the ranks exchange them, and every rank folds all of them in split order -- the
same partials in the same order as one GPU, hence the same bits.

The exchange is an all-gather of the *owned* rows only (half the volume of an
all-reduce over the whole partial arrays): each rank packs the rows
``vosti_cp_segments`` lists for it into one buffer, padded to the longest
rank's count, ``all_gather_into_tensor`` brings all buffers to all ranks, and
every rank copies the other ranks' rows to their places.  Packing and copying
are index copies (no arithmetic); the collective is NCCL on GPU tensors and
gloo on CPU tensors.  Every kernel of the library reads this GPU's memory only:
no peer pointer is handed to a kernel.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import numpy as np
import torch

from . import binding as vb


@dataclass
class ExchangePlan:
    """Which partial rows each rank owns, for one call's metadata."""
    world: int
    n_rows: int                    # partial rows of the call
    rows_of: List[np.ndarray]      # per rank: ascending int64 row indices
    pad_rows: int                  # rows of one rank's send buffer (the longest rank's count)

    @property
    def counts(self) -> List[int]:
        return [len(r) for r in self.rows_of]


def exchange_plan(cfg, q_lens, start_pos, seq_lens, world: int) -> ExchangePlan:
    """Host-only (no GPU needed): the rows of every rank, from the library's own layout rule."""
    rows_of, n_rows = [], 0
    for rank in range(world):
        seg, n_rows = vb.vosti_cp_segments(cfg, q_lens, start_pos, seq_lens, rank, world)
        if len(seg):
            rows_of.append(np.concatenate([np.arange(a, a + n, dtype=np.int64) for a, n in seg]))
        else:
            rows_of.append(np.zeros(0, dtype=np.int64))
    return ExchangePlan(world, int(n_rows), rows_of, max([len(r) for r in rows_of] + [1]))


def exchange_partials(u: torch.Tensor, mz: torch.Tensor, plan: ExchangePlan, rank: int, group=None) -> int:
    """u: [n_rows, D] fp32, mz: [n_rows, 2] fp32 (views of this rank's partial arrays, its own
    rows filled).  On return every rank's rows are in place on every rank.  Returns the bytes
    this rank sent.  With one rank nothing moves."""
    if plan.world == 1:
        return 0
    import torch.distributed as dist
    D = u.shape[1]
    dev = u.device
    idx = [torch.from_numpy(r).to(dev) for r in plan.rows_of]
    send = torch.zeros(plan.pad_rows, D + 2, dtype=torch.float32, device=dev)
    mine = idx[rank]
    if len(mine):
        send[:len(mine), :D] = u.index_select(0, mine)
        send[:len(mine), D:] = mz.index_select(0, mine)
    recv = torch.empty(plan.world * plan.pad_rows, D + 2, dtype=torch.float32, device=dev)
    dist.all_gather_into_tensor(recv, send, group=group)
    for r in range(plan.world):
        if r == rank or len(idx[r]) == 0:
            continue
        part = recv[r * plan.pad_rows:r * plan.pad_rows + len(idx[r])]
        u.index_copy_(0, idx[r], part[:, :D])
        mz.index_copy_(0, idx[r], part[:, D:])
    return int(send.numel() * 4)


def cp_paged_attention(ctx: vb.Context, q, out, lse, q_lens, start_pos, seq_lens, block_tables,
                       softmax_scale: float, rank: int, world: int, group=None,
                       plan: Optional[ExchangePlan] = None) -> ExchangePlan:
    """One context-parallel attention call on this rank (all ranks call it with the same q and
    lengths; `block_tables` needs valid page ids only for the splits this rank owns).  Runs on
    torch's current stream.  Returns the exchange plan (pass it back in while the metadata
    stays the same to skip its construction)."""
    if plan is None:
        plan = exchange_plan(ctx.cfg, q_lens, start_pos, seq_lens, world)
    u, mz = vb.vosti_cp_partial(ctx, q, q_lens, start_pos, seq_lens, block_tables, softmax_scale, rank, world)
    D = ctx.cfg.head_dim
    exchange_partials(u.view(-1, D), mz.view(-1, 2), plan, rank, group)
    vb.vosti_cp_combine(ctx, out, lse, q_lens, start_pos, seq_lens)
    return plan
