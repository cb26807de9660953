"""KV-head sharding (the tensor-parallel layout of serving engines): rank g of W holds the pool
slices and the query heads of KV heads [g Hkv / W, (g + 1) Hkv / W).  The independent unit of the
attention op is (request, KV head) and no arithmetic crosses it, so every rank runs the ordinary
entry points on its own heads with a context of Hq / W query and Hkv / W KV heads, the output
bits of a head are those of the single-GPU call, and the only exchange is an all-gather of the
output head slices (or none, when a row-parallel projection follows).  Every kernel reads this
GPU's memory only.
"""
from __future__ import annotations

from typing import Optional

import torch

from . import binding as vb
from .inputs import Geometry


def local_geometry(geo: Geometry, world: int) -> Geometry:
    """The geometry one rank sees: the group size (query heads per KV head) is unchanged."""
    if geo.n_kv_heads % world:
        raise ValueError(f"{geo.n_kv_heads} KV heads do not divide over {world} ranks")
    return Geometry(geo.n_q_heads // world, geo.n_kv_heads // world, geo.head_dim, geo.page_size)


def head_slice(t: torch.Tensor, rank: int, world: int, dim: int = 1) -> torch.Tensor:
    """The heads of rank `rank` of a [rows, heads, d] tensor (query or new K/V rows), contiguous."""
    n = t.shape[dim] // world
    return t.narrow(dim, rank * n, n).contiguous()


def gather_heads(out_local: torch.Tensor, world: int, group=None) -> torch.Tensor:
    """All-gather of the output head slices: [T, Hq / W, d] on every rank -> [T, Hq, d] on every
    rank (heads in rank order, as the single-GPU layout has them).  NCCL on GPU tensors, gloo on CPU."""
    if world == 1:
        return out_local
    import torch.distributed as dist
    T, hl, d = out_local.shape
    flat = torch.empty(world * T, hl, d, dtype=out_local.dtype, device=out_local.device)
    dist.all_gather_into_tensor(flat, out_local.contiguous(), group=group)
    return flat.view(world, T, hl, d).permute(1, 0, 2, 3).reshape(T, world * hl, d).contiguous()


def head_parallel_attention(ctx: vb.Context, q_local, out_local, q_lens, start_pos, seq_lens, block_tables,
                            softmax_scale: float, world: int, group=None, gather: bool = True) -> Optional[torch.Tensor]:
    """One attention call on this rank's heads (ctx was created with the local geometry over the
    rank's pool slice).  Returns the gathered [T, Hq, d] output, or None with gather=False."""
    vb.vosti_paged_attention(ctx, q_local, out_local, q_lens, start_pos, seq_lens, block_tables, softmax_scale)
    return gather_heads(out_local, world, group) if gather else None
