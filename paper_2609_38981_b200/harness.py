"""Device-side plumbing shared by the tests, the smoke check and the benchmark:
allocate the page pool with torch, create a library context, move tensors, and
call the C-ABI entry points through :mod:`binding`.  No attention arithmetic
lives here.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np
import torch

from . import binding as vb
from .inputs import Geometry, RequestContent, block_table_array


def _as_i16(t: torch.Tensor) -> torch.Tensor:
    return t.contiguous().view(torch.int16)


class DeviceCache:
    """A page pool on the GPU plus the library context bound to it."""

    def __init__(self, geo: Geometry, num_pages: int, max_batch: int, max_total_q: int,
                 max_seq_len: int, pool_fill: str = "zeros", flags: int = 0, device="cuda:0",
                 fill_seed: int = 1234):
        self.geo = geo
        self.device = torch.device(device)
        shape = (num_pages, geo.n_kv_heads, 2, geo.page_size, geo.head_dim)
        if pool_fill == "zeros":
            pool = torch.zeros(shape, dtype=torch.bfloat16, device=self.device)
        elif pool_fill == "random":
            g = torch.Generator(device=self.device)
            g.manual_seed(fill_seed)
            pool = torch.empty(shape, dtype=torch.bfloat16, device=self.device)
            pool.normal_(0.0, 3.0, generator=g)
        elif pool_fill == "nan":
            # alternating NaN / +Inf / -Inf bit patterns
            pat = torch.tensor([0x7FC0, 0x7F80, -128, 0x7FFF], dtype=torch.int16, device=self.device)
            n = int(np.prod(shape))
            pool = pat.repeat((n + 3) // 4)[:n].view(torch.bfloat16).reshape(shape).contiguous()
        else:
            raise ValueError(pool_fill)
        if pool.data_ptr() % 1024:  # the library wants the pool 1024-byte aligned; small torch blocks are not
            n = pool.numel()
            raw = torch.empty(n + 512, dtype=torch.bfloat16, device=self.device)
            off = (-raw.data_ptr() % 1024) // 2
            aligned = raw[off:off + n].view(shape)
            aligned.copy_(pool)
            pool = aligned
        self.pool = pool
        self.ctx = vb.vosti_create(geo.n_q_heads, geo.n_kv_heads, geo.head_dim, geo.page_size,
                                   pool, max_batch, max_total_q, max_seq_len, flags=flags)
        self.max_total_q = max_total_q
        self.max_batch = max_batch

    def close(self):
        self.ctx.close()

    # -- the two operations, taking CPU or CUDA bf16 tensors ------------------
    def append(self, k_new: torch.Tensor, v_new: torch.Tensor, q_lens, start_pos, block_tables,
               stream=None) -> None:
        k = k_new.to(self.device).contiguous()
        v = v_new.to(self.device).contiguous()
        vb.vosti_kv_append(self.ctx, k, v, q_lens, start_pos, block_tables, stream=stream)

    def attend(self, q: torch.Tensor, q_lens, start_pos, seq_lens, block_tables, scale: float,
               stream=None) -> torch.Tensor:
        qd = q.to(self.device).contiguous()
        out = torch.empty_like(qd)
        # poison the output so that rows the kernels fail to write are noticed
        _as_i16(out).fill_(0x7FC1)
        vb.vosti_paged_attention(self.ctx, qd, out, q_lens, start_pos, seq_lens, block_tables,
                                 scale, stream=stream)
        return out

    def attend_ex(self, q: torch.Tensor, q_lens, start_pos, seq_lens, block_tables, scale: float,
                  window: int = 0, want_lse: bool = False, stream=None):
        """Attention with a sliding window and / or the log-sum-exp output.
        Returns (out, lse) with lse an fp32 [T, Hq] tensor or None."""
        qd = q.to(self.device).contiguous()
        out = torch.empty_like(qd)
        _as_i16(out).fill_(0x7FC1)
        lse = None
        if want_lse:
            lse = torch.full(qd.shape[:2], float("nan"), dtype=torch.float32, device=self.device)
        vb.vosti_paged_attention_ex(self.ctx, qd, out, lse, q_lens, start_pos, seq_lens, block_tables,
                                    scale, window=window, stream=stream)
        return out, lse

    def upload(self, reqs: Sequence[RequestContent], tables: Sequence[Sequence[int]],
               upto: Optional[Sequence[int]] = None) -> None:
        """Write positions [0, upto_r) of every request into the pool through
        vosti_kv_append, in calls of at most max_total_q tokens."""
        upto = [r.n for r in reqs] if upto is None else list(upto)
        bt = block_table_array(tables)
        pend = [(i, 0) for i in range(len(reqs)) if upto[i] > 0]
        while pend:
            budget, call, nxt = self.max_total_q, [], []
            for i, at in pend:
                if budget == 0 or len(call) == self.max_batch:
                    nxt.append((i, at))
                    continue
                take = min(budget, upto[i] - at)
                call.append((i, at, take))
                budget -= take
                if at + take < upto[i]:
                    nxt.append((i, at + take))
            idx = [i for i, _, _ in call]
            k = torch.cat([reqs[i].k[a:a + t] for i, a, t in call])
            v = torch.cat([reqs[i].v[a:a + t] for i, a, t in call])
            self.append(k, v, [t for _, _, t in call], [a for _, a, _ in call], bt[idx])
            pend = nxt
        torch.cuda.synchronize(self.device)


def bf16_bits(t: torch.Tensor) -> torch.Tensor:
    """bf16 tensor -> int16 CPU tensor of its bits, for exact comparison."""
    return _as_i16(t.detach().cpu())
