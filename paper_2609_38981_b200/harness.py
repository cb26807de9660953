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


GUARD_BYTES = 16384
GUARD_BYTE = 0xA5


class Guarded:
    """A device buffer with a poisoned guard region before and after it (the stand-in for a
    memory checker: a kernel that writes outside what it was given changes a guard)."""

    def __init__(self, nbytes: int, device, align: int = 1024, what: str = "buffer"):
        self.what = what
        self.raw = torch.empty(nbytes + 2 * GUARD_BYTES + align, dtype=torch.uint8, device=device)
        self.off = GUARD_BYTES + (-(self.raw.data_ptr() + GUARD_BYTES)) % align
        self.nbytes = nbytes
        self.raw[:self.off] = GUARD_BYTE
        self.raw[self.off + nbytes:] = GUARD_BYTE

    @property
    def payload(self) -> torch.Tensor:
        return self.raw[self.off:self.off + self.nbytes]

    def check(self) -> None:
        before, after = self.raw[:self.off], self.raw[self.off + self.nbytes:]
        ok = bool((before == GUARD_BYTE).all()) and bool((after == GUARD_BYTE).all())
        if not ok:
            bad = (before != GUARD_BYTE).nonzero().flatten()
            where = f"{self.off - int(bad[-1])} bytes before it" if bad.numel() else \
                f"{int((after != GUARD_BYTE).nonzero().flatten()[0])} bytes after it"
            raise AssertionError(f"guard region of the {self.what} overwritten ({where})")


class DeviceCache:
    """A page pool on the GPU plus the library context bound to it."""

    def __init__(self, geo: Geometry, num_pages: int, max_batch: int, max_total_q: int,
                 max_seq_len: int, pool_fill: str = "zeros", flags: int = 0, device="cuda:0",
                 fill_seed: int = 1234):
        self.geo = geo
        self.device = torch.device(device)
        shape = (num_pages, geo.n_kv_heads, 2, geo.page_size, geo.head_dim)
        n = int(np.prod(shape))
        # pool and workspace sit between guard regions (the library wants both 1024-byte aligned)
        self._pool_guard = Guarded(2 * n, self.device, what="page pool")
        pool = self._pool_guard.payload.view(torch.bfloat16).view(shape)
        if pool_fill == "zeros":
            pool.zero_()
        elif pool_fill == "random":
            g = torch.Generator(device=self.device)
            g.manual_seed(fill_seed)
            pool.normal_(0.0, 3.0, generator=g)
        elif pool_fill == "nan":
            # alternating NaN / +Inf / -Inf bit patterns
            pat = torch.tensor([0x7FC0, 0x7F80, -128, 0x7FFF], dtype=torch.int16, device=self.device)
            pool.view(torch.int16).view(-1).copy_(pat.repeat((n + 3) // 4)[:n])
        else:
            raise ValueError(pool_fill)
        self.pool = pool
        cfg = vb.make_config(geo.n_q_heads, geo.n_kv_heads, geo.head_dim, geo.page_size, num_pages, max_batch,
                             max_total_q, max_seq_len, flags=flags)
        self._ws_guard = Guarded(vb.vosti_workspace_bytes(cfg), self.device, what="workspace")
        self.ctx = vb.vosti_create(geo.n_q_heads, geo.n_kv_heads, geo.head_dim, geo.page_size,
                                   pool, max_batch, max_total_q, max_seq_len, flags=flags,
                                   workspace=self._ws_guard.payload)
        self.max_total_q = max_total_q
        self.max_batch = max_batch

    def check_guards(self) -> None:
        """Raises if anything wrote before or after the pool or the workspace."""
        self._pool_guard.check()
        self._ws_guard.check()

    def close(self):
        if getattr(self.ctx, "handle", None):
            torch.cuda.synchronize(self.device)
            self.check_guards()
        self.ctx.close()

    def _guarded_io(self, q: torch.Tensor):
        """Q and O of one call, each between guard regions; O poisoned so that rows the kernels
        fail to write are noticed."""
        nbytes = q.numel() * q.element_size()
        gq = Guarded(nbytes, self.device, align=256, what="query rows")
        go = Guarded(nbytes, self.device, align=256, what="output rows")
        qd = gq.payload.view(torch.bfloat16).view(q.shape)
        qd.copy_(q)
        out = go.payload.view(torch.bfloat16).view(q.shape)
        _as_i16(out).fill_(0x7FC1)
        return gq, go, qd, out

    def _check_call(self, gq: "Guarded", go: "Guarded") -> None:
        torch.cuda.synchronize(self.device)
        gq.check()
        go.check()
        self.check_guards()

    # -- the two operations, taking CPU or CUDA bf16 tensors ------------------
    def append(self, k_new: torch.Tensor, v_new: torch.Tensor, q_lens, start_pos, block_tables,
               stream=None) -> None:
        k = k_new.to(self.device).contiguous()
        v = v_new.to(self.device).contiguous()
        vb.vosti_kv_append(self.ctx, k, v, q_lens, start_pos, block_tables, stream=stream)

    def attend(self, q: torch.Tensor, q_lens, start_pos, seq_lens, block_tables, scale: float,
               stream=None) -> torch.Tensor:
        gq, go, qd, out = self._guarded_io(q)
        vb.vosti_paged_attention(self.ctx, qd, out, q_lens, start_pos, seq_lens, block_tables,
                                 scale, stream=stream)
        self._check_call(gq, go)
        return out

    def attend_ex(self, q: torch.Tensor, q_lens, start_pos, seq_lens, block_tables, scale: float,
                  window: int = 0, want_lse: bool = False, stream=None):
        """Attention with a sliding window and / or the log-sum-exp output.
        Returns (out, lse) with lse an fp32 [T, Hq] tensor or None."""
        gq, go, qd, out = self._guarded_io(q)
        lse = None
        if want_lse:
            lse = torch.full(qd.shape[:2], float("nan"), dtype=torch.float32, device=self.device)
        vb.vosti_paged_attention_ex(self.ctx, qd, out, lse, q_lens, start_pos, seq_lens, block_tables,
                                    scale, window=window, stream=stream)
        self._check_call(gq, go)
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
