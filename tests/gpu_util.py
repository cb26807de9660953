"""Helpers for the GPU tests: run call schedules through the C-ABI and collect
output rows per (request, position); run the same logical requests through the
CPU oracle."""
from __future__ import annotations

from typing import Dict, List, Sequence, Tuple

import numpy as np
import torch

from paper_2609_38981_b200 import inputs
from paper_2609_38981_b200.harness import DeviceCache, bf16_bits

Call = List[Tuple[int, int, int]]          # (request index, start position, q_len)


def run_schedule(cache: DeviceCache, reqs, tables, schedule: Sequence[Call], scale: float,
                 stride=None, fill=-1, append=True, seq_lens_override=None, window=None,
                 lse_out=None, drop_pages_before_window=False) -> Dict[int, torch.Tensor]:
    """Each call appends its tokens then attends.  Returns, per request, an int16
    tensor [n, Hq, d] with the bf16 bits of every computed row (rows never
    computed stay at a sentinel).

    window: None = the plain entry point; an int = the extended one with that
    sliding window.  lse_out: a dict that receives, per request, an int32 tensor
    [n, Hq] with the fp32 bits of the log-sum-exp.  drop_pages_before_window:
    replace the block-table entries the extended entry point promises not to
    read by -1."""
    geo = cache.geo
    outs = {i: torch.full((r.n, geo.n_q_heads, geo.head_dim), 0x7FC2, dtype=torch.int16)
            for i, r in enumerate(reqs)}
    if lse_out is not None:
        for i, r in enumerate(reqs):
            lse_out.setdefault(i, torch.full((r.n, geo.n_q_heads), 0x7FC00002, dtype=torch.int32))
    for call in schedule:
        idx = [i for i, _, _ in call]
        starts = [s for _, s, _ in call]
        qls = [q for _, _, q in call]
        bt = inputs.block_table_array([tables[i] for i in idx], stride=stride, fill=fill)
        if append:
            k = torch.cat([reqs[i].k[s:s + q] for i, s, q in call])
            v = torch.cat([reqs[i].v[s:s + q] for i, s, q in call])
            cache.append(k, v, qls, starts, bt)
        seq = [s + q for s, q in zip(starts, qls)] if seq_lens_override is None else \
            [seq_lens_override[i] for i in idx]
        qt = torch.cat([reqs[i].q_rows(s, q) for i, s, q in call])
        if window is None and lse_out is None:
            out = bf16_bits(cache.attend(qt, qls, starts, seq, bt, scale))
            lse = None
        else:
            bt_call = bt
            if drop_pages_before_window and window:
                bt_call = bt.copy()
                for row, s in enumerate(starts):
                    bt_call[row, :max(0, s - window + 1) // geo.page_size] = -1
            o, lse = cache.attend_ex(qt, qls, starts, seq, bt_call, scale, window=window or 0,
                                     want_lse=lse_out is not None)
            out = bf16_bits(o)
            if lse is not None:
                lse = lse.cpu().view(torch.int32)
        at = 0
        for i, s, q in call:
            outs[i][s:s + q] = out[at:at + q]
            if lse is not None:
                lse_out[i][s:s + q] = lse[at:at + q]
            at += q
    return outs


def chunked(n: int, chunk: int, start: int = 0) -> List[Tuple[int, int]]:
    return [(s, min(chunk, n - s)) for s in range(start, n, chunk)]


def oracle_rows(reqs, scale):
    """Dense fp64 oracle output for every position of every request."""
    from oracle import oracle
    return [oracle.attention_dense(inputs.bits(r.q), inputs.bits(r.k), inputs.bits(r.v), r.q0, scale)
            for r in reqs]


def widen_bits(t: torch.Tensor) -> np.ndarray:
    return t.view(torch.bfloat16).to(torch.float64).numpy()


def assert_parity(got_bits: torch.Tensor, ref: np.ndarray, what=""):
    """The stated tolerance: max abs error <= 1e-2, mean abs error <= 1e-3."""
    err = np.abs(widen_bits(got_bits) - ref)
    assert np.isfinite(err).all(), f"{what}: non-finite output"
    assert err.max() <= 1e-2, f"{what}: max abs err {err.max():.3e}"
    assert err.mean() <= 1e-3, f"{what}: mean abs err {err.mean():.3e}"
    return float(err.max()), float(err.mean())


def assert_same_bits(a: torch.Tensor, b: torch.Tensor, what=""):
    if not torch.equal(a, b):
        bad = (a != b).reshape(a.shape[0], -1).any(dim=1).nonzero().flatten()
        raise AssertionError(f"{what}: {bad.numel()} of {a.shape[0]} rows differ bitwise, "
                             f"first at positions {bad[:8].tolist()}")


def compact_host_pool(w):
    """The oracle's view of a workload: a host pool holding only the used pages
    (page ids renumbered in order of first use; shared pages stay shared) filled
    from the requests' logical content, and the renumbered block tables."""
    from oracle import oracle
    geo = w.geo
    seen, tables = {}, []
    for tb in w.tables:
        tables.append([seen.setdefault(p, len(seen)) for p in tb])
    pool = np.zeros((len(seen), geo.n_kv_heads, 2, geo.page_size, geo.head_dim), dtype=np.uint16)
    for r, tb in zip(w.requests, tables):
        oracle.kv_append(pool, inputs.bits(r.k), inputs.bits(r.v), [r.n], [0],
                         inputs.block_table_array([tb]))
    return pool, inputs.block_table_array(tables)


def sampled_parity(w, out_bits, n_samples, seed=0, window=0):
    """Compare `n_samples` random (request, token, head) outputs of a workload's
    call against the oracle's paged front-end.  out_bits: int16 [T, Hq, d]."""
    from oracle import oracle
    geo = w.geo
    rng = np.random.default_rng(seed)
    pool, bt = compact_host_pool(w)
    sel = []
    for _ in range(n_samples):
        r = int(rng.integers(0, w.batch))
        sel.append((r, int(rng.integers(0, w.q_lens[r])), int(rng.integers(0, geo.n_q_heads))))
    sel = np.array(sel, dtype=np.int32)
    ref = oracle.paged_attention(inputs.bits(w.packed_q()), pool, w.q_lens, w.start_pos, w.seq_lens,
                                 bt, n_kv_heads=geo.n_kv_heads, page_size=geo.page_size,
                                 scale=geo.head_dim ** -0.5, sel=sel, window=window)
    row0 = np.concatenate([[0], np.cumsum(w.q_lens)])
    got = np.stack([widen_bits(out_bits[row0[r] + i, h]) for r, i, h in sel])
    err = np.abs(got - ref)
    assert np.isfinite(got).all()
    assert err.max() <= 1e-2 and err.mean() <= 1e-3, (err.max(), err.mean())
    return float(err.max()), float(err.mean())


def full_parity(w, out_bits):
    """Every (request, token, head) output of a workload's call against the oracle's paged
    front-end (feasible where the query rows are few: decode and speculative batches)."""
    from oracle import oracle
    geo = w.geo
    pool, bt = compact_host_pool(w)
    ref = oracle.paged_attention(inputs.bits(w.packed_q()), pool, w.q_lens, w.start_pos, w.seq_lens,
                                 bt, n_kv_heads=geo.n_kv_heads, page_size=geo.page_size,
                                 scale=geo.head_dim ** -0.5)
    return assert_parity(out_bits, ref, f"{w.name}: all {out_bits.shape[0] * out_bits.shape[1]} rows vs oracle")


def drifting_request(geo, seed, index, n, step=37, jump=0.5, gain=64.0):
    """A request whose scores climb with the key position: every `step` keys the component of K
    along a fixed direction grows by `jump`, and every query carries `gain` along that direction,
    so the scaled score rises by several units of the lazy reference maximum's step inside one
    split and the reference has to move (alpha != 1, U rescaled) again and again.  Such a softmax
    is sharply peaked -- an output is close to one or two value rows instead of an average of many
    -- so the values are scaled by 1/4 (exact in bf16) to keep outputs in the range the absolute
    tolerance was derived for."""
    r = inputs.make_request(geo, seed, index, n)
    ramp = (torch.arange(n) // step).to(torch.float32) * jump
    k = r.k.to(torch.float32)
    k[:, :, 0] += ramp[:, None]
    q = r.q.to(torch.float32)
    q[:, :, 0] += gain
    v = (r.v.to(torch.float32) * 0.25).to(torch.bfloat16)
    return inputs.RequestContent(n=n, q0=0, k=k.to(torch.bfloat16), v=v, q=q.to(torch.bfloat16))
