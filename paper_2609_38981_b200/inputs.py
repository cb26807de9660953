"""Seeded synthetic inputs shaped like the paper's serving workloads.

This module only draws data and lays out page tables.  It contains none of
the attention arithmetic and is the one module that both the CUDA-path tests
and the CPU oracle's tests may import.

Recipe (every tensor is reproducible from ``(seed, request index)`` alone, so
a request's content never depends on its batch companions):

* values: ``torch.randn`` (CPU generator) in fp32, rounded to bf16;
* lengths: ``torch.randint`` on inclusive ranges;
* page placement: a prefix of ``torch.randperm(num_pages)``.

The five workload recipes mirror the decode-heavy / chunked-prefill /
shared-prefix / long-context speculative serving shapes (Llama-3-8B-like
attention geometry: 32 query heads, 8 KV heads, head_dim 128, page size 16).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np
import torch

BASE_SEED = 38981


@dataclass(frozen=True)
class Geometry:
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    page_size: int = 16

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def page_elems(self) -> int:
        """bf16 elements in one page: [Hkv][K|V][P][d]."""
        return self.n_kv_heads * 2 * self.page_size * self.head_dim

    @property
    def kv_bytes_per_token(self) -> int:
        return self.n_kv_heads * 2 * self.head_dim * 2


LLAMA8B = Geometry(32, 8, 128, 16)
TINY = Geometry(4, 2, 64, 16)
LONGCTX = Geometry(64, 8, 128, 16)


def generator(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    return g


def randn_bf16(gen: torch.Generator, *shape: int) -> torch.Tensor:
    return torch.randn(*shape, generator=gen, dtype=torch.float32).to(torch.bfloat16)


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 CPU tensor -> numpy uint16 view of the same bits."""
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def from_bits(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)


def draw_lengths(gen: torch.Generator, lo: int, hi: int, n: int) -> List[int]:
    """n integers uniform on the inclusive range [lo, hi]."""
    return [int(x) for x in torch.randint(lo, hi + 1, (n,), generator=gen)]


@dataclass
class RequestContent:
    """Logical content of one request: K/V for positions 0..n-1 and query
    vectors for positions q0..n-1."""
    n: int
    q0: int
    k: torch.Tensor  # [n, Hkv, d] bf16
    v: torch.Tensor  # [n, Hkv, d] bf16
    q: torch.Tensor  # [n - q0, Hq, d] bf16

    def q_rows(self, start: int, q_len: int) -> torch.Tensor:
        assert start >= self.q0 and start + q_len <= self.n
        return self.q[start - self.q0:start - self.q0 + q_len]


def make_request(geo: Geometry, seed: int, index: int, n: int, q0: int = 0) -> RequestContent:
    gen = generator(seed * 1000003 + index)
    k = randn_bf16(gen, n, geo.n_kv_heads, geo.head_dim)
    v = randn_bf16(gen, n, geo.n_kv_heads, geo.head_dim)
    q = randn_bf16(gen, n - q0, geo.n_q_heads, geo.head_dim)
    return RequestContent(n=n, q0=q0, k=k, v=v, q=q)


def pages_needed(n: int, page_size: int) -> int:
    return (n + page_size - 1) // page_size


def draw_pages(gen: torch.Generator, num_pages: int, count: int) -> List[int]:
    """`count` distinct page ids, a prefix of a seeded permutation of the pool."""
    assert count <= num_pages
    return [int(x) for x in torch.randperm(num_pages, generator=gen)[:count]]


def block_table_array(tables: Sequence[Sequence[int]], stride: Optional[int] = None,
                      fill: int = -1) -> np.ndarray:
    """Rows of page ids -> int32 [B, stride]; unused trailing entries = fill."""
    width = max([len(t) for t in tables] + [1])
    stride = width if stride is None else stride
    assert stride >= width
    out = np.full((len(tables), stride), fill, dtype=np.int32)
    for r, t in enumerate(tables):
        out[r, :len(t)] = np.asarray(t, dtype=np.int32)
    return out


@dataclass
class Workload:
    """One batch shape: contents, page tables and the call that the benchmark
    times (append q_len new tokens per request, then attend)."""
    name: str
    geo: Geometry
    num_pages: int
    seed: int
    requests: List[RequestContent]
    tables: List[List[int]]            # per request page ids (logical block order)
    q_lens: List[int]
    start_pos: List[int]
    seq_lens: List[int]
    notes: dict = field(default_factory=dict)

    @property
    def batch(self) -> int:
        return len(self.requests)

    @property
    def total_q(self) -> int:
        return int(sum(self.q_lens))

    def kv_bytes(self) -> int:
        """Algorithmic KV bytes one attention call must read: every visible
        (request, kv-head, key token) once = 2*d*2 bytes each.  For request r
        the keys 0 .. start+q_len-1 are visible to at least one row."""
        tok = sum(s + q for s, q in zip(self.start_pos, self.q_lens) if q > 0)
        return tok * self.geo.kv_bytes_per_token

    def packed_q(self) -> torch.Tensor:
        return torch.cat([r.q_rows(s, q) for r, s, q in
                          zip(self.requests, self.start_pos, self.q_lens)], dim=0)

    def packed_new_kv(self):
        k = torch.cat([r.k[s:s + q] for r, s, q in
                       zip(self.requests, self.start_pos, self.q_lens)], dim=0)
        v = torch.cat([r.v[s:s + q] for r, s, q in
                       zip(self.requests, self.start_pos, self.q_lens)], dim=0)
        return k, v


def _assign_private_pages(gen, geo, num_pages, lengths):
    need = [pages_needed(n, geo.page_size) for n in lengths]
    ids = draw_pages(gen, num_pages, sum(need))
    tables, at = [], 0
    for c in need:
        tables.append(ids[at:at + c])
        at += c
    return tables


def decode_heavy(batch: int = 64, lo: int = 512, hi: int = 4096, num_pages: int = 200_000,
                 geo: Geometry = LLAMA8B, seed: int = BASE_SEED * 10 + 2) -> Workload:
    """Decode-heavy batch: one query token per request, contexts uniform in
    [lo, hi], pages scattered at random over a large pool."""
    gen = generator(seed)
    ctx = draw_lengths(gen, lo, hi, batch)
    reqs = [make_request(geo, seed, i, n, q0=n - 1) for i, n in enumerate(ctx)]
    tables = _assign_private_pages(gen, geo, num_pages, ctx)
    return Workload("decode_heavy", geo, num_pages, seed, reqs, tables,
                    q_lens=[1] * batch, start_pos=[n - 1 for n in ctx], seq_lens=list(ctx))


def mixed_chunked_prefill(n_prefill: int = 8, chunk: int = 512, prior_hi: int = 8192,
                          n_decode: int = 56, dec_lo: int = 1024, dec_hi: int = 4096,
                          num_pages: int = 200_000, geo: Geometry = LLAMA8B,
                          seed: int = BASE_SEED * 10 + 3) -> Workload:
    """Chunked-prefill requests (a `chunk`-token chunk after a prior context
    uniform in [0, prior_hi]) co-batched with single-token decodes."""
    gen = generator(seed)
    prior = draw_lengths(gen, 0, prior_hi, n_prefill)
    dctx = draw_lengths(gen, dec_lo, dec_hi, n_decode)
    reqs, q_lens, start = [], [], []
    for i, pr in enumerate(prior):
        reqs.append(make_request(geo, seed, i, pr + chunk, q0=pr))
        q_lens.append(chunk)
        start.append(pr)
    for i, n in enumerate(dctx):
        reqs.append(make_request(geo, seed, n_prefill + i, n, q0=n - 1))
        q_lens.append(1)
        start.append(n - 1)
    lengths = [r.n for r in reqs]
    tables = _assign_private_pages(gen, geo, num_pages, lengths)
    return Workload("mixed_chunked_prefill", geo, num_pages, seed, reqs, tables, q_lens, start,
                    list(lengths), notes={"n_prefill": n_prefill, "chunk": chunk})


def prefix_sharing(batch: int = 128, prefix: int = 2048, suf_lo: int = 64, suf_hi: int = 512,
                   num_pages: int = 200_000, geo: Geometry = LLAMA8B,
                   seed: int = BASE_SEED * 10 + 4, shared: bool = True) -> Workload:
    """`batch` requests with one common `prefix`-token prefix, a private
    suffix and one decode token.  shared=True stores the whole pages of the
    prefix once; shared=False gives every request private copies.  Pages are
    shared whole: a prefix that ends inside a page has that page private."""
    gen = generator(seed)
    suf = draw_lengths(gen, suf_lo, suf_hi, batch)
    common = make_request(geo, seed, 10_000_019, prefix, q0=prefix)
    reqs = []
    for i, s in enumerate(suf):
        own = make_request(geo, seed, i, s + 1, q0=s)
        reqs.append(RequestContent(
            n=prefix + s + 1, q0=prefix + s,
            k=torch.cat([common.k, own.k]), v=torch.cat([common.v, own.v]), q=own.q))
    P = geo.page_size
    full = prefix // P
    lengths = [r.n for r in reqs]
    if shared:
        need = [pages_needed(n, P) - full for n in lengths]
        ids = draw_pages(gen, num_pages, full + sum(need))
        shared_ids, at, tables = ids[:full], full, []
        for c in need:
            tables.append(shared_ids + ids[at:at + c])
            at += c
    else:
        tables = _assign_private_pages(gen, geo, num_pages, lengths)
    return Workload("prefix_sharing" if shared else "prefix_private", geo, num_pages, seed, reqs,
                    tables, q_lens=[1] * batch, start_pos=[n - 1 for n in lengths],
                    seq_lens=list(lengths), notes={"prefix": prefix, "shared_pages": full})


def long_context_speculative(batch: int = 8, lo: int = 32768, hi: int = 131072,
                             q_hi: int = 4, num_pages: int = 60_000, geo: Geometry = LONGCTX,
                             seed: int = BASE_SEED * 10 + 5) -> Workload:
    """Long contexts with 1..q_hi query tokens per request (draft-token
    verification)."""
    gen = generator(seed)
    ctx = draw_lengths(gen, lo, hi, batch)
    ql = draw_lengths(gen, 1, q_hi, batch)
    reqs = [make_request(geo, seed, i, n, q0=n - q) for i, (n, q) in enumerate(zip(ctx, ql))]
    tables = _assign_private_pages(gen, geo, num_pages, ctx)
    return Workload("long_context_speculative", geo, num_pages, seed, reqs, tables, q_lens=ql,
                    start_pos=[n - q for n, q in zip(ctx, ql)], seq_lens=list(ctx))


def tiny_requests(geo: Geometry = TINY, contexts: Sequence[int] = (37, 100, 250),
                  seed: int = BASE_SEED * 10 + 1) -> List[RequestContent]:
    """Contents of the tiny invariance case (query vectors at every position)."""
    return [make_request(geo, seed, i, n, q0=0) for i, n in enumerate(contexts)]
