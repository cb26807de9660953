"""The prefix-cache manager driving the attention op (the paper's KV-cache
figure, end to end on the GPU): a request that reuses cached prefix pages and
prefills only its suffix gets, bit for bit, the outputs of a cold run; shared
pages are never written again; eviction and recomputation re-establish the
same values in other physical pages."""
import numpy as np
import pytest
import torch

from paper_2609_38981_b200 import inputs

pytestmark = pytest.mark.gpu

GEO = inputs.Geometry(8, 2, 128, 16)
VOCAB, MAXLEN = 64, 512


def model(seed=4321):
    """Stand-in for the layers below attention: Q, K, V rows as a fixed function of
    (token, position), so that equal causal prefixes give equal KV values."""
    g = inputs.generator(seed)
    tabs = {}
    for name, heads in (("q", GEO.n_q_heads), ("k", GEO.n_kv_heads), ("v", GEO.n_kv_heads)):
        tabs[name] = (torch.randn(VOCAB, heads, GEO.head_dim, generator=g),
                      torch.randn(MAXLEN, heads, GEO.head_dim, generator=g))

    def rows(name, tokens, start):
        tok, pos = tabs[name]
        t = torch.as_tensor(tokens, dtype=torch.long)
        p = torch.arange(start, start + len(tokens))
        return (tok[t] + 0.5 * pos[p]).to(torch.bfloat16)
    return rows


class Engine:
    """A minimal serving loop: the manager decides pages, the library moves KV and attends."""

    def __init__(self, num_pages):
        from paper_2609_38981_b200.harness import DeviceCache
        from paper_2609_38981_b200.cache import PrefixCache
        self.dev = DeviceCache(GEO, num_pages, max_batch=8, max_total_q=1024, max_seq_len=MAXLEN, pool_fill="nan")
        self.mgr = PrefixCache(num_pages, GEO.page_size)
        self.rows = model()
        self.tokens = {}
        self.done = {}

    def admit(self, rid, tokens):
        cached = self.mgr.admit(rid, tokens)
        self.tokens[rid], self.done[rid] = list(tokens), cached
        return cached

    def step(self, work):
        """work: {request: number of new positions}.  One engine step: append + attend, then
        report and cross the step boundary.  Returns {request: (start, int16 output bits)}."""
        from paper_2609_38981_b200.harness import bf16_bits
        ids = list(work)
        starts = [self.done[r] for r in ids]
        qls = [work[r] for r in ids]
        tables = [self.mgr.block_table(r) for r in ids]
        bt = inputs.block_table_array(tables)
        k = torch.cat([self.rows("k", self.tokens[r][s:s + n], s) for r, s, n in zip(ids, starts, qls)])
        v = torch.cat([self.rows("v", self.tokens[r][s:s + n], s) for r, s, n in zip(ids, starts, qls)])
        q = torch.cat([self.rows("q", self.tokens[r][s:s + n], s) for r, s, n in zip(ids, starts, qls)])
        self.dev.append(k, v, qls, starts, bt)
        out = bf16_bits(self.dev.attend(q, qls, starts, [s + n for s, n in zip(starts, qls)], bt,
                                        GEO.head_dim ** -0.5))
        res, at = {}, 0
        for r, s, n in zip(ids, starts, qls):
            res[r] = (s, out[at:at + n])
            at += n
            self.done[r] = s + n
            self.mgr.computed(r, s + n)
        self.mgr.step_boundary()
        assert self.mgr.check() == ""
        return res

    def run_to_end(self, rid, chunk):
        outs = {}
        while self.done[rid] < len(self.tokens[rid]):
            n = min(chunk, len(self.tokens[rid]) - self.done[rid])
            s, o = self.step({rid: n})[rid]
            for i in range(n):
                outs[s + i] = o[i]
        return outs

    def finish(self, rid):
        self.mgr.finish(rid)
        del self.tokens[rid], self.done[rid]

    def close(self):
        self.dev.close()
        self.mgr.close()


def cold(tokens, chunk=64):
    e = Engine(64)
    e.admit(0, tokens)
    outs = e.run_to_end(0, chunk)
    e.close()
    return outs


def same(a, b, positions, what):
    for p in positions:
        assert torch.equal(a[p], b[p]), f"{what}: position {p} differs bitwise"


def test_reuse_equals_cold_and_shared_pages_are_not_rewritten():
    rng = np.random.default_rng(7)
    stem = rng.integers(0, VOCAB, size=150).tolist()
    A = stem
    B = stem[:100] + rng.integers(0, VOCAB, size=70).tolist()
    cold_a, cold_b = cold(A), cold(B)
    # the cold run everything else is compared with is within the stated tolerance of the fp64 oracle
    import gpu_util as gu
    from oracle import oracle
    rows = model()
    ref = oracle.attention_dense(inputs.bits(rows("q", A, 0)), inputs.bits(rows("k", A, 0)),
                                 inputs.bits(rows("v", A, 0)), 0, GEO.head_dim ** -0.5)
    gu.assert_parity(torch.stack([cold_a[p] for p in range(len(A))]), ref, "cold run vs oracle")
    e = Engine(64)
    assert e.admit(1, A) == 0
    out_a = e.run_to_end(1, 64)
    same(out_a, cold_a, range(150), "A in the shared engine")
    # B shares 100 tokens with A: six whole pages are hits, it prefills from position 96
    assert e.admit(2, B) == 96
    shared = e.mgr.block_table(2)[:6]
    assert shared == e.mgr.block_table(1)[:6]
    snapshot = e.dev.pool[shared].clone()
    out_b = e.run_to_end(2, 50)
    assert sorted(out_b) == list(range(96, 170))
    same(out_b, cold_b, range(96, 170), "B after reuse")
    assert torch.equal(e.dev.pool[shared].view(torch.int16), snapshot.view(torch.int16))  # immutable
    # decode both together, one token each, and compare with cold decode of the same histories
    nxt = {1: 17, 2: 23}
    for r, t in nxt.items():
        e.mgr.append(r, [t])
        e.tokens[r].append(t)
    res = e.step({1: 1, 2: 1})
    assert torch.equal(res[1][1][0], cold(A + [17])[150]) and torch.equal(res[2][1][0], cold(B + [23])[170])
    e.close()


def test_evicted_pages_are_recomputed_to_the_same_values_elsewhere():
    rng = np.random.default_rng(8)
    A = rng.integers(0, VOCAB, size=130).tolist()
    cold_a = cold(A)
    e = Engine(12)                                   # 9 pages for A, little room beside
    e.admit(1, A)
    e.run_to_end(1, 64)
    first_tables = e.mgr.block_table(1)
    e.finish(1)
    assert e.mgr.stats()["retained"] == 8            # the eight whole pages stay, the tail page is freed
    # a stranger takes 9 pages: 4 free + 5 evicted leaves of A's chain (deepest first)
    S = rng.integers(0, VOCAB, size=140).tolist()
    e.admit(2, S)
    e.run_to_end(2, 140)
    e.finish(2)
    assert e.mgr.stats()["evicted_pages"] >= 5
    # A again: the surviving head of its chain is reused, the rest recomputed in whatever pages there are
    cached = e.admit(3, A)
    assert 0 < cached <= 48 and cached % 16 == 0
    out = e.run_to_end(3, 37)
    same(out, cold_a, range(cached, 130), "A after eviction and recomputation")
    assert e.mgr.block_table(3)[:cached // 16] == first_tables[:cached // 16]
    e.close()
