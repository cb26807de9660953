"""A whole decoder layer around the attention op -- RMS norm, QKV projection,
rotary embedding, KV append + paged attention, output projection, residual,
RMS norm, gated MLP, residual -- with every reduction and contraction done by
this library's batch-invariant kernels (the elementwise steps are per-element
torch expressions).  The paper's claim, checked end to end on the GPU: the
layer's output for a (request, position) is bitwise the same whether the request
runs alone in one prefill call, in chunks co-batched with strangers, token by
token, or on top of prefix pages another request left in the cache."""
import numpy as np
import pytest
import torch

from paper_2609_38981_b200 import inputs

pytestmark = pytest.mark.gpu

GEO = inputs.Geometry(8, 2, 128, 16)
D_MODEL, D_FFN, VOCAB, MAXLEN = 1024, 2816, 97, 1024
EPS = 1e-5


class Layer:
    def __init__(self, seed=11):
        g = torch.Generator(device="cuda")
        g.manual_seed(seed)

        def w(n, k):
            return (torch.randn(n, k, device="cuda", generator=g) * k ** -0.5).to(torch.bfloat16)
        qkv_out = (GEO.n_q_heads + 2 * GEO.n_kv_heads) * GEO.head_dim
        self.emb = torch.randn(VOCAB, D_MODEL, device="cuda", generator=g).to(torch.bfloat16)
        self.w_qkv, self.w_o = w(qkv_out, D_MODEL), w(D_MODEL, GEO.n_q_heads * GEO.head_dim)
        self.w_gu, self.w_d = w(2 * D_FFN, D_MODEL), w(D_MODEL, D_FFN)
        self.g1 = (1 + 0.1 * torch.randn(D_MODEL, device="cuda", generator=g)).to(torch.bfloat16)
        self.g2 = (1 + 0.1 * torch.randn(D_MODEL, device="cuda", generator=g)).to(torch.bfloat16)
        half = GEO.head_dim // 2
        inv = 10000.0 ** (-torch.arange(half, device="cuda", dtype=torch.float32) / half)
        ang = torch.arange(MAXLEN, device="cuda", dtype=torch.float32)[:, None] * inv[None, :]
        self.cos, self.sin = ang.cos(), ang.sin()

    def rope(self, t, pos):
        """t [T, H, d] bf16, pos [T]: per-element fp32 arithmetic, one rounding to bf16."""
        c, s = self.cos[pos][:, None, :], self.sin[pos][:, None, :]
        a, b = t[..., :GEO.head_dim // 2].float(), t[..., GEO.head_dim // 2:].float()
        return torch.cat([a * c - b * s, a * s + b * c], dim=-1).to(torch.bfloat16)

    def forward(self, dev, tokens, positions, q_lens, starts, block_tables):
        """One call of the layer on packed token rows.  Returns [T, D_MODEL] bf16."""
        from paper_2609_38981_b200 import linear as vl
        T = len(tokens)
        x = self.emb[torch.as_tensor(tokens, device="cuda")]
        pos = torch.as_tensor(positions, device="cuda")
        ws = torch.empty(64 << 20, dtype=torch.uint8, device="cuda")       # lets small calls use the split schedule
        h = vl.vosti_rmsnorm(x, self.g1, EPS)
        qkv = vl.vosti_linear(h, self.w_qkv, workspace=ws).view(T, -1, GEO.head_dim)
        q = self.rope(qkv[:, :GEO.n_q_heads], pos).contiguous()
        k = self.rope(qkv[:, GEO.n_q_heads:GEO.n_q_heads + GEO.n_kv_heads], pos).contiguous()
        v = qkv[:, GEO.n_q_heads + GEO.n_kv_heads:].contiguous()
        dev.append(k, v, q_lens, starts, block_tables)
        seq = [s + n for s, n in zip(starts, q_lens)]
        att = dev.attend(q, q_lens, starts, seq, block_tables, GEO.head_dim ** -0.5)
        o = vl.vosti_linear(att.view(T, -1).contiguous(), self.w_o, workspace=ws)
        x1 = (x.float() + o.float()).to(torch.bfloat16)
        h2 = vl.vosti_rmsnorm(x1, self.g2, EPS)
        gu = vl.vosti_linear(h2, self.w_gu, workspace=ws)
        gate, up = gu[:, :D_FFN].float(), gu[:, D_FFN:].float()
        act = (gate * torch.sigmoid(gate) * up).to(torch.bfloat16).contiguous()
        down = vl.vosti_linear(act, self.w_d, workspace=ws)
        return (x1.float() + down.float()).to(torch.bfloat16)


def run(layer, requests, schedule, num_pages=256, tables=None, cache=None):
    """schedule: list of calls, each a list of (request index, start, count).  Returns per
    request an int16 tensor [n, D_MODEL] of output bits."""
    from paper_2609_38981_b200.harness import DeviceCache, bf16_bits
    dev = cache or DeviceCache(GEO, num_pages, max_batch=16, max_total_q=2048, max_seq_len=MAXLEN, pool_fill="nan")
    if tables is None:
        tables = inputs._assign_private_pages(inputs.generator(5), GEO, num_pages, [len(r) for r in requests])
    outs = {i: torch.full((len(r), D_MODEL), 0x7FC2, dtype=torch.int16) for i, r in enumerate(requests)}
    for call in schedule:
        toks = [t for i, s, n in call for t in requests[i][s:s + n]]
        poss = [p for i, s, n in call for p in range(s, s + n)]
        bt = inputs.block_table_array([tables[i] for i, _, _ in call])
        y = bf16_bits(layer.forward(dev, toks, poss, [n for _, _, n in call], [s for _, s, _ in call], bt))
        at = 0
        for i, s, n in call:
            outs[i][s:s + n] = y[at:at + n]
            at += n
    if cache is None:
        dev.close()
    return outs


@pytest.fixture(scope="module")
def setup():
    rng = np.random.default_rng(21)
    lens = (1, 37, 130, 300, 520)
    requests = [rng.integers(0, VOCAB, size=n).tolist() for n in lens]
    layer = Layer()
    alone = {}
    for i, r in enumerate(requests):
        alone[i] = run(layer, requests, [[(i, 0, len(r))]])[i]
    return layer, requests, alone


def test_cobatched_and_chunked_prefill(setup):
    layer, requests, alone = setup
    outs = run(layer, requests, [[(i, 0, len(r)) for i, r in enumerate(requests)]])
    for i in outs:
        assert torch.equal(outs[i], alone[i]), f"co-batched: request {i}"
    for chunk in (16, 100):
        steps = max(-(-len(r) // chunk) for r in requests)
        sched = [[(i, c * chunk, min(chunk, len(r) - c * chunk)) for i, r in enumerate(requests) if c * chunk < len(r)]
                 for c in range(steps)]
        outs = run(layer, requests, sched)
        for i in outs:
            assert torch.equal(outs[i], alone[i]), f"chunk {chunk}: request {i}"


def test_decode_after_prefill(setup):
    """Prefill all but the last 6 positions in one call each, then decode them one token at a
    time, all requests together."""
    layer, requests, alone = setup
    tail = {i: min(6, len(r) - 1) for i, r in enumerate(requests)}
    sched = [[(i, 0, len(r) - tail[i]) for i, r in enumerate(requests)]]
    for d in range(6):
        call = [(i, len(r) - tail[i] + d, 1) for i, r in enumerate(requests) if d < tail[i]]
        if call:
            sched.append(call)
    outs = run(layer, requests, sched)
    for i in outs:
        assert torch.equal(outs[i], alone[i]), f"decode tail: request {i}"


def test_prefix_reuse_through_the_cache_manager(setup):
    """Request B shares its first 200 tokens with request A, which ran earlier: the manager hands
    B the pages A registered, B computes only its suffix, and gets the bits of its cold run."""
    from paper_2609_38981_b200.cache import PrefixCache
    from paper_2609_38981_b200.harness import DeviceCache
    layer, requests, _ = setup
    rng = np.random.default_rng(22)
    a = requests[4][:400]
    b = a[:200] + rng.integers(0, VOCAB, size=150).tolist()
    cold = run(layer, [b], [[(0, 0, len(b))]])[0]
    mgr = PrefixCache(256, GEO.page_size)
    dev = DeviceCache(GEO, 256, max_batch=16, max_total_q=2048, max_seq_len=MAXLEN, pool_fill="nan")
    assert mgr.admit(1, a) == 0
    run(layer, [a], [[(0, 0, len(a))]], tables=[mgr.block_table(1)], cache=dev)
    mgr.computed(1, len(a))
    mgr.step_boundary()
    cached = mgr.admit(2, b)
    assert cached == 192                                  # twelve whole pages of the shared 200 tokens
    out = run(layer, [b], [[(0, cached, len(b) - cached)]], tables=[mgr.block_table(2)], cache=dev)[0]
    assert torch.equal(out[cached:], cold[cached:])
    assert mgr.check() == ""
    dev.close()
    mgr.close()


def test_a_whole_layer_decode_step_replays_from_a_cuda_graph(setup):
    """One capture of a decode step of the layer -- RMS norm, QKV projection, rotary embedding, device-side
    planning, KV append, attention, output projection, MLP -- with positions and block tables in device
    memory; every replay equals the eager, host-planned step bit for bit."""
    from paper_2609_38981_b200 import binding as vb
    from paper_2609_38981_b200 import linear as vl
    from paper_2609_38981_b200.harness import DeviceCache, bf16_bits
    layer, requests, alone = setup
    reqs = [r for r in requests if len(r) > 12]
    B, tail = len(reqs), 6
    tables = inputs._assign_private_pages(inputs.generator(9), GEO, 256, [len(r) for r in reqs])
    dev = DeviceCache(GEO, 256, max_batch=16, max_total_q=2048, max_seq_len=MAXLEN, pool_fill="nan")
    # prefill eagerly (host-planned), all but the last `tail` positions
    run(layer, reqs, [[(i, 0, len(r) - tail) for i, r in enumerate(reqs)]], tables=tables, cache=dev)
    bt = torch.from_numpy(inputs.block_table_array(tables)).cuda()
    tok = torch.zeros(B, dtype=torch.long, device="cuda")
    pos = torch.zeros(B, dtype=torch.int32, device="cuda")
    ones = torch.ones(B, dtype=torch.int32, device="cuda")
    plan = torch.empty(vb.vosti_device_plan_bytes(dev.ctx), dtype=torch.uint8, device="cuda")
    ws = torch.empty(64 << 20, dtype=torch.uint8, device="cuda")
    y = torch.zeros((B, D_MODEL), dtype=torch.bfloat16, device="cuda")

    def step():
        x = layer.emb[tok]
        p = pos.long()
        h = vl.vosti_rmsnorm(x, layer.g1, EPS)
        qkv = vl.vosti_linear(h, layer.w_qkv, workspace=ws).view(B, -1, GEO.head_dim)
        q = layer.rope(qkv[:, :GEO.n_q_heads], p).contiguous()
        k = layer.rope(qkv[:, GEO.n_q_heads:GEO.n_q_heads + GEO.n_kv_heads], p).contiguous()
        v = qkv[:, GEO.n_q_heads + GEO.n_kv_heads:].contiguous()
        att = torch.empty_like(q)
        vb.vosti_plan_device(dev.ctx, plan, ones, pos, bt, 1)
        vb.vosti_kv_append_planned(dev.ctx, plan, k, v, bt, 1)
        vb.vosti_paged_attention_planned(dev.ctx, plan, q, att, None, bt, 1, GEO.head_dim ** -0.5)
        o = vl.vosti_linear(att.view(B, -1), layer.w_o, workspace=ws)
        x1 = (x.float() + o.float()).to(torch.bfloat16)
        h2 = vl.vosti_rmsnorm(x1, layer.g2, EPS)
        gu = vl.vosti_linear(h2, layer.w_gu, workspace=ws)
        gate, up = gu[:, :D_FFN].float(), gu[:, D_FFN:].float()
        act = (gate * torch.sigmoid(gate) * up).to(torch.bfloat16).contiguous()
        down = vl.vosti_linear(act, layer.w_d, workspace=ws)
        y.copy_((x1.float() + down.float()).to(torch.bfloat16))

    def load(d):
        tok.copy_(torch.tensor([r[len(r) - tail + d] for r in reqs]))
        pos.copy_(torch.tensor([len(r) - tail + d for r in reqs], dtype=torch.int32))

    load(0)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()                                  # warm-up outside capture (writes position len - tail, as replay 0 will)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    index = {id(r): i for i, r in enumerate(requests)}
    for d in range(tail):
        load(d)
        graph.replay()
        got = bf16_bits(y)
        for j, r in enumerate(reqs):
            want = alone[index[id(r)]][len(r) - tail + d]
            assert torch.equal(got[j], want), f"replay {d}, request {j}: differs from its run alone"
    assert vb.vosti_poll_device_status(dev.ctx) == vb.VOSTI_OK and vl.vosti_linear_poll_status() == 0
    dev.close()
