"""Device-planned decode steps: lengths, start positions and block tables in
device memory, planned by a kernel, so that a step can be captured once in a
CUDA graph and replayed with other metadata.  The outputs, the log-sum-exp and
the KV written to the pool must be, bit for bit, those of the host-planned
calls for the same logical requests; metadata outside the premises sets the
device status word and faults nothing."""
import numpy as np
import pytest
import torch

from paper_2609_38981_b200 import inputs

pytestmark = pytest.mark.gpu

GEOS = {
    "d128_g4": (inputs.Geometry(8, 2, 128, 16), 4),      # geometry, largest q_len that stays split-parallel (tested)
    "d64_g2": (inputs.TINY, 4),
    "d128_g8": (inputs.Geometry(8, 1, 128, 16), 4),
    "d128_g16": (inputs.Geometry(16, 1, 128, 16), 2),
}
# contexts around page, tile and split edges; each request also has a tail of positions to decode
CONTEXTS = (1, 17, 64, 300, 511, 512, 513, 1030, 1600)
TAIL = 13
NUM_PAGES = 1024
MAXLEN = 2048


class Env:
    def __init__(self, geo):
        from paper_2609_38981_b200.harness import DeviceCache
        self.geo = geo
        self.scale = geo.head_dim ** -0.5
        self.reqs = [inputs.make_request(geo, 777, i, n + TAIL) for i, n in enumerate(CONTEXTS)]
        self.tables = inputs._assign_private_pages(inputs.generator(777), geo, NUM_PAGES, [r.n for r in self.reqs])
        self.bt = inputs.block_table_array(self.tables)
        self.new_cache = lambda: DeviceCache(geo, NUM_PAGES, max_batch=16, max_total_q=2048, max_seq_len=MAXLEN,
                                             pool_fill="nan")

    def prefill(self, cache):
        cache.upload(self.reqs, self.tables, upto=list(CONTEXTS))

    def rows(self, call):
        q = torch.cat([self.reqs[i].q_rows(s, n) for i, s, n in call if n > 0]).cuda().contiguous()
        k = torch.cat([self.reqs[i].k[s:s + n] for i, s, n in call if n > 0]).cuda().contiguous()
        v = torch.cat([self.reqs[i].v[s:s + n] for i, s, n in call if n > 0]).cuda().contiguous()
        return q, k, v


@pytest.fixture(scope="module", params=list(GEOS))
def env(request):
    geo, max_q = GEOS[request.param]
    e = Env(geo)
    e.max_q = max_q
    return e


def host_step(env, cache, call):
    from paper_2609_38981_b200 import binding as vb
    q, k, v = env.rows(call)
    ql, st = [n for _, _, n in call], [s for _, s, _ in call]
    vb.vosti_kv_append(cache.ctx, k, v, ql, st, env.bt)
    out = torch.empty_like(q)
    out.view(torch.int16).fill_(0x7FC1)
    lse = torch.full(q.shape[:2], float("nan"), dtype=torch.float32, device="cuda")
    vb.vosti_paged_attention_ex(cache.ctx, q, out, lse, ql, st, [s + n for _, s, n in call], env.bt, env.scale)
    return out, lse


def device_step(env, cache, plan, call, max_q_len):
    from paper_2609_38981_b200 import binding as vb
    q, k, v = env.rows(call)
    ql = torch.tensor([n for _, _, n in call], dtype=torch.int32, device="cuda")
    st = torch.tensor([s for _, s, _ in call], dtype=torch.int32, device="cuda")
    bt = torch.from_numpy(env.bt).cuda()
    out = torch.empty_like(q)
    out.view(torch.int16).fill_(0x7FC1)
    lse = torch.full(q.shape[:2], float("nan"), dtype=torch.float32, device="cuda")
    vb.vosti_plan_device(cache.ctx, plan, ql, st, bt, max_q_len)
    vb.vosti_kv_append_planned(cache.ctx, plan, k, v, bt, max_q_len)
    vb.vosti_paged_attention_planned(cache.ctx, plan, q, out, lse, bt, max_q_len, env.scale)
    return out, lse


def new_plan(cache):
    from paper_2609_38981_b200 import binding as vb
    n = vb.vosti_device_plan_bytes(cache.ctx)
    assert n > 0
    return torch.empty(n, dtype=torch.uint8, device="cuda")


def same(a, b, what):
    assert torch.equal(a.view(torch.int16), b.view(torch.int16)), f"{what}: outputs differ bitwise"


def test_decode_and_speculative_steps_equal_the_host_planned_calls(env):
    from paper_2609_38981_b200 import binding as vb
    host, dev = env.new_cache(), env.new_cache()
    env.prefill(host)
    env.prefill(dev)
    plan = new_plan(dev)
    done = list(CONTEXTS)
    rng = np.random.default_rng(5)
    for step in range(6):
        # a mix of query lengths per request, zero included (a request that sits a step out)
        ql = [int(rng.integers(0, env.max_q + 1)) for _ in CONTEXTS] if step else [1] * len(CONTEXTS)
        ql = [min(n, c + TAIL - d) for n, c, d in zip(ql, CONTEXTS, done)]
        if sum(ql) == 0:
            ql[0] = 1
        call = [(i, done[i], ql[i]) for i in range(len(CONTEXTS))]
        oh, lh = host_step(env, host, call)
        od, ld = device_step(env, dev, plan, call, env.max_q)
        same(od, oh, f"step {step}, q_lens {ql}")
        assert torch.equal(ld.view(torch.int32), lh.view(torch.int32)), f"step {step}: log-sum-exp differs bitwise"
        if step < 2:   # and directly against the fp64 oracle (not only against the host-planned GPU path)
            import gpu_util as gu
            if not hasattr(env, "oracle"):
                env.oracle = gu.oracle_rows(env.reqs, env.scale)
            ref = np.concatenate([env.oracle[i][s:s + n] for i, s, n in call if n > 0])
            gu.assert_parity(od.cpu().view(torch.int16), ref, f"device-planned step {step} vs oracle")
        assert not (od.view(torch.int16) == 0x7FC1).any()
        done = [d + n for d, n in zip(done, ql)]
    used = sorted({p for t in env.tables for p in t})
    assert torch.equal(host.pool[used].view(torch.int16), dev.pool[used].view(torch.int16))   # appended KV
    assert vb.vosti_poll_device_status(dev.ctx) == vb.VOSTI_OK
    host.close()
    dev.close()


def test_a_captured_graph_replays_with_new_metadata(env):
    """One capture of plan + append + attention; every replay advances the device-side start
    positions and refills the static Q / K / V buffers."""
    from paper_2609_38981_b200 import binding as vb
    geo, B = env.geo, len(CONTEXTS)
    host, dev = env.new_cache(), env.new_cache()
    env.prefill(host)
    env.prefill(dev)
    plan = new_plan(dev)
    ql = torch.ones(B, dtype=torch.int32, device="cuda")
    st = torch.tensor(CONTEXTS, dtype=torch.int32, device="cuda")
    bt = torch.from_numpy(env.bt).cuda()
    q = torch.zeros((B, geo.n_q_heads, geo.head_dim), dtype=torch.bfloat16, device="cuda")
    k = torch.zeros((B, geo.n_kv_heads, geo.head_dim), dtype=torch.bfloat16, device="cuda")
    v = torch.zeros_like(k)
    out = torch.zeros_like(q)
    lse = torch.zeros((B, geo.n_q_heads), dtype=torch.float32, device="cuda")

    def fill(step):
        call = [(i, CONTEXTS[i] + step, 1) for i in range(B)]
        qs, ks, vs = env.rows(call)
        q.copy_(qs)
        k.copy_(ks)
        v.copy_(vs)
        st.copy_(torch.tensor([s for _, s, _ in call], dtype=torch.int32))
        return call

    fill(0)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):          # one eager run first: lazy module loading must not happen under capture
        vb.vosti_plan_device(dev.ctx, plan, ql, st, bt, 1)
        vb.vosti_paged_attention_planned(dev.ctx, plan, q, out, lse, bt, 1, env.scale)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        vb.vosti_plan_device(dev.ctx, plan, ql, st, bt, 1)
        vb.vosti_kv_append_planned(dev.ctx, plan, k, v, bt, 1)
        vb.vosti_paged_attention_planned(dev.ctx, plan, q, out, lse, bt, 1, env.scale)
    for step in range(TAIL):
        call = fill(step)
        out.view(torch.int16).fill_(0x7FC1)
        graph.replay()
        oh, lh = host_step(env, host, call)
        same(out, oh, f"replay {step}")
        assert torch.equal(lse.view(torch.int32), lh.view(torch.int32)), f"replay {step}: log-sum-exp differs"
    assert vb.vosti_poll_device_status(dev.ctx) == vb.VOSTI_OK
    host.close()
    dev.close()


def test_bad_metadata_sets_the_status_word_and_spares_the_rest(env):
    from paper_2609_38981_b200 import binding as vb
    host, dev = env.new_cache(), env.new_cache()
    env.prefill(host)
    env.prefill(dev)
    plan = new_plan(dev)
    call = [(i, CONTEXTS[i], 1) for i in range(len(CONTEXTS))]
    oh, _ = host_step(env, host, call)
    q, k, v = env.rows(call)
    st = torch.tensor(CONTEXTS, dtype=torch.int32, device="cuda")
    bt = torch.from_numpy(env.bt).cuda()
    # request 3 claims more query rows than the call allows, request 5 a negative start
    ql = torch.ones(len(CONTEXTS), dtype=torch.int32, device="cuda")
    for bad_ql, bad_st in (({3: env.max_q + 1}, {}), ({}, {5: -4}), ({2: -1}, {}), ({}, {6: MAXLEN})):
        ql2, st2 = ql.clone(), st.clone()
        for i, x in bad_ql.items():
            ql2[i] = x
        for i, x in bad_st.items():
            st2[i] = x
        out = torch.empty_like(q)
        out.view(torch.int16).fill_(0x7FC1)
        vb.vosti_plan_device(dev.ctx, plan, ql2, st2, bt, env.max_q)
        vb.vosti_paged_attention_planned(dev.ctx, plan, q, out, None, bt, env.max_q, env.scale)
        assert vb.vosti_poll_device_status(dev.ctx) == vb.VOSTI_ERR_OUT_OF_RANGE
        assert vb.vosti_poll_device_status(dev.ctx) == vb.VOSTI_OK          # cleared by the read
    # a page id outside the pool: reported, never written through
    bt_bad = bt.clone()
    bt_bad[4, CONTEXTS[4] // 16] = NUM_PAGES + 5
    snapshot = dev.pool.clone()
    vb.vosti_plan_device(dev.ctx, plan, ql, st, bt_bad, 1)
    vb.vosti_kv_append_planned(dev.ctx, plan, k, v, bt_bad, 1)
    assert vb.vosti_poll_device_status(dev.ctx) == vb.VOSTI_ERR_OUT_OF_RANGE
    touched = sorted({env.tables[i][CONTEXTS[i] // 16] for i in range(len(CONTEXTS)) if i != 4})
    rest = [p for p in range(NUM_PAGES) if p not in touched]
    assert torch.equal(dev.pool[rest].view(torch.int16), snapshot[rest].view(torch.int16))
    # and a clean step afterwards is right again (the append above wrote every request but the fourth)
    vb.vosti_plan_device(dev.ctx, plan, ql, st, bt, 1)
    vb.vosti_kv_append_planned(dev.ctx, plan, k, v, bt, 1)
    out = torch.empty_like(q)
    vb.vosti_paged_attention_planned(dev.ctx, plan, q, out, None, bt, 1, env.scale)
    same(out, oh, "after the rejected steps")
    assert vb.vosti_poll_device_status(dev.ctx) == vb.VOSTI_OK
    # host-detectable errors are returned by the call
    with pytest.raises(vb.VostiError) as e:
        vb.vosti_plan_device(dev.ctx, plan, ql, st, bt, 40)
    assert e.value.status == vb.VOSTI_ERR_UNSUPPORTED_CONFIG
    host.close()
    dev.close()


def test_one_plan_serves_the_contexts_of_several_layers(env):
    """A plan written through one context drives another context of the same configuration
    (another layer's pool): planning happens once per step, not once per layer."""
    from paper_2609_38981_b200 import binding as vb
    host, layer_a, layer_b = env.new_cache(), env.new_cache(), env.new_cache()
    env.prefill(host)
    env.prefill(layer_b)
    plan = new_plan(layer_a)
    call = [(i, CONTEXTS[i], 1) for i in range(len(CONTEXTS))]
    oh, lh = host_step(env, host, call)
    q, k, v = env.rows(call)
    ql = torch.ones(len(CONTEXTS), dtype=torch.int32, device="cuda")
    st = torch.tensor(CONTEXTS, dtype=torch.int32, device="cuda")
    bt = torch.from_numpy(env.bt).cuda()
    out = torch.empty_like(q)
    lse = torch.empty(q.shape[:2], dtype=torch.float32, device="cuda")
    vb.vosti_plan_device(layer_a.ctx, plan, ql, st, bt, 1)
    vb.vosti_kv_append_planned(layer_b.ctx, plan, k, v, bt, 1)
    vb.vosti_paged_attention_planned(layer_b.ctx, plan, q, out, lse, bt, 1, env.scale)
    same(out, oh, "plan from another context")
    assert torch.equal(lse.view(torch.int32), lh.view(torch.int32))
    for c in (host, layer_a, layer_b):
        assert vb.vosti_poll_device_status(c.ctx) == vb.VOSTI_OK
        c.close()


@pytest.mark.parametrize("batch", [300, 1500])
def test_large_batches_are_planned_in_chunks(batch):
    """More requests than the planner has threads (and than its shared-memory prefix holds):
    the scan carries over chunks of requests and the item search falls back to global memory."""
    from paper_2609_38981_b200 import binding as vb
    from paper_2609_38981_b200.harness import DeviceCache
    geo = inputs.Geometry(8, 2, 128, 16)
    scale = geo.head_dim ** -0.5
    rng = np.random.default_rng(batch)
    ctx = [int(x) for x in rng.integers(1, 700, size=batch)]
    ctx[:4] = [511, 512, 513, 1]
    qls = [int(x) for x in rng.integers(0, 5, size=batch)]          # decode, speculative, idle
    qls[:4] = [4, 1, 2, 1]
    n_pages = sum(inputs.pages_needed(c + q, geo.page_size) for c, q in zip(ctx, qls))
    num_pages = n_pages + 64
    reqs = [inputs.make_request(geo, 4321, i, c + q) for i, (c, q) in enumerate(zip(ctx, qls))]
    tables = inputs._assign_private_pages(inputs.generator(batch), geo, num_pages, [r.n for r in reqs])
    bt = inputs.block_table_array(tables)
    mk = lambda: DeviceCache(geo, num_pages, max_batch=2048, max_total_q=8192, max_seq_len=1024, pool_fill="nan")
    host, dev = mk(), mk()
    for c in (host, dev):
        c.upload(reqs, tables, upto=ctx)
    call = [(i, ctx[i], qls[i]) for i in range(batch)]
    q = torch.cat([reqs[i].q_rows(s, n) for i, s, n in call if n > 0]).cuda().contiguous()
    k = torch.cat([reqs[i].k[s:s + n] for i, s, n in call if n > 0]).cuda().contiguous()
    v = torch.cat([reqs[i].v[s:s + n] for i, s, n in call if n > 0]).cuda().contiguous()
    oh, od = torch.empty_like(q), torch.empty_like(q)
    for o in (oh, od):
        o.view(torch.int16).fill_(0x7FC1)
    lh = torch.full(q.shape[:2], float("nan"), dtype=torch.float32, device="cuda")
    ld = lh.clone()
    vb.vosti_kv_append(host.ctx, k, v, qls, ctx, bt)
    vb.vosti_paged_attention_ex(host.ctx, q, oh, lh, qls, ctx, [c + n for c, n in zip(ctx, qls)], bt, scale)
    plan = new_plan(dev)
    ql_d = torch.tensor(qls, dtype=torch.int32, device="cuda")
    st_d = torch.tensor(ctx, dtype=torch.int32, device="cuda")
    bt_d = torch.from_numpy(bt).cuda()
    vb.vosti_plan_device(dev.ctx, plan, ql_d, st_d, bt_d, 4)
    vb.vosti_kv_append_planned(dev.ctx, plan, k, v, bt_d, 4)
    vb.vosti_paged_attention_planned(dev.ctx, plan, q, od, ld, bt_d, 4, scale)
    same(od, oh, f"batch {batch}")
    assert torch.equal(ld.view(torch.int32), lh.view(torch.int32))
    assert not (od.view(torch.int16) == 0x7FC1).any()
    assert vb.vosti_poll_device_status(dev.ctx) == vb.VOSTI_OK
    assert vb.vosti_last_schedule(host.ctx)[0] > batch          # more items than requests: several splits and groups
    host.close()
    dev.close()


@pytest.mark.parametrize("window", [64, 100, 513, 700, 5000])
def test_sliding_window_steps_equal_the_host_planned_calls(env, window):
    """Decode and speculative steps under a sliding window: items start at the split that holds
    the first visible key, the first and last split of a row group may both be partial, and
    block-table entries wholly before the window hold -1 (pages given back)."""
    from paper_2609_38981_b200 import binding as vb
    host, dev = env.new_cache(), env.new_cache()
    env.prefill(host)
    env.prefill(dev)
    plan = new_plan(dev)
    done = list(CONTEXTS)
    rng = np.random.default_rng(window)
    for step in range(4):
        ql = [int(rng.integers(0, env.max_q + 1)) for _ in CONTEXTS] if step else [1] * len(CONTEXTS)
        ql = [min(n, c + TAIL - d) for n, c, d in zip(ql, CONTEXTS, done)]
        if sum(ql) == 0:
            ql[0] = 1
        call = [(i, done[i], ql[i]) for i in range(len(CONTEXTS))]
        q, k, v = env.rows(call)
        st = [s for _, s, _ in call]
        # pages wholly before the window of the request's first row: freed
        bt_w = env.bt.copy()
        for row, s in enumerate(st):
            bt_w[row, :max(0, s - window + 1) // env.geo.page_size] = -1
        vb.vosti_kv_append(host.ctx, k, v, ql, st, env.bt)
        oh = torch.empty_like(q)
        lh = torch.full(q.shape[:2], float("nan"), dtype=torch.float32, device="cuda")
        vb.vosti_paged_attention_ex(host.ctx, q, oh, lh, ql, st, [s + n for s, n in zip(st, ql)], bt_w, env.scale,
                                    window=window)
        ql_d = torch.tensor(ql, dtype=torch.int32, device="cuda")
        st_d = torch.tensor(st, dtype=torch.int32, device="cuda")
        bt_d = torch.from_numpy(bt_w).cuda()
        od = torch.empty_like(q)
        od.view(torch.int16).fill_(0x7FC1)
        ld = torch.full(q.shape[:2], float("nan"), dtype=torch.float32, device="cuda")
        vb.vosti_plan_device(dev.ctx, plan, ql_d, st_d, bt_d, env.max_q, window=window)
        vb.vosti_kv_append_planned(dev.ctx, plan, k, v, bt_d, env.max_q)
        vb.vosti_paged_attention_planned(dev.ctx, plan, q, od, ld, bt_d, env.max_q, env.scale, window=window)
        same(od, oh, f"window {window}, step {step}, q_lens {ql}")
        assert torch.equal(ld.view(torch.int32), lh.view(torch.int32)), f"window {window}, step {step}: log-sum-exp"
        assert not (od.view(torch.int16) == 0x7FC1).any()
        done = [d + n for d, n in zip(done, ql)]
    assert vb.vosti_poll_device_status(dev.ctx) == vb.VOSTI_OK
    host.close()
    dev.close()
