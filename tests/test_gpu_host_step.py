"""The host-buffer step (copy inputs up, append, attend, copy the output down)
in its waiting and its pipelined form: both return, bit for bit, what the
device-tensor calls return for the same schedule, whatever the number of steps
in flight, and each step sees the KV the steps before it appended."""
import numpy as np
import pytest
import torch

from paper_2609_38981_b200 import inputs

pytestmark = pytest.mark.gpu

GEO = inputs.TINY
CONTEXTS = (37, 100, 250, 700)
SCALE = GEO.head_dim ** -0.5
NUM_PAGES = 256


def schedule(reqs):
    """A prefill call for all but the last 9 positions of every request, one speculative
    call of 3 tokens, then 6 single-token decode steps -- co-batched throughout."""
    calls = [[(i, 0, r.n - 9) for i, r in enumerate(reqs)],
             [(i, r.n - 9, 3) for i, r in enumerate(reqs)]]
    for d in range(6):
        calls.append([(i, r.n - 6 + d, 1) for i, r in enumerate(reqs)])
    return calls


@pytest.fixture(scope="module")
def env():
    from paper_2609_38981_b200.harness import DeviceCache
    import gpu_util as gu
    reqs = inputs.tiny_requests(GEO, CONTEXTS)
    tables = inputs._assign_private_pages(inputs.generator(3), GEO, NUM_PAGES, CONTEXTS)

    def cache():
        return DeviceCache(GEO, NUM_PAGES, max_batch=8, max_total_q=2048, max_seq_len=1024, pool_fill="nan")
    c = cache()
    want = gu.run_schedule(c, reqs, tables, schedule(reqs), SCALE)
    c.close()
    for i in want:
        assert (want[i] != 0x7FC2).all()
    # the device-tensor result every host-buffer variant is compared with is itself within the
    # stated tolerance of the fp64 oracle
    for i, ref in enumerate(gu.oracle_rows(reqs, SCALE)):
        gu.assert_parity(want[i], ref, f"device calls vs oracle, request {i}")
    return dict(reqs=reqs, tables=tables, cache=cache, want=want, gu=gu)


def host_buffers(reqs, tables, call):
    pin = lambda t: t.contiguous().pin_memory()
    q = pin(torch.cat([reqs[i].q_rows(s, n) for i, s, n in call]))
    k = pin(torch.cat([reqs[i].k[s:s + n] for i, s, n in call]))
    v = pin(torch.cat([reqs[i].v[s:s + n] for i, s, n in call]))
    out = torch.full_like(q, float("nan")).pin_memory()
    bt = inputs.block_table_array([tables[i] for i, _, _ in call])
    return q, k, v, out, bt


def collect(reqs, done):
    outs = {i: torch.full((r.n, GEO.n_q_heads, GEO.head_dim), 0x7FC2, dtype=torch.int16) for i, r in enumerate(reqs)}
    for call, out in done:
        bits, at = out.view(torch.int16), 0
        for i, s, n in call:
            outs[i][s:s + n] = bits[at:at + n]
            at += n
    return outs


def test_waiting_step_matches_the_device_calls(env):
    from paper_2609_38981_b200 import binding as vb
    reqs, tables = env["reqs"], env["tables"]
    c = env["cache"]()
    done = []
    for call in schedule(reqs):
        q, k, v, out, bt = host_buffers(reqs, tables, call)
        vb.vosti_step_host(c.ctx, q, out, k, v, [n for _, _, n in call], [s for _, s, _ in call],
                           [s + n for _, s, n in call], bt, SCALE)
        done.append((call, out.clone()))
    assert vb.vosti_poll_device_status(c.ctx) == vb.VOSTI_OK
    c.close()
    outs = collect(reqs, done)
    for i in outs:
        env["gu"].assert_same_bits(outs[i], env["want"][i], f"waiting host step, request {i}")


@pytest.mark.parametrize("lag", [0, 1, 2, 3, 8])
def test_pipelined_steps_match_whatever_the_depth(env, lag):
    """`lag` steps are left pending before the oldest is waited for; beyond the library's
    depth the issue call itself waits for the oldest, and its ticket still reads as done."""
    from paper_2609_38981_b200 import binding as vb
    reqs, tables = env["reqs"], env["tables"]
    c = env["cache"]()
    pending, done = [], []
    for call in schedule(reqs):
        q, k, v, out, bt = host_buffers(reqs, tables, call)
        t = vb.vosti_step_host_async(c.ctx, q, out, k, v, [n for _, _, n in call], [s for _, s, _ in call],
                                     [s + n for _, s, n in call], bt, SCALE)
        pending.append((t, call, (q, k, v, out)))
        while len(pending) > lag:
            t0, call0, bufs = pending.pop(0)
            vb.vosti_step_host_wait(c.ctx, t0)
            done.append((call0, bufs[3]))
    for t0, call0, bufs in pending:
        vb.vosti_step_host_wait(c.ctx, t0)
        vb.vosti_step_host_wait(c.ctx, t0)              # a second wait on the same ticket returns at once
        done.append((call0, bufs[3]))
    assert [t for t, _, _ in pending] == sorted(t for t, _, _ in pending)
    assert vb.vosti_poll_device_status(c.ctx) == vb.VOSTI_OK
    with pytest.raises(vb.VostiError):
        vb.vosti_step_host_wait(c.ctx, 10 ** 6)         # never issued
    c.close()
    outs = collect(reqs, done)
    for i in outs:
        env["gu"].assert_same_bits(outs[i], env["want"][i], f"pipelined host steps (lag {lag}), request {i}")


def test_an_empty_step_is_a_step(env):
    from paper_2609_38981_b200 import binding as vb
    c = env["cache"]()
    e = torch.empty((0, GEO.n_q_heads, GEO.head_dim), dtype=torch.bfloat16)
    ek = torch.empty((0, GEO.n_kv_heads, GEO.head_dim), dtype=torch.bfloat16)
    t = vb.vosti_step_host_async(c.ctx, e, e, ek, ek, [0], [0], [0], np.zeros((1, 1), np.int32), SCALE)
    vb.vosti_step_host_wait(c.ctx, t)
    c.close()
