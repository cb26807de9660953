"""The two options of App. A on the GPU path: the sliding-window mask (a key is
visible iff p - w < j <= p) and the auxiliary log-sum-exp output.

Same bar as the plain path: within the stated tolerance of the fp64 oracle, and
bit for bit the same whatever the batch composition, chunking, prefill / decode
split or page placement.  Key tiles and splits stay absolute under a window, so
a window at least as long as the context must reproduce the unwindowed bits."""
import numpy as np
import pytest
import torch

from paper_2609_38981_b200 import inputs

pytestmark = pytest.mark.gpu

GEOS = {
    "d64_g2": inputs.TINY,
    "d128_g4": inputs.Geometry(8, 2, 128, 16),
    "d128_g8": inputs.Geometry(8, 1, 128, 16),
}
CONTEXTS = (1, 16, 100, 513, 1025, 1600)
WINDOWS = (1, 17, 64, 100, 512, 600, 1500)
NUM_PAGES = 512


@pytest.fixture(scope="module", params=list(GEOS))
def env(request):
    from paper_2609_38981_b200.harness import DeviceCache
    import gpu_util as gu
    geo = GEOS[request.param]
    scale = geo.head_dim ** -0.5
    reqs = [inputs.make_request(geo, 777, i, n) for i, n in enumerate(CONTEXTS)]
    gen = inputs.generator(777)
    tables = inputs._assign_private_pages(gen, geo, NUM_PAGES, CONTEXTS)

    def cache(fill="zeros"):
        return DeviceCache(geo, NUM_PAGES, max_batch=16, max_total_q=8192, max_seq_len=2048,
                           pool_fill=fill)

    # canonical per window (None = plain entry point): each request alone, one full-length call
    canon, canon_lse = {}, {}

    def canonical(window):
        if window not in canon:
            c = cache()
            outs, lses = {}, {}
            for i, r in enumerate(reqs):
                one = None if window is None else {}
                outs[i] = gu.run_schedule(c, reqs, tables, [[(i, 0, r.n)]], scale, window=window,
                                          lse_out=one)[i]
                lses[i] = None if one is None else one[i]
            c.close()
            canon[window], canon_lse[window] = outs, lses
        return canon[window], canon_lse[window]

    return dict(geo=geo, scale=scale, reqs=reqs, tables=tables, cache=cache, canonical=canonical, gu=gu)


def oracle_window(env, window):
    from oracle import oracle
    return [oracle.attention_dense(inputs.bits(r.q), inputs.bits(r.k), inputs.bits(r.v), r.q0,
                                   env["scale"], window=window, return_lse=True) for r in env["reqs"]]


def f32(bits_i32: torch.Tensor) -> np.ndarray:
    return bits_i32.view(torch.float32).to(torch.float64).numpy()


def check_bits(env, outs, lses, window, what, rows=None):
    gu = env["gu"]
    canon, canon_lse = env["canonical"](window)
    for i in outs:
        lo, hi = (0, env["reqs"][i].n) if rows is None else rows(i)
        gu.assert_same_bits(outs[i][lo:hi], canon[i][lo:hi], f"{what}, window {window}, request {i}")
        if lses is not None:
            gu.assert_same_bits(lses[i][lo:hi], canon_lse[i][lo:hi],
                                f"{what}, window {window}, log-sum-exp of request {i}")


@pytest.mark.parametrize("window", (0,) + WINDOWS)
def test_parity_with_oracle(env, window):
    """Output within max 1e-2 / mean 1e-3; log-sum-exp (fp32, values of order 1..10,
    approximated exponentials and logarithm with relative error ~1e-7, sums of up to
    1600 terms) within 1e-4 + 1e-5 |ref|."""
    canon, canon_lse = env["canonical"](window)
    ref = oracle_window(env, window)
    for i in canon:
        env["gu"].assert_parity(canon[i], ref[i][0], f"window {window}, request {i}")
        got = f32(canon_lse[i])
        assert np.isfinite(got).all()
        err = np.abs(got - ref[i][1])
        assert (err <= 1e-4 + 1e-5 * np.abs(ref[i][1])).all(), (window, i, float(err.max()))


def test_window_zero_and_plain_entry_point_agree(env):
    plain, _ = env["canonical"](None)
    zero, _ = env["canonical"](0)
    for i in plain:
        env["gu"].assert_same_bits(zero[i], plain[i], f"window 0 vs plain, request {i}")


def test_window_covering_the_context_changes_nothing(env):
    """w > p for every row: the mask adds nothing, tiles and splits are the same."""
    plain, plain_lse = env["canonical"](0)
    wide, wide_lse = env["canonical"](5000)
    for i in plain:
        env["gu"].assert_same_bits(wide[i], plain[i], f"request {i}")
        env["gu"].assert_same_bits(wide_lse[i], plain_lse[i], f"log-sum-exp of request {i}")
    # and with w = p + 1 exactly for the last row of each request
    c = env["cache"]()
    c.upload(env["reqs"], env["tables"])
    for i, r in enumerate(env["reqs"]):
        one = {}
        outs = env["gu"].run_schedule(c, env["reqs"], env["tables"], [[(i, r.n - 1, 1)]], env["scale"],
                                      append=False, window=r.n, lse_out=one)
        env["gu"].assert_same_bits(outs[i][r.n - 1:], plain[i][r.n - 1:], f"w = n, request {i}")
        env["gu"].assert_same_bits(one[i][r.n - 1:], plain_lse[i][r.n - 1:], f"w = n, lse of request {i}")
    c.close()


@pytest.mark.parametrize("window", (0, 17, 100, 600))
def test_cobatched_prefill(env, window):
    c = env["cache"]("random")
    lses = {}
    outs = env["gu"].run_schedule(c, env["reqs"], env["tables"],
                                  [[(i, 0, r.n) for i, r in enumerate(env["reqs"])]], env["scale"],
                                  window=window, lse_out=lses)
    check_bits(env, outs, lses, window, "co-batched")
    c.close()


@pytest.mark.parametrize("window", (0, 17, 100, 600))
@pytest.mark.parametrize("chunk", (7, 64, 500))
def test_chunked_prefill(env, window, chunk):
    """Chunks of 7 run split-parallel, the larger ones on the tile kernel.  The pages a
    window has left behind are withheld from the block table (entries -1) and the pool
    starts out non-finite, so a read of anything outside the window shows."""
    gu, reqs = env["gu"], env["reqs"]
    c = env["cache"]("nan")
    per = {i: gu.chunked(r.n, chunk) for i, r in enumerate(reqs)}
    steps = max(len(v) for v in per.values())
    sched = [[(i, *per[i][s]) for i in per if s < len(per[i])] for s in range(steps)]
    lses = {}
    outs = gu.run_schedule(c, reqs, env["tables"], sched, env["scale"], window=window, lse_out=lses,
                           drop_pages_before_window=True)
    check_bits(env, outs, lses, window, f"chunk {chunk}")
    c.close()


@pytest.mark.parametrize("window", (1, 17, 100, 512, 600))
@pytest.mark.parametrize("ql", (1, 4))
def test_decode_and_speculative_tail(env, window, ql):
    """The last 8 positions by split-parallel calls of q_len 1 or 4 after one prefill call."""
    gu, reqs = env["gu"], env["reqs"]
    c = env["cache"]("nan")
    tail = {i: min(8, r.n) for i, r in enumerate(reqs)}
    sched = [[(i, 0, r.n - tail[i]) for i, r in enumerate(reqs) if r.n > tail[i]]]
    for w in range(8 // ql):
        sched.append([(i, r.n - tail[i] + w * ql, ql) for i, r in enumerate(reqs)
                      if w * ql + ql <= tail[i]])
    sched = [s for s in sched if s]
    lses = {}
    outs = gu.run_schedule(c, reqs, env["tables"], sched, env["scale"], window=window, lse_out=lses,
                           drop_pages_before_window=True)
    check_bits(env, outs, lses, window, f"tail q_len {ql}", rows=lambda i: (0, reqs[i].n - tail[i] % ql))
    c.close()


@pytest.mark.parametrize("window", (100, 600))
def test_decode_every_position_across_a_split_edge(env, window):
    """Single-token decode at positions 500..1130 step 7 of the longest request: the window's
    first key crosses tile and split edges (first split 0 -> 1) along the way."""
    gu, reqs = env["gu"], env["reqs"]
    i = len(reqs) - 1
    c = env["cache"]()
    c.upload(reqs, env["tables"])
    pos = list(range(500, 531)) + list(range(531, 1131, 7))
    sched = [[(i, p, 1)] for p in pos]
    lses = {}
    outs = gu.run_schedule(c, reqs, env["tables"], sched, env["scale"], append=False,
                           seq_lens_override={i: reqs[i].n}, window=window, lse_out=lses)
    canon, canon_lse = env["canonical"](window)
    idx = torch.tensor(pos)
    gu.assert_same_bits(outs[i][idx], canon[i][idx], f"decode, window {window}")
    gu.assert_same_bits(lses[i][idx], canon_lse[i][idx], f"decode, window {window}, log-sum-exp")
    c.close()


def test_lse_pointer_is_optional_and_does_not_change_the_output(env):
    gu, reqs = env["gu"], env["reqs"]
    c = env["cache"]()
    outs = gu.run_schedule(c, reqs, env["tables"], [[(i, 0, r.n) for i, r in enumerate(reqs)]],
                           env["scale"], window=100)
    check_bits(env, outs, None, 100, "no log-sum-exp requested")
    c.close()


def test_negative_window_is_rejected(env):
    from paper_2609_38981_b200 import binding as vb
    c = env["cache"]()
    r = env["reqs"][2]
    bt = inputs.block_table_array([env["tables"][2]])
    with pytest.raises(vb.VostiError):
        c.attend_ex(r.q_rows(0, 4), [4], [0], [4], bt, env["scale"], window=-1)
    c.close()


def test_windowed_decode_batch_sampled_against_the_paged_oracle():
    """A decode batch in the shape of the benchmark's workload (smaller pool), window 1000:
    sampled outputs against the oracle's paged front-end."""
    from paper_2609_38981_b200.harness import DeviceCache, bf16_bits
    import gpu_util as gu
    w = inputs.decode_heavy(batch=24, lo=512, hi=4096, num_pages=12_000, seed=5)
    geo = w.geo
    c = DeviceCache(geo, 12_000, max_batch=w.batch, max_total_q=4096, max_seq_len=4096 + 16)
    c.upload(w.requests, w.tables)
    bt = inputs.block_table_array(w.tables)
    out, _ = c.attend_ex(w.packed_q(), w.q_lens, w.start_pos, w.seq_lens, bt, geo.head_dim ** -0.5,
                         window=1000)
    gu.sampled_parity(w, bf16_bits(out), 96, seed=3, window=1000)
    c.close()
