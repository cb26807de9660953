"""Pins for the fp64 CPU oracle: checks against things other than itself.

Closed forms, a hand-worked example, brute-force dense attention written
independently in numpy, a library routine (torch SDPA in fp64), and the
invariances the definition implies.  Each pin is chosen so that a plausible
mistake (dropped scale, wrong sign, off-by-one in the causal position,
transposed operand, wrong KV head) fails at least one of them.
"""
import os

import numpy as np
import pytest
import torch

from oracle import oracle
from paper_2609_38981_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf(x):
    """float array -> bf16 bits (uint16), asserting exact representability."""
    t = torch.as_tensor(np.asarray(x, dtype=np.float32))
    b = t.to(torch.bfloat16)
    assert torch.equal(b.to(torch.float32), t), "test value not exact in bf16"
    return inputs.bits(b)


def widen(bits_arr):
    return inputs.from_bits(bits_arr).to(torch.float64).numpy()


def rand_bits(gen, *shape):
    return inputs.bits(inputs.randn_bf16(gen, *shape))


def brute_force(q, k, v, start, scale):
    """Dense softmax(QK^T + mask)V with an explicit [rows, keys] matrix."""
    qf, kf, vf = widen(q), widen(k), widen(v)
    s, Hq, d = qf.shape
    n, Hkv, _ = kf.shape
    G = Hq // Hkv
    out = np.zeros((s, Hq, d))
    for h in range(Hq):
        kap = h // G
        S = scale * (qf[:, h, :] @ kf[:, kap, :].T)          # [s, n]
        pos = start + np.arange(s)[:, None]
        S = np.where(np.arange(n)[None, :] <= pos, S, -np.inf)
        W = np.exp(S - S.max(axis=1, keepdims=True))
        W /= W.sum(axis=1, keepdims=True)
        out[:, h, :] = W @ vf[:, kap, :]
    return out


# ---------------------------------------------------------------- closed forms

def test_golden_two_key_logistic():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "two_key_logistic.txt"))
            if l.strip() and not l.startswith("#")]
    q = bf([[[1, 0]], [[1, 0]]])
    k = bf([[[0, 0]], [[1, 0]]])
    v = bf([[[1, -2]], [[3, 4]]])
    out = oracle.attention_dense(q, k, v, start=0, scale=1.0)
    for p, o0, o1 in rows:
        np.testing.assert_allclose(out[int(p), 0], [float(o0), float(o1)], rtol=0, atol=1e-15)


def test_single_key_returns_its_value():
    gen = inputs.generator(1)
    q, k, v = rand_bits(gen, 1, 4, 64), rand_bits(gen, 1, 2, 64), rand_bits(gen, 1, 2, 64)
    out = oracle.attention_dense(q, k, v, start=0, scale=0.125)
    vf = widen(v)
    for h in range(4):
        assert np.array_equal(out[0, h], vf[0, h // 2])


def test_identical_keys_give_prefix_mean_of_values():
    gen = inputs.generator(2)
    n = 23
    q = rand_bits(gen, n, 4, 32)
    k1 = rand_bits(gen, 1, 2, 32)
    k = np.repeat(k1, n, axis=0)
    v = rand_bits(gen, n, 2, 32)
    out = oracle.attention_dense(q, k, v, start=0, scale=0.3)
    vf = widen(v)
    for p in range(n):
        for h in range(4):
            np.testing.assert_allclose(out[p, h], vf[:p + 1, h // 2].mean(axis=0), rtol=1e-13,
                                       atol=1e-14)


@pytest.mark.parametrize("start,s", [(0, 19), (7, 12), (18, 1)])
def test_zero_scale_gives_prefix_mean_per_position(start, s):
    """sigma = 0 makes every visible weight equal, so row i must be the mean of
    V[0..start+i]: pins the causal position rule one position at a time."""
    gen = inputs.generator(3)
    n = 19
    q, k, v = rand_bits(gen, s, 2, 16), rand_bits(gen, n, 1, 16), rand_bits(gen, n, 1, 16)
    out = oracle.attention_dense(q, k, v, start=start, scale=0.0)
    vf = widen(v)
    for i in range(s):
        np.testing.assert_allclose(out[i, 0], vf[:start + i + 1, 0].mean(axis=0), rtol=1e-13,
                                   atol=1e-14)


def test_dominant_key_and_no_leak_from_the_future():
    gen = inputs.generator(4)
    n, d, jstar = 12, 64, 7
    q1 = inputs.randn_bf16(gen, 1, 1, d)
    q = inputs.bits(q1.repeat(n, 1, 1))
    k = inputs.randn_bf16(gen, n, 1, d) * 0.25
    k[jstar, 0] = q1[0, 0] * 64              # exact power-of-two scaling
    v = rand_bits(gen, n, 1, d)
    out = oracle.attention_dense(q, inputs.bits(k.to(torch.bfloat16)), v, start=0, scale=0.125)
    vf = widen(v)
    for p in range(n):
        err = np.abs(out[p, 0] - vf[jstar, 0]).max()
        if p >= jstar:
            assert err < 1e-12
        else:
            assert err > 1e-2, "a masked future key leaked into the output"


def test_weights_sum_to_one():
    gen = inputs.generator(5)
    n = 40
    q, k = rand_bits(gen, n, 4, 64), rand_bits(gen, n, 2, 64)
    v = bf(np.ones((n, 2, 64)))
    out = oracle.attention_dense(q, k, v, start=0, scale=0.125)
    np.testing.assert_allclose(out, 1.0, rtol=0, atol=1e-14)


def test_common_score_offset_leaves_output_unchanged():
    """Adding the same vector w to every key shifts every score of a row by
    scale*q.w, which softmax ignores.  Integer data keeps K + w exact in bf16."""
    rng = np.random.default_rng(6)
    n, d = 17, 16
    q = bf(rng.integers(-3, 4, (n, 2, d)))
    k = rng.integers(-4, 5, (n, 1, d))
    w = rng.integers(-3, 4, (1, 1, d))
    v = rand_bits(inputs.generator(6), n, 1, d)
    a = oracle.attention_dense(q, bf(k), v, start=0, scale=0.05)
    b = oracle.attention_dense(q, bf(k + w), v, start=0, scale=0.05)
    np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-13)


def test_query_head_reads_kv_head_h_div_g():
    gen = inputs.generator(7)
    n, Hq, Hkv, d = 9, 8, 2, 16
    q, k = rand_bits(gen, n, Hq, d), rand_bits(gen, n, Hkv, d)
    v = np.zeros((n, Hkv, d))
    for kap in range(Hkv):
        v[:, kap, :] = kap + 1
    out = oracle.attention_dense(q, k, bf(v), start=0, scale=0.25)
    for h in range(Hq):
        np.testing.assert_allclose(out[:, h, :], h // (Hq // Hkv) + 1, rtol=0, atol=1e-14)


# ------------------------------------------------- brute force and library routine

@pytest.mark.parametrize("s,n,start,Hq,Hkv,d", [
    (5, 5, 0, 4, 2, 8), (3, 11, 8, 6, 3, 16), (1, 64, 63, 4, 1, 32), (13, 40, 20, 2, 2, 64),
    (7, 30, 5, 4, 2, 8),      # start + s < n: later keys present but masked
])
def test_against_brute_force_dense(s, n, start, Hq, Hkv, d):
    gen = inputs.generator(100 + s + n)
    q, k, v = rand_bits(gen, s, Hq, d), rand_bits(gen, n, Hkv, d), rand_bits(gen, n, Hkv, d)
    scale = 1.0 / np.sqrt(d)
    out = oracle.attention_dense(q, k, v, start=start, scale=scale)
    np.testing.assert_allclose(out, brute_force(q, k, v, start, scale), rtol=1e-12, atol=1e-13)


def test_against_torch_sdpa_fp64():
    gen = inputs.generator(8)
    s, n, start, Hq, Hkv, d = 9, 33, 24, 8, 2, 64
    q, k, v = rand_bits(gen, s, Hq, d), rand_bits(gen, n, Hkv, d), rand_bits(gen, n, Hkv, d)
    scale = 0.11
    out = oracle.attention_dense(q, k, v, start=start, scale=scale)
    G = Hq // Hkv
    qt = torch.from_numpy(widen(q)).permute(1, 0, 2)                     # [Hq, s, d]
    kt = torch.from_numpy(widen(k)).permute(1, 0, 2).repeat_interleave(G, dim=0)
    vt = torch.from_numpy(widen(v)).permute(1, 0, 2).repeat_interleave(G, dim=0)
    mask = torch.arange(n)[None, :] <= (start + torch.arange(s))[:, None]
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, attn_mask=mask, scale=scale)
    np.testing.assert_allclose(out, ref.permute(1, 0, 2).numpy(), rtol=1e-12, atol=1e-13)


# ---------------------------------------------------------------- paged front-end

def _paged_setup(seed, geo, contexts, num_pages):
    reqs = [inputs.make_request(geo, seed, i, n) for i, n in enumerate(contexts)]
    return reqs


def _fill_pool(geo, num_pages, reqs, tables, garbage_seed=None):
    P, d, Hkv = geo.page_size, geo.head_dim, geo.n_kv_heads
    if garbage_seed is None:
        pool = np.zeros((num_pages, Hkv, 2, P, d), dtype=np.uint16)
    else:
        pool = rand_bits(inputs.generator(garbage_seed), num_pages, Hkv, 2, P, d).copy()
    for r, tab in zip(reqs, tables):                      # logical map, written out by hand
        kb, vb = inputs.bits(r.k), inputs.bits(r.v)
        for j in range(r.n):
            pool[tab[j // P], :, 0, j % P, :] = kb[j]
            pool[tab[j // P], :, 1, j % P, :] = vb[j]
    return pool


def test_paged_equals_dense_under_any_page_placement():
    geo = inputs.TINY
    contexts = (37, 100, 250)
    reqs = _paged_setup(11, geo, contexts, 64)
    scale = geo.head_dim ** -0.5
    dense = [oracle.attention_dense(inputs.bits(r.q), inputs.bits(r.k), inputs.bits(r.v), 0, scale)
             for r in reqs]
    for perm_seed in (0, 1, 2):
        gen = inputs.generator(500 + perm_seed)
        tables = inputs._assign_private_pages(gen, geo, 64, contexts)
        pool = _fill_pool(geo, 64, reqs, tables, garbage_seed=perm_seed or None)
        bt = inputs.block_table_array(tables, stride=24, fill=-1)
        q = inputs.bits(torch.cat([r.q for r in reqs]))
        out = oracle.paged_attention(q, pool, contexts, [0, 0, 0], contexts, bt,
                                     n_kv_heads=geo.n_kv_heads, page_size=geo.page_size,
                                     scale=scale)
        at = 0
        for r, ref in zip(reqs, dense):
            assert np.array_equal(out[at:at + r.n], ref)   # same sums in the same order
            at += r.n


def test_paged_chunking_batch_order_and_selection():
    geo = inputs.TINY
    contexts = (37, 100)
    reqs = _paged_setup(12, geo, contexts, 32)
    tables = inputs._assign_private_pages(inputs.generator(77), geo, 32, contexts)
    pool = _fill_pool(geo, 32, reqs, tables)
    bt = inputs.block_table_array(tables)
    scale = 0.125
    kw = dict(n_kv_heads=geo.n_kv_heads, page_size=geo.page_size, scale=scale)
    full = oracle.paged_attention(inputs.bits(torch.cat([r.q for r in reqs])), pool, contexts,
                                  [0, 0], contexts, bt, **kw)
    # chunk [20, 37) of request 0 with request order swapped, seq_len larger than start+q_len
    q = inputs.bits(torch.cat([reqs[1].q_rows(90, 10), reqs[0].q_rows(20, 10)]))
    part = oracle.paged_attention(q, pool, [10, 10], [90, 20], [100, 37], bt[::-1], **kw)
    assert np.array_equal(part[:10], full[37 + 90:37 + 100])
    assert np.array_equal(part[10:], full[20:30])
    sel = np.array([[1, 3, 2], [0, 9, 0]], dtype=np.int32)
    picked = oracle.paged_attention(q, pool, [10, 10], [90, 20], [100, 37], bt[::-1], sel=sel, **kw)
    assert np.array_equal(picked[0], part[10 + 3, 2]) and np.array_equal(picked[1], part[9, 0])


def test_paged_rejects_bad_metadata():
    geo = inputs.TINY
    pool = np.zeros((4, 2, 2, 16, 64), dtype=np.uint16)
    q = np.zeros((1, 4, 64), dtype=np.uint16)
    kw = dict(n_kv_heads=2, page_size=16, scale=1.0)
    with pytest.raises(ValueError):     # page id out of range
        oracle.paged_attention(q, pool, [1], [0], [1], np.array([[9]], np.int32), **kw)
    with pytest.raises(ValueError):     # start + q_len > seq_len
        oracle.paged_attention(q, pool, [1], [5], [5], np.array([[0]], np.int32), **kw)
    with pytest.raises(ValueError):     # table too short
        oracle.paged_attention(q, pool, [1], [16], [17], np.array([[0]], np.int32), **kw)


# ---------------------------------------------------------------- kv append

def test_kv_append_follows_the_logical_map_and_touches_nothing_else():
    geo = inputs.TINY
    P = geo.page_size
    gen = inputs.generator(21)
    reqs = _paged_setup(21, geo, (45, 18), 16)
    tables = inputs._assign_private_pages(gen, geo, 16, (45, 18))
    bt = inputs.block_table_array(tables, stride=5, fill=-1)
    garbage = rand_bits(gen, 16, geo.n_kv_heads, 2, P, geo.head_dim).copy()
    pool = garbage.copy()
    # two chunks per request: [0,30)+[30,45) and [0,1)+[1,18)
    for starts, lens in (([0, 0], [30, 1]), ([30, 1], [15, 17])):
        k = inputs.bits(torch.cat([r.k[s:s + l] for r, s, l in zip(reqs, starts, lens)]))
        v = inputs.bits(torch.cat([r.v[s:s + l] for r, s, l in zip(reqs, starts, lens)]))
        oracle.kv_append(pool, k, v, lens, starts, bt)
    written = np.zeros(pool.shape, dtype=bool)
    for r, tab in zip(reqs, tables):
        kb, vb = inputs.bits(r.k), inputs.bits(r.v)
        for j in range(r.n):
            assert np.array_equal(pool[tab[j // P], :, 0, j % P, :], kb[j])
            assert np.array_equal(pool[tab[j // P], :, 1, j % P, :], vb[j])
            written[tab[j // P], :, :, j % P, :] = True
    assert np.array_equal(pool[~written], garbage[~written])
    with pytest.raises(ValueError):
        oracle.kv_append(pool, k, v, lens, [70, 1], bt)     # position beyond the table


# ------------------------------------------------- sliding window and log-sum-exp

def brute_force_window(q, k, v, start, scale, window):
    """Dense attention with the window mask written out: p - w < j <= p."""
    qf, kf, vf = widen(q), widen(k), widen(v)
    s, Hq, d = qf.shape
    n, Hkv, _ = kf.shape
    G = Hq // Hkv
    out = np.zeros((s, Hq, d))
    lse = np.zeros((s, Hq))
    pos = start + np.arange(s)[:, None]
    j = np.arange(n)[None, :]
    vis = (j <= pos) & ((j > pos - window) if window > 0 else True)
    for h in range(Hq):
        S = scale * (qf[:, h, :] @ kf[:, h // G, :].T)
        S = np.where(vis, S, -np.inf)
        mx = S.max(axis=1, keepdims=True)
        W = np.exp(S - mx)
        Z = W.sum(axis=1, keepdims=True)
        out[:, h, :] = (W / Z) @ vf[:, h // G, :]
        lse[:, h] = (mx + np.log(Z))[:, 0]
    return out, lse


@pytest.mark.parametrize("window", [1, 2, 5, 16, 17, 1000])
def test_window_against_brute_force_and_lse(window):
    gen = inputs.generator(300 + window)
    s, n, start, Hq, Hkv, d = 11, 29, 18, 4, 2, 16
    q, k, v = rand_bits(gen, s, Hq, d), rand_bits(gen, n, Hkv, d), rand_bits(gen, n, Hkv, d)
    out, lse = oracle.attention_dense(q, k, v, start, 0.21, window=window, return_lse=True)
    ref, ref_lse = brute_force_window(q, k, v, start, 0.21, window)
    np.testing.assert_allclose(out, ref, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(lse, ref_lse, rtol=1e-12, atol=1e-13)


def test_window_closed_forms():
    gen = inputs.generator(31)
    n, d = 21, 8
    q, k, v = rand_bits(gen, n, 2, d), rand_bits(gen, n, 1, d), rand_bits(gen, n, 1, d)
    vf = widen(v)
    # a window of one sees only the key at the row's own position
    out = oracle.attention_dense(q, k, v, 0, 0.4, window=1)
    for p in range(n):
        assert np.array_equal(out[p, 0], vf[p, 0]) and np.array_equal(out[p, 1], vf[p, 0])
    # a window at least as long as the prefix changes nothing
    assert np.array_equal(oracle.attention_dense(q, k, v, 0, 0.4, window=n),
                          oracle.attention_dense(q, k, v, 0, 0.4))
    # sigma = 0: the mean of the last w values, and lse = log(number of visible keys)
    out, lse = oracle.attention_dense(q, k, v, 0, 0.0, window=4, return_lse=True)
    for p in range(n):
        lo = max(0, p - 3)
        np.testing.assert_allclose(out[p, 0], vf[lo:p + 1, 0].mean(axis=0), rtol=1e-13, atol=1e-14)
        np.testing.assert_allclose(lse[p], np.log(p + 1 - lo), rtol=1e-13, atol=1e-14)


def test_lse_against_scipy_logsumexp():
    from scipy.special import logsumexp
    gen = inputs.generator(32)
    n, d = 40, 32
    q, k, v = rand_bits(gen, n, 2, d), rand_bits(gen, n, 2, d), rand_bits(gen, n, 2, d)
    _, lse = oracle.attention_dense(q, k, v, 0, 0.3, return_lse=True)
    qf, kf = widen(q), widen(k)
    for p in (0, 7, 39):
        for h in range(2):
            np.testing.assert_allclose(lse[p, h], logsumexp(0.3 * (kf[:p + 1, h] @ qf[p, h])), rtol=1e-13)


def test_paged_window_equals_dense_window():
    geo = inputs.TINY
    reqs = _paged_setup(41, geo, (90,), 16)
    tables = inputs._assign_private_pages(inputs.generator(41), geo, 16, (90,))
    pool = _fill_pool(geo, 16, reqs, tables, garbage_seed=5)
    r = reqs[0]
    dense, dlse = oracle.attention_dense(inputs.bits(r.q), inputs.bits(r.k), inputs.bits(r.v), 0, 0.125,
                                         window=20, return_lse=True)
    paged, plse = oracle.paged_attention(inputs.bits(r.q), pool, [90], [0], [90],
                                         inputs.block_table_array(tables), n_kv_heads=2, page_size=16,
                                         scale=0.125, window=20, return_lse=True)
    assert np.array_equal(dense, paged) and np.array_equal(dlse, plse)
