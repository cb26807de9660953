"""Batch-invariant linear layer and RMS normalisation on the GPU.

Parity with the fp64 oracle, and the row-level contract of Sec. "Relational
Kernel Contracts": a token row's output bits are the same whether it runs alone
(M = 1) or at any place in a batch of any size."""
import numpy as np
import pytest
import torch

from paper_2609_38981_b200 import inputs

pytestmark = pytest.mark.gpu

SHAPES = [(256, 64), (128, 192), (384, 512), (1024, 4096), (768, 1024)]     # (N, K): B_N 256, 128, 128, 256, 256
BATCHES = (1, 2, 3, 127, 128, 129, 300, 1000)


def data(N, K, M, seed):
    g = inputs.generator(seed)
    x = inputs.randn_bf16(g, M, K)
    w = (inputs.randn_bf16(g, N, K).float() * K ** -0.5).to(torch.bfloat16)
    return x, w


def widen(t):
    return t.float().double().cpu().numpy()


def workspace(M, N, K):
    """Room for the split schedule (the library decides whether to use it)."""
    from paper_2609_38981_b200 import linear as vl
    return torch.empty(max(vl.vosti_linear_workspace_bytes(M, N, K), 16), dtype=torch.uint8, device="cuda")


@pytest.mark.parametrize("N,K", SHAPES)
def test_linear_parity_with_the_oracle(N, K):
    """fp32 accumulation of exact bf16 products over K terms, one rounding to bf16: the error is
    at most half a bf16 ulp of the result (2^-9 relative) plus the accumulation error, bounded by
    K * 2^-24 * sum|x_k w_k|; checked as |err| <= 2^-8 |ref| + 2^-20 * sum_k |x_k||w_k|."""
    from oracle import linear_oracle as lo
    from paper_2609_38981_b200 import linear as vl
    for M in (1, 130, 517):
        x, w = data(N, K, M, 11)
        y = vl.vosti_linear(x.cuda(), w.cuda(), workspace=workspace(M, N, K) if M != 130 else None)
        ref = lo.linear(inputs.bits(x), inputs.bits(w))
        mag = np.abs(widen(x)) @ np.abs(widen(w)).T
        err = np.abs(widen(y) - ref)
        assert np.isfinite(widen(y)).all()
        assert (err <= 2.0 ** -8 * np.abs(ref) + 2.0 ** -20 * mag).all(), (N, K, M, float(err.max()))
    assert vl.vosti_linear_poll_status() == 0


@pytest.mark.parametrize("N,K", SHAPES)
def test_row_level_contract(N, K):
    """Every row of every batch equals its singleton run bit for bit, wherever it sits, and
    whichever schedule computes it: whole tiles per CTA (no workspace) or the K segments of a
    tile spread over CTAs (workspace given, few row tiles)."""
    from paper_2609_38981_b200 import linear as vl
    from paper_2609_38981_b200.harness import bf16_bits
    x, w = data(N, K, 1000, 12)
    xd, wd = x.cuda(), w.cuda()
    rows = list(range(0, 1000, 37))
    single = torch.cat([bf16_bits(vl.vosti_linear(xd[i:i + 1].contiguous(), wd)) for i in rows])
    single_split = torch.cat([bf16_bits(vl.vosti_linear(xd[i:i + 1].contiguous(), wd, workspace=workspace(1, N, K)))
                              for i in rows])
    assert torch.equal(single, single_split), "the two schedules disagree on a singleton run"
    for M in BATCHES:
        for ws in (None, workspace(M, N, K)):
            y = bf16_bits(vl.vosti_linear(xd[:M].contiguous(), wd, workspace=ws))
            for j, i in enumerate(rows):
                if i < M:
                    assert torch.equal(y[i], single[j]), (N, K, M, i, ws is not None)
    # the same rows in another order and with strangers in between
    perm = torch.randperm(1000, generator=inputs.generator(5))
    y = bf16_bits(vl.vosti_linear(xd[perm.cuda()].contiguous(), wd))
    inv = torch.empty_like(perm)
    inv[perm] = torch.arange(1000)
    for j, i in enumerate(rows):
        assert torch.equal(y[inv[i]], single[j]), (N, K, "permuted", i)


@pytest.mark.parametrize("N,K,n_seg", [(1024, 4096, 4), (512, 2048, 2), (256, 8192, 8), (256, 6144, 6),
                                       (128, 3072, 3), (256, 9216, 9), (768, 1024, 1)])
def test_every_schedule_gives_the_same_bits(N, K, n_seg):
    """The K segments of a tile computed by one CTA in turn (whole tiles), by one CTA each with the
    sums added from a workspace by a second kernel, or by the CTAs of a cluster that add the sums out
    of each other's shared memory (a power of two; 6, 3 and 9 segments, whose column shares are uneven;
    9 is a cluster beyond the portable size): same bits, for a single row, ragged and several row tiles.  A schedule that does not apply
    is refused."""
    from paper_2609_38981_b200 import binding as vb
    from paper_2609_38981_b200 import linear as vl
    from paper_2609_38981_b200.harness import bf16_bits
    assert vl.vosti_linear_segments(N, K) == n_seg
    x, w = data(N, K, 300, 21)
    xd, wd = x.cuda(), w.cuda()
    for M in (1, 5, 128, 200, 300):
        xm = xd[:M].contiguous()
        whole = bf16_bits(vl.vosti_linear(xm, wd, schedule=vl.VOSTI_LINEAR_WHOLE_TILES))
        assert torch.equal(bf16_bits(vl.vosti_linear(xm, wd, workspace=workspace(M, N, K))), whole), (M, "auto")
        assert torch.equal(bf16_bits(vl.vosti_linear(xm, wd)), whole), (M, "auto, no workspace")
        if n_seg > 1:
            y = vl.vosti_linear(xm, wd, workspace=workspace(M, N, K), schedule=vl.VOSTI_LINEAR_SPLIT_WORKSPACE)
            assert torch.equal(bf16_bits(y), whole), (M, "workspace")
        if 2 <= n_seg <= 16:
            y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
            vl.vosti_linear(xm, wd, y, schedule=vl.VOSTI_LINEAR_SPLIT_CLUSTER)
            assert torch.equal(bf16_bits(y), whole), (M, "cluster")
        else:
            with pytest.raises(vb.VostiError):
                vl.vosti_linear(xm, wd, schedule=vl.VOSTI_LINEAR_SPLIT_CLUSTER)
    assert vl.vosti_linear_poll_status() == 0


def test_tile_shape_and_segments_are_functions_of_the_weight_only():
    from paper_2609_38981_b200 import linear as vl
    assert vl.vosti_linear_tile_shape(4096, 4096) == (128, 256, 64)
    assert vl.vosti_linear_tile_shape(384, 64) == (128, 128, 64)
    # floor(148 / column tiles), at most K / 1024, at least 1
    assert vl.vosti_linear_segments(4096, 4096) == 4        # 16 column tiles -> 9, capped by 4096 / 1024
    assert vl.vosti_linear_segments(4096, 14336) == 9       # 144 (column tile, segment) units: one wave of 148 SMs
    assert vl.vosti_linear_segments(28672, 4096) == 1       # 112 column tiles already fill the SMs
    assert vl.vosti_linear_segments(256, 64) == 1
    assert vl.vosti_linear_workspace_bytes(64, 4096, 4096) == 4 * 64 * 4096 * 4


def test_rmsnorm_parity_and_row_independence():
    """Per row: a sum of K squares in fp32 (relative error ~K 2^-24), one correctly rounded
    reciprocal square root, two multiplications and one rounding to bf16: |err| <= 2^-8 |ref| + 1e-6."""
    from oracle import linear_oracle as lo
    from paper_2609_38981_b200 import linear as vl
    from paper_2609_38981_b200.harness import bf16_bits
    g = inputs.generator(3)
    for K in (8, 64, 4096, 5120):
        x = inputs.randn_bf16(g, 300, K)
        x[7] = 0                                      # a zero row: finite thanks to eps
        wgt = (1.0 + 0.1 * inputs.randn_bf16(g, K).float()).to(torch.bfloat16)
        y = vl.vosti_rmsnorm(x.cuda(), wgt.cuda(), 1e-5)
        ref = lo.rmsnorm(inputs.bits(x), inputs.bits(wgt), 1e-5)
        err = np.abs(widen(y) - ref)
        assert np.isfinite(widen(y)).all() and (err <= 2.0 ** -8 * np.abs(ref) + 1e-6).all(), (K, float(err.max()))
        one = torch.cat([bf16_bits(vl.vosti_rmsnorm(x[i:i + 1].cuda(), wgt.cuda(), 1e-5)) for i in (0, 7, 150, 299)])
        full = bf16_bits(y)
        for j, i in enumerate((0, 7, 150, 299)):
            assert torch.equal(full[i], one[j]), (K, i)
    # in place
    xd = inputs.randn_bf16(g, 40, 256).cuda()
    want = bf16_bits(vl.vosti_rmsnorm(xd, wgt[:256].contiguous().cuda(), 1e-6))
    vl.vosti_rmsnorm(xd, wgt[:256].contiguous().cuda(), 1e-6, y=xd)
    assert torch.equal(bf16_bits(xd), want)


def test_argument_checks():
    from paper_2609_38981_b200 import binding as vb, linear as vl
    x = torch.zeros(4, 64, dtype=torch.bfloat16, device="cuda")
    for N, K in ((100, 64), (128, 48)):
        with pytest.raises(vb.VostiError) as e:
            vl.vosti_linear(torch.zeros(4, K, dtype=torch.bfloat16, device="cuda"),
                            torch.zeros(N, K, dtype=torch.bfloat16, device="cuda"))
        assert e.value.status == vb.VOSTI_ERR_UNSUPPORTED_CONFIG
    assert vl.vosti_linear(x[:0].contiguous(), torch.zeros(128, 64, dtype=torch.bfloat16, device="cuda")).shape == (0, 128)


@pytest.mark.parametrize("N,K,M", [(4096, 1024, 4096), (4096, 4096, 3900), (6144, 2048, 2500)])
def test_cta_pair_kernel_gives_the_bits_of_the_single_cta_kernel(N, K, M):
    """Large problems run on CTA pairs (tcgen05.mma cta_group::2, 256 x 256 tiles); small ones on
    single CTAs.  The choice depends on M, so the bits must not: every row of the large call
    equals the same row computed in a call of 128 rows.  Ragged M: the last pair of the second
    shape has 60 rows, so its second CTA owns no row at all."""
    from oracle import linear_oracle as lo
    from paper_2609_38981_b200 import linear as vl
    from paper_2609_38981_b200.harness import bf16_bits
    x, w = data(N, K, M, 13)
    xd, wd = x.cuda(), w.cuda()
    y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    vl.vosti_linear(xd, wd, y)
    assert vl.vosti_linear_poll_status() == 0
    big = bf16_bits(y)
    for r0 in list(range(0, M, 1024)) + [M - 128]:
        part = bf16_bits(vl.vosti_linear(xd[r0:r0 + 128].contiguous(), wd))
        assert torch.equal(big[r0:r0 + 128], part), f"rows {r0}..{r0 + 127} differ between the two kernels"
    rows = [0, 127, 128, 255, 256, M - 1]
    ref = lo.linear(inputs.bits(x[rows]), inputs.bits(w))
    mag = np.abs(widen(x[rows])) @ np.abs(widen(w)).T
    err = np.abs(widen(y[rows]) - ref)
    assert (err <= 2.0 ** -8 * np.abs(ref) + 2.0 ** -20 * mag).all(), float(err.max())
