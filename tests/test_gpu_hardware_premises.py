"""The hardware facts the numerical contract rests on, checked on the GPU the suite runs on
(vosti_selftest_mma): tcgen05.mma and mma.sync.m16n8k16 give the same bits for the same
chunk order, in the score form (both operands K-major from shared memory) and in the value
form (weights from tensor memory, values MN-major); an output row depends on its own operand
row only (rows permuted -> outputs permuted); a zero weight contributes exactly nothing,
whatever finite value it multiplies.  The oracle's view of the same product bounds the error."""
import numpy as np
import pytest
import torch

from paper_2609_38981_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2609_38981_b200.harness import DeviceCache
    c = DeviceCache(inputs.TINY, 16, max_batch=1, max_total_q=16, max_seq_len=64)
    yield c
    c.close()


def products(ctx, a, b, mode):
    from paper_2609_38981_b200 import binding as vb
    ad, bd = a.cuda().contiguous(), b.cuda().contiguous()
    d_tc = torch.full((128, 64), float("nan"), device="cuda")
    d_warp = torch.full((128, 64), float("nan"), device="cuda")
    vb.vosti_selftest_mma(ctx.ctx, ad, bd, mode, d_tc, d_warp)
    torch.cuda.synchronize()
    assert vb.vosti_poll_device_status(ctx.ctx) == vb.VOSTI_OK
    return d_tc.cpu(), d_warp.cpu()


def operands(seed, wide):
    g = inputs.generator(seed)
    a = torch.randn(128, 64, generator=g)
    b = torch.randn(64, 64, generator=g)
    if wide:   # wide dynamic range: rows and columns scaled by powers of two over 2^-20 .. 2^20
        a = a * torch.exp2(torch.randint(-20, 21, (128, 1), generator=g).float())
        b = b * torch.exp2(torch.randint(-20, 21, (1, 64), generator=g).float())
    return a.to(torch.bfloat16), b.to(torch.bfloat16)


@pytest.mark.parametrize("mode", (0, 1), ids=("score_form", "value_form"))
@pytest.mark.parametrize("wide", (False, True), ids=("unit_range", "wide_range"))
def test_tensor_memory_mma_and_warp_mma_give_the_same_bits(ctx, mode, wide):
    for seed in (1, 2, 3):
        a, b = operands(seed, wide)
        d_tc, d_warp = products(ctx, a, b, mode)
        assert torch.equal(d_tc.view(torch.int32), d_warp.view(torch.int32)), (mode, wide, seed)
        # and both are the product: fp64 of the exact bf16 operands, fp32 accumulation error only
        ref = a.double() @ (b.double().t() if mode == 0 else b.double())
        scale = (a.double().abs() @ (b.double().abs().t() if mode == 0 else b.double().abs())).clamp_min(1e-30)
        assert float(((d_tc.double() - ref).abs() / scale).max()) < 1e-5


@pytest.mark.parametrize("mode", (0, 1), ids=("score_form", "value_form"))
def test_an_output_row_depends_on_its_own_operand_row_only(ctx, mode):
    a, b = operands(11, True)
    base_tc, base_warp = products(ctx, a, b, mode)
    perm = torch.randperm(128, generator=inputs.generator(5))
    p_tc, p_warp = products(ctx, a[perm].contiguous(), b, mode)
    assert torch.equal(p_tc.view(torch.int32), base_tc[perm].view(torch.int32))
    assert torch.equal(p_warp.view(torch.int32), base_warp[perm].view(torch.int32))
    # other rows replaced by huge values: row 7 keeps its bits
    a2 = (torch.ones_like(a.float()) * 3e38).to(torch.bfloat16)
    a2[7] = a[7]
    q_tc, q_warp = products(ctx, a2, b, mode)
    assert torch.equal(q_tc[7].view(torch.int32), base_tc[7].view(torch.int32))
    assert torch.equal(q_warp[7].view(torch.int32), base_warp[7].view(torch.int32))


def test_a_zero_weight_contributes_exactly_nothing(ctx):
    """Value form: weights of the last 24 keys are zero; what those keys' values are (finite)
    must not matter, and must equal the product with those values set to zero."""
    w, v = operands(21, False)
    w = w.clone()
    w[:, 40:] = 0
    big = v.clone()
    big[40:] = (torch.randn(24, 64, generator=inputs.generator(22)) * 1e30).to(torch.bfloat16)
    zero = v.clone()
    zero[40:] = 0
    neg = v.clone()
    neg[40:] = -v[40:]
    outs = [products(ctx, w, x, 1) for x in (v, big, zero, neg)]
    for d_tc, d_warp in outs[1:]:
        # the sign of an exact zero may differ (0 * negative = -0): compare after adding +0, as the output rule does
        assert torch.equal((d_tc + 0.0).view(torch.int32), (outs[0][0] + 0.0).view(torch.int32))
        assert torch.equal((d_warp + 0.0).view(torch.int32), (outs[0][1] + 0.0).view(torch.int32))
