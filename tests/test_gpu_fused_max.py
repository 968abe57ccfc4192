"""The fused entry points (max reduction and quantization in one kernel) must give exactly
what the two separate calls give, which in turn are checked against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2112_10769_b200 import binding, inputs

from test_gpu_parity import luq_inputs, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    c.close()


SIZES = [2, 6, 8, 10, 1000, 4098, 65536, (1 << 20) + 2, 3_000_004, 20_000_000]


@pytest.mark.parametrize("n", SIZES)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_fused_int4_matches_oracle(ctx, n, dtype):
    x = np.random.default_rng(n).standard_normal(n).astype(np.float32)
    x[n // 2] = np.float32(-7.25)                       # the maximum sits in the middle, negative
    if dtype == "bf16":
        x = inputs.to_bf16_bits(x)
    mx, _ = oracle.amax(x)
    want, s_want, _ = oracle.quant_int4(x, mx)
    xd = to_dev(x)
    ob = torch.full((n,), 0x5A, dtype=torch.int8, device="cuda")
    for _ in range(2):                                  # twice: the barrier's counters must be left clean
        amax, codes, scale = ctx.amax_quant_int4(xd, operand=ob)
        assert amax.item() == mx and scale.item() == s_want
        np.testing.assert_array_equal(codes.cpu().numpy(), want)
    c2, s2 = ctx.quant_int4(xd, ctx.amax(xd))
    assert torch.equal(c2, codes) and s2.item() == scale.item()
    v = oracle.dequant(want, n, 1.0, "int4") * 16.0
    np.testing.assert_array_equal(ob.cpu().numpy(), v.astype(np.int8))
    assert ctx.status() == 0


@pytest.mark.parametrize("n", SIZES)
@pytest.mark.parametrize("dtype,ns", [("f32", 1), ("f32", 2), ("bf16", 1), ("bf16", 3)])
def test_fused_luq_matches_oracle(ctx, n, dtype, ns):
    x = luq_inputs(n, 600 + n)
    if dtype == "bf16":
        x = inputs.to_bf16_bits(x)
    mx, _ = oracle.amax(x)
    seed = 31 + n
    want, a_want, _ = oracle.quant_luq(x, mx, seed, ns)
    xd = to_dev(x)
    ob = torch.full((ns * n,), 0x5A, dtype=torch.int8, device="cuda")
    for _ in range(2):
        amax, codes, alpha = ctx.amax_quant_grad(xd, seed, ns, operand=ob)
        assert amax.item() == mx and alpha.item() == a_want
        np.testing.assert_array_equal(codes.cpu().numpy().reshape(ns, -1), want)
    got = ob.cpu().numpy().reshape(ns, n)
    for s in range(ns):
        np.testing.assert_array_equal(got[s], oracle.dequant(want[s], n, 1.0, "luq").astype(np.int8))
    assert ctx.status() == 0


def test_fused_special_tensors(ctx):
    z = to_dev(np.zeros(10_000, dtype=np.float32))
    amax, codes, scale = ctx.amax_quant_int4(z)
    assert amax.item() == 0 and scale.item() == 0 and not codes.any().item()
    amax, codes, alpha = ctx.amax_quant_grad(z, 1, 2)
    assert amax.item() == 0 and alpha.item() == 0 and not codes.any().item()
    assert ctx.status() == 0
    x = np.ones(10_000, dtype=np.float32)
    x[777] = np.inf
    amax, codes, scale = ctx.amax_quant_int4(to_dev(x))
    assert np.isinf(amax.item()) and scale.item() == 0 and not codes.any().item()
    assert ctx.status() & binding.STATUS_NONFINITE
    x[777] = np.nan
    amax, codes, alpha = ctx.amax_quant_grad(to_dev(x), 3, 1)
    assert np.isnan(amax.item()) and alpha.item() == 0 and not codes.any().item()
    assert ctx.status() & binding.STATUS_NONFINITE
    # the separate calls still work after the fused ones (shared scratch counters are clean)
    y = to_dev(luq_inputs(100_000, 5))
    c1, a1 = ctx.quant_grad(y, ctx.amax(y), 9, 1)
    _, c2, a2 = ctx.amax_quant_grad(y, 9, 1)
    assert torch.equal(c1, c2) and a1.item() == a2.item()
    assert ctx.status() == 0


def test_fused_and_separate_calls_interleave(ctx):
    """amax, the in-hindsight quantizer and the fused kernels share the context's scratch words."""
    x = luq_inputs(300_000, 12)
    xd = to_dev(x)
    mx = oracle.amax(x)[0]
    for i in range(3):
        assert ctx.amax(xd).item() == mx
        amax, _, _ = ctx.amax_quant_grad(xd, i, 2)
        assert amax.item() == mx
        m_hat = torch.tensor([float(mx)], device="cuda")
        _, _, measured = ctx.quant_grad_hindsight(xd, m_hat, 0.1, i, 1)
        assert measured.item() == mx
        amax, _, _ = ctx.amax_quant_int4(xd)
        assert amax.item() == mx
    assert ctx.status() == 0
