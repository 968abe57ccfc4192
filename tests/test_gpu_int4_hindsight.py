"""In-hindsight range for the INT4 tensors (Sec. 7 applied to activations and weights): ONE kernel
quantizes with the clip estimate of earlier steps, measures this tensor's maximum and replaces the
estimate.  Codes, scale, operand bytes, measured maximum and estimate bit-exact against the oracle
over sequences of steps; the forward product on such codes against the oracle's product."""
import numpy as np
import pytest
import torch

import oracle
from paper_2112_10769_b200 import binding, inputs

from test_gpu_parity import assert_gemm_close, scalar, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture()
def ctx():
    c = binding.Context(0)
    yield c
    assert c.status() == 0
    c.close()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("n", [6, 4098, 200_006, (1 << 21) + 2])
def test_sequence_matches_oracle(ctx, dtype, n):
    """Six steps whose scale jumps around: the estimate lags, some steps saturate."""
    eta = 0.1
    scales = [1.0, 0.4, 5.0, 0.05, 2.0, 1.0]
    base = np.random.default_rng(n).standard_normal(n).astype(np.float32)
    first = inputs.to_bf16_bits(base) if dtype == "bf16" else base
    c_hat_o = oracle.amax(first)[0]
    c_hat_d = scalar(float(c_hat_o))
    saturated = 0
    for step, sc in enumerate(scales):
        x = (base * np.float32(sc)).astype(np.float32)
        x[step % n] = np.float32(0.0)
        if dtype == "bf16":
            x = inputs.to_bf16_bits(x)
        want, s_want, fl, meas_want, next_want = oracle.quant_int4_hindsight(x, c_hat_o, eta)
        ob = torch.full((n + 16,), 0x5A, dtype=torch.int8, device="cuda")
        codes, scale, measured = ctx.quant_int4_hindsight(to_dev(x), c_hat_d, eta, operand=ob)
        assert fl == 0 and scale.item() == s_want and measured.item() == meas_want
        assert c_hat_d.item() == next_want
        np.testing.assert_array_equal(codes.cpu().numpy(), want)
        q = oracle.unpack(want, n).astype(np.int64)
        q = np.where(q >= 8, q - 16, q)
        np.testing.assert_array_equal(ob[:n].cpu().numpy(), (16 * q).astype(np.int8))
        assert (ob[n:] == 0x5A).all().item()
        saturated += int(meas_want > c_hat_o)
        c_hat_o = next_want
    assert saturated >= 2
    # without operand bytes: the same codes
    again = scalar(float(c_hat_o))
    c1, _, _ = ctx.quant_int4_hindsight(to_dev(x), again, eta)
    want, _, _, _, _ = oracle.quant_int4_hindsight(x, c_hat_o, eta)
    np.testing.assert_array_equal(c1.cpu().numpy(), want)


def test_unusable_estimate_recovers_and_argument_errors(ctx):
    x = np.random.default_rng(2).standard_normal(50_000).astype(np.float32)
    xd = to_dev(x)
    c_hat = scalar(0.0)
    codes, scale, measured = ctx.quant_int4_hindsight(xd, c_hat, 0.1)
    assert scale.item() == 0 and not codes.any().item()
    assert measured.item() == oracle.amax(x)[0]
    assert c_hat.item() == oracle.hindsight_next(measured.item(), 0.0, 0.1)
    codes, scale, _ = ctx.quant_int4_hindsight(xd, c_hat, 0.1)
    assert scale.item() > 0 and codes.any().item()
    with pytest.raises(binding.LuqError):
        ctx.quant_int4_hindsight(xd, c_hat, -0.5)
    # a non-finite element: reported, wins the measured maximum, codes stay defined
    y = x.copy(); y[7] = np.inf
    c_hat = scalar(1.0)
    codes, scale, measured = ctx.quant_int4_hindsight(to_dev(y), c_hat, 0.1)
    want, _, _ = oracle.quant_int4(y, np.float32(1.0))
    np.testing.assert_array_equal(codes.cpu().numpy(), want)
    assert np.isinf(measured.item()) and ctx.status() == binding.STATUS_NONFINITE


@pytest.mark.parametrize("kind", ["int4", "luq"])
def test_a_non_finite_step_does_not_poison_the_estimate(ctx, kind):
    """Steps [finite, Inf element, finite, finite]: the step with the Inf is flagged and leaves the
    estimate as it was, so the steps after it quantize normally again; estimates, measured maxima and
    codes follow the oracle through the whole sequence."""
    n, eta = 70_002, 0.1
    base = np.random.default_rng(5).standard_normal(n).astype(np.float32)
    est_o = np.float32(np.abs(base).max())
    est_d = scalar(float(est_o))
    for step in range(4):
        x = (base * np.float32(1.0 + 0.1 * step)).astype(np.float32)
        if step == 1:
            x[n // 2] = np.inf
        if kind == "int4":
            want, s_want, fl, meas, nxt = oracle.quant_int4_hindsight(x, est_o, eta)
            codes, scale, measured = ctx.quant_int4_hindsight(to_dev(x), est_d, eta)
        else:
            want, s_want, fl, meas, nxt = oracle.quant_luq_hindsight(x, est_o, eta, seed=step)
            codes, scale, measured = ctx.quant_grad_hindsight(to_dev(x), est_d, eta, step)
        np.testing.assert_array_equal(codes.cpu().numpy().reshape(want.shape), want)
        assert scale.item() == s_want
        assert measured.item() == meas or (np.isinf(meas) and np.isinf(measured.item()))
        assert est_d.item() == nxt and np.isfinite(nxt)
        assert ctx.status() == (binding.STATUS_NONFINITE if step == 1 else 0) == fl
        if step == 1:
            assert nxt == est_o                      # unchanged by the non-finite measurement
        if step >= 2:
            assert codes.any().item()                # quantizing normally again
        est_o = nxt
    # an estimate that is itself unusable is replaced by the first finite measurement
    for bad in (0.0, float("inf"), float("nan")):
        est_d = scalar(bad)
        x = base
        if kind == "int4":
            ctx.quant_int4_hindsight(to_dev(x), est_d, eta)
        else:
            ctx.quant_grad_hindsight(to_dev(x), est_d, eta, 0)
        ctx.status()
        assert est_d.item() == np.abs(base).max() == oracle.hindsight_next(np.abs(base).max(), bad, eta)


def test_forward_product_on_hindsight_codes(ctx):
    M, K, N = 1024, 512, 320
    A, W, _ = inputs.small_layer(M, K, N, 77)
    Ad, Wd = to_dev(A), to_dev(W)
    ca_hat = scalar(float(oracle.amax(A)[0]) * 0.6)          # a lagging estimate: the top saturates
    cw_hat = scalar(float(oracle.amax(W)[0]) * 1.3)
    oa, osa, _, _, _ = oracle.quant_int4_hindsight(A, np.float32(ca_hat.item()), 0.1)
    ow, osw, _, _, _ = oracle.quant_int4_hindsight(W, np.float32(cw_hat.item()), 0.1)
    bw = torch.empty(N * K, dtype=torch.int8, device="cuda")
    ca, sa, _ = ctx.quant_int4_hindsight(Ad, ca_hat, 0.1)
    cw, sw, _ = ctx.quant_int4_hindsight(Wd, cw_hat, 0.1, operand=bw)
    np.testing.assert_array_equal(ca.cpu().numpy(), oa)
    np.testing.assert_array_equal(cw.cpu().numpy(), ow)
    Z = ctx.gemm_fwd(ca, sa, cw, sw, M, N, K, w_operand=bw)
    assert_gemm_close(Z.cpu().numpy(), oracle.gemm_fwd(oa, float(osa), ow, float(osw), M, N, K))
