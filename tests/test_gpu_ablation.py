"""The other gradient quantizers of the paper's ablation (Sec. 4): one region of the LUQ grid
deterministic ("FP4", "FP4 + SR", stochastic underflow alone), and the uniform INT4 grid with
stochastic rounding ("INT4 unbiased").  Codes, scale and operand bytes bit-exact against the
oracle; the backward and update products on INT4 gradient codes within 1e-5 of the float64
product of the oracle's dequantized operands."""
import numpy as np
import pytest
import torch

import oracle
from paper_2112_10769_b200 import binding, inputs

from test_gpu_parity import assert_gemm_close, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture()
def ctx():
    c = binding.Context(0)
    yield c
    assert c.status() == 0
    c.close()


def gradient(n, seed, dtype):
    # magnitudes over twelve binades: about a third of the elements lie inside the range
    x = inputs.log_uniform_magnitudes(n, -12, 0, seed)
    if dtype == "bf16":
        x = inputs.to_bf16_bits(x)
    return x


def luq_bytes(codes_plane, n):
    nib = oracle.unpack(codes_plane, n).astype(np.int64)
    c = nib & 7
    mag = np.where(c > 0, 1 << np.maximum(c - 1, 0), 0)
    return np.where(nib & 8, -mag, mag).astype(np.int8)


def int4_bytes(codes_plane, n):
    q = oracle.unpack(codes_plane, n).astype(np.int64)
    q = np.where(q >= 8, q - 16, q)
    return (16 * q).astype(np.int8)


@pytest.mark.parametrize("n", [2, 6, 10, 1000, 4098, 65536, (1 << 20) + 2, 3_000_004])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("scheme", [binding.SCHEME_FP4, binding.SCHEME_FP4_SR, binding.SCHEME_FP4_SU,
                                    binding.SCHEME_LUQ])
def test_partially_unbiased_arms_bit_exact(ctx, n, dtype, scheme):
    ns = 2 if n % 4 == 0 or n > 5000 else 1
    x = gradient(n, 7 * n + scheme, dtype)
    mx, _ = oracle.amax(x)
    sr, su = bool(scheme & 1), bool(scheme & 2)
    want, a_want, _ = oracle.quant_fp_ablation(x, mx, 1234 + n, sr, su, n_samples=ns)
    xd = to_dev(x)
    ob = torch.full((ns * n + 16,), 0x5A, dtype=torch.int8, device="cuda")
    codes, alpha = ctx.quant_grad_ablation(xd, ctx.amax(xd), 1234 + n, scheme, ns, operand=ob)
    assert alpha.item() == a_want
    np.testing.assert_array_equal(codes.cpu().numpy(), want)
    got_bytes = ob.cpu().numpy()
    for s in range(ns):
        np.testing.assert_array_equal(got_bytes[s * n:(s + 1) * n], luq_bytes(want[s], n))
    assert (got_bytes[ns * n:] == 0x5A).all()
    # without operand bytes the codes are the same
    codes2, _ = ctx.quant_grad_ablation(xd, ctx.amax(xd), 1234 + n, scheme, ns)
    assert torch.equal(codes2, codes)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("scheme", [binding.SCHEME_FP4, binding.SCHEME_FP4_SR, binding.SCHEME_FP4_SU,
                                    binding.SCHEME_LUQ])
def test_arms_on_heavy_tailed_gradients(ctx, dtype, scheme):
    """The benchmark's gradient distribution: nearly every warp lies below alpha as a whole and takes
    the kernel's short route, the few others the general one."""
    n, ns = (1 << 21) + 4098, 2
    x = inputs.lognormal_gradient((n,), inputs.SWEEP_MU, inputs.SWEEP_SIGMA, inputs.SWEEP_ZERO_FRAC, 60 + scheme)
    if dtype == "bf16":
        x = inputs.to_bf16_bits(x)
    mx, _ = oracle.amax(x)
    alpha = float(oracle.luq_alpha(mx))
    mag = np.abs(oracle.widen(x))
    per_warp = mag[: n // 128 * 128].reshape(-1, 128).max(axis=1)
    assert 0.5 < (per_warp < alpha).mean() < 1.0                      # both routes are taken
    want, a_want, _ = oracle.quant_fp_ablation(x, mx, 4321, bool(scheme & 1), bool(scheme & 2), n_samples=ns)
    xd = to_dev(x)
    ob = torch.empty(ns * n, dtype=torch.int8, device="cuda")
    codes, al = ctx.quant_grad_ablation(xd, ctx.amax(xd), 4321, scheme, ns, operand=ob)
    assert al.item() == a_want
    np.testing.assert_array_equal(codes.cpu().numpy(), want)
    got_bytes = ob.cpu().numpy()
    for s in range(ns):
        np.testing.assert_array_equal(got_bytes[s * n:(s + 1) * n], luq_bytes(want[s], n))


def test_the_arms_meet_the_library_s_own_quantizers_at_the_ends(ctx):
    """Both regions stochastic is luq_quant_grad, neither is luq_quant_grad_nearest."""
    for dtype in ("f32", "bf16"):
        x = gradient(300_000, 5, dtype)
        xd = to_dev(x)
        mx = ctx.amax(xd)
        luq, a0 = ctx.quant_grad(xd, mx, 99, 2)
        both, a1 = ctx.quant_grad_ablation(xd, mx, 99, binding.SCHEME_LUQ, 2)
        assert torch.equal(luq, both) and a0.item() == a1.item()
        near, _ = ctx.quant_grad_nearest(xd, mx)
        none, _ = ctx.quant_grad_ablation(xd, mx, 99, binding.SCHEME_FP4, 1)
        assert torch.equal(near, none)


@pytest.mark.parametrize("kmax", [2, 6])
def test_arms_on_other_level_counts(ctx, kmax):
    ctx.set_option(binding.OPT_LEVELS, kmax)
    x = gradient(200_000, 40 + kmax, "f32")
    mx, _ = oracle.amax(x)
    xd = to_dev(x)
    for scheme in (binding.SCHEME_FP4_SR, binding.SCHEME_FP4_SU):
        want, a_want, _ = oracle.quant_fp_ablation(x, mx, 8, bool(scheme & 1), bool(scheme & 2), kmax=kmax)
        codes, alpha = ctx.quant_grad_ablation(xd, ctx.amax(xd), 8, scheme)
        assert alpha.item() == a_want
        np.testing.assert_array_equal(codes.cpu().numpy(), want)


@pytest.mark.parametrize("exponent", [-99, -70, -30, 30, 95])
def test_arms_at_extreme_scales(ctx, exponent):
    x = (gradient(50_000, 400 + exponent, "f32").astype(np.float64) * 2.0 ** exponent).astype(np.float32)
    mx, _ = oracle.amax(x)
    xd = to_dev(x)
    for scheme in (binding.SCHEME_FP4_SR, binding.SCHEME_FP4_SU, binding.SCHEME_INT4_SR):
        if scheme == binding.SCHEME_INT4_SR:
            want, s_want, _ = oracle.quant_int4_sr(x, mx, 21)
        else:
            want, s_want, _ = oracle.quant_fp_ablation(x, mx, 21, bool(scheme & 1), bool(scheme & 2))
        codes, scale = ctx.quant_grad_ablation(xd, ctx.amax(xd), 21, scheme)
        assert scale.item() == s_want
        np.testing.assert_array_equal(codes.cpu().numpy(), want)


@pytest.mark.parametrize("n", [2, 6, 10, 1000, 4098, 65536, (1 << 20) + 2, 3_000_004])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_int4_stochastic_rounding_bit_exact(ctx, n, dtype):
    ns = 2 if n % 4 == 0 or n > 5000 else 1
    x = np.random.default_rng(n).standard_normal(n).astype(np.float32)
    if dtype == "bf16":
        x = inputs.to_bf16_bits(x)
    mx, _ = oracle.amax(x)
    want, s_want, _ = oracle.quant_int4_sr(x, mx, 77 + n, n_samples=ns)
    xd = to_dev(x)
    ob = torch.full((ns * n + 16,), 0x5A, dtype=torch.int8, device="cuda")
    codes, scale = ctx.quant_grad_ablation(xd, ctx.amax(xd), 77 + n, binding.SCHEME_INT4_SR, ns, operand=ob)
    assert scale.item() == s_want
    np.testing.assert_array_equal(codes.cpu().numpy(), want)
    got_bytes = ob.cpu().numpy()
    for s in range(ns):
        np.testing.assert_array_equal(got_bytes[s * n:(s + 1) * n], int4_bytes(want[s], n))
    assert (got_bytes[ns * n:] == 0x5A).all()


def test_int4_stochastic_rounding_specials(ctx):
    y = np.array([9.0, -9.0, np.nan, 7.0, -7.0, 0.25, -0.0, 0.0, 3.5, -3.5], dtype=np.float32)
    seven = torch.tensor([7.0], device="cuda")
    for seed in range(8):
        codes, scale = ctx.quant_grad_ablation(to_dev(y), seven, seed, binding.SCHEME_INT4_SR)
        want, s_want, _ = oracle.quant_int4_sr(y, np.float32(7.0), seed)
        assert scale.item() == s_want == 1.0
        np.testing.assert_array_equal(codes.cpu().numpy(), want)
    z = to_dev(np.zeros(1000, dtype=np.float32))
    codes, scale = ctx.quant_grad_ablation(z, ctx.amax(z), 1, binding.SCHEME_INT4_SR)
    assert scale.item() == 0 and not codes.any().item()
    bad = torch.tensor([float("inf")], device="cuda")
    codes, scale = ctx.quant_grad_ablation(to_dev(y), bad, 1, binding.SCHEME_FP4_SR)
    assert scale.item() == 0 and not codes.any().item()
    assert ctx.status() == binding.STATUS_NONFINITE
    with pytest.raises(binding.LuqError):
        ctx.quant_grad_ablation(to_dev(y), seven, 1, 5)


@pytest.mark.parametrize("mma_kind", [0, 2])
@pytest.mark.parametrize("M,K,N,ns,with_bytes", [(300, 160, 96, 1, False), (300, 160, 96, 2, True),
                                                 (1024, 1024, 1024, 1, True), (1152, 1056, 800, 2, False)])
def test_backward_and_update_products_on_int4_gradient_codes(ctx, M, K, N, ns, with_bytes, mma_kind):
    A, W, G = inputs.small_layer(M, K, N, 500 + M)
    Ad, Wd, Gd = to_dev(A), to_dev(W), to_dev(G)
    ca, sa = ctx.quant_int4(Ad, ctx.amax(Ad))
    cw, sw = ctx.quant_int4(Wd, ctx.amax(Wd))
    bg = torch.empty(ns * M * N, dtype=torch.int8, device="cuda") if with_bytes else None
    cg, sg = ctx.quant_grad_ablation(Gd, ctx.amax(Gd), 31, binding.SCHEME_INT4_SR, ns, operand=bg)
    og, osg, _ = oracle.quant_int4_sr(G, oracle.amax(G)[0], 31, n_samples=ns)
    np.testing.assert_array_equal(cg.cpu().numpy(), og)
    ctx.set_option(binding.OPT_GRADIENT_INT4, 1)
    ctx.set_option(binding.OPT_MMA_KIND, mma_kind)
    try:
        dA = ctx.gemm_bwd(cg, sg, ns, cw, sw, M, N, K, g_operand=bg)
        dW = ctx.gemm_wgrad(cg, sg, ns, ca, sa, M, N, K, g_operand=bg)
    finally:
        ctx.set_option(binding.OPT_MMA_KIND, 2)
        ctx.set_option(binding.OPT_GRADIENT_INT4, 0)
    assert_gemm_close(dA.cpu().numpy(), oracle.gemm_general("bwd", og, "int4", float(osg), ns, cw.cpu().numpy(), "int4",
                                                            sw.item(), M, N, K))
    assert_gemm_close(dW.cpu().numpy(), oracle.gemm_general("wgrad", og, "int4", float(osg), ns, ca.cpu().numpy(), "int4",
                                                            sa.item(), M, N, K))
    # the option matters: read as LUQ codes the same nibbles give another product
    dA_luq = ctx.gemm_bwd(cg, sg, ns, cw, sw, M, N, K)
    assert not torch.equal(dA_luq, dA)
