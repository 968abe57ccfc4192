"""LUQ_OPT_SUM_SAMPLES: with several samples the quantizer writes ONE operand plane, the sum of the
samples' int8 values, and the backward / update products read it as one sample and divide by the
sample count.  By linearity that is the mean of the per-sample products; everything is exact in the
int32 accumulator, so the codes must stay those of the oracle, the plane must be the sum of the
oracle's per-sample values, and the products must equal the per-sample-plane products bit for bit
(and the oracle's within the usual tolerance)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2112_10769_b200 import binding, inputs

from test_gpu_parity import assert_gemm_close, luq_inputs, to_dev
from test_gpu_operand_bytes import fresh_bytes, want_bytes

pytestmark = pytest.mark.gpu


@pytest.fixture()
def ctx():
    c = binding.Context(0)
    c.set_option(binding.OPT_SUM_SAMPLES, 1)
    yield c
    assert c.status() == 0
    c.close()


@pytest.fixture()
def plain():
    c = binding.Context(0)
    yield c
    c.close()


@pytest.mark.parametrize("n", [2, 6, 10, 1000, 4098, 65536, (1 << 20) + 2, 3_000_004])
@pytest.mark.parametrize("dtype,ns,kmax", [("f32", 2, 4), ("bf16", 2, 4), ("f32", 3, 5), ("bf16", 7, 4), ("f32", 2, 2)])
def test_summed_plane_is_the_sum_of_the_oracle_samples(ctx, n, dtype, ns, kmax):
    x = luq_inputs(n, 8100 + n)
    if n >= 1000:
        x[::7] *= 64.0          # some warps leave the underflow bin: both routes of the kernel
    if dtype == "bf16":
        x = inputs.to_bf16_bits(x)
    ctx.set_option(binding.OPT_LEVELS, kmax)
    mx, _ = oracle.amax(x)
    seed = 4242 + n
    want, a_want, _ = oracle.quant_luq(x, mx, seed, ns, kmax=kmax)
    xd = to_dev(x)
    ob = fresh_bytes(n + 16)
    codes, alpha = ctx.quant_grad(xd, ctx.amax(xd), seed, ns, operand=ob)
    np.testing.assert_array_equal(codes.cpu().numpy().reshape(ns, -1), want)
    assert alpha.item() == a_want
    total = sum(want_bytes(want[s], n, "luq").astype(np.int32) for s in range(ns))
    assert np.abs(total).max() <= 127
    np.testing.assert_array_equal(ob[:n].cpu().numpy(), total.astype(np.int8))
    assert (ob[n:] == 0x5A).all().item()           # one plane, nothing behind it


def test_other_entry_points_write_the_same_plane(ctx):
    n, ns, seed = 200_000, 2, 77
    x = luq_inputs(n, 5)
    xd = to_dev(x)
    ref = fresh_bytes(n)
    c0, a0 = ctx.quant_grad(xd, ctx.amax(xd), seed, ns, operand=ref)
    ob = fresh_bytes(n)
    amax, c1, a1 = ctx.amax_quant_grad(xd, seed, ns, operand=ob)        # fused max + quantizer
    assert torch.equal(c0, c1) and torch.equal(ob, ref) and a0.item() == a1.item()
    est = ctx.amax(xd).clone()
    ob2 = fresh_bytes(n)
    c2, a2, _ = ctx.quant_grad_hindsight(xd, est, 0.1, seed, ns, False, operand=ob2)   # estimate = true maximum
    assert torch.equal(c0, c2) and torch.equal(ob2, ref)


def test_unusable_scale_and_limits(ctx):
    n, ns = 4100, 2
    xd = torch.zeros(n, device="cuda")
    ob = fresh_bytes(n + 8)
    codes, alpha = ctx.quant_grad(xd, ctx.amax(xd), 1, ns, operand=ob)
    assert not codes.any().item() and alpha.item() == 0 and not ob[:n].any().item() and (ob[n:] == 0x5A).all().item()
    # two samples of magnitude 2^6 could sum to 128 and leave int8; the ablation's kernels write one plane per sample
    ctx.set_option(binding.OPT_LEVELS, 6)
    x = to_dev(luq_inputs(n, 3))
    with pytest.raises(binding.LuqError):
        ctx.quant_grad(x, ctx.amax(x), 1, 2, operand=fresh_bytes(n))
    ctx.set_option(binding.OPT_LEVELS, 4)
    with pytest.raises(binding.LuqError):
        ctx.quant_grad_ablation(x, ctx.amax(x), 1, binding.SCHEME_FP4_SR, 2, operand=fresh_bytes(2 * n))
    # without operand bytes, or with one sample, the option changes nothing
    c1, a1 = ctx.quant_grad(x, ctx.amax(x), 9, 2)
    want, a_want, _ = oracle.quant_luq(luq_inputs(n, 3), oracle.amax(luq_inputs(n, 3))[0], 9, 2)
    np.testing.assert_array_equal(c1.cpu().numpy().reshape(2, -1), want)


SHAPES = [(256, 256, 256), (300, 160, 96), (1000, 64, 32), (2048, 256, 2304), (130, 416, 224)]


@pytest.mark.parametrize("M,K,N", SHAPES)
@pytest.mark.parametrize("ns", [2, 3])
def test_products_equal_the_per_sample_products(ctx, plain, M, K, N, ns):
    kmax = 4 if ns == 2 else 5
    ctx.set_option(binding.OPT_LEVELS, kmax); plain.set_option(binding.OPT_LEVELS, kmax)
    A, W, G = inputs.small_layer(M, K, N, 900 + M + N)
    Ad, Wd, Gd = to_dev(A), to_dev(W), to_dev(G)
    seed = 31
    bw, ba = fresh_bytes(N * K), fresh_bytes(M * K)
    cw, sw = ctx.quant_int4(Wd, ctx.amax(Wd), operand=bw)
    ca, sa = ctx.quant_int4(Ad, ctx.amax(Ad), operand=ba)
    one = fresh_bytes(M * N)
    cg, al = ctx.quant_grad(Gd, ctx.amax(Gd), seed, ns, operand=one)
    per = fresh_bytes(ns * M * N)
    cg2, al2 = plain.quant_grad(Gd, plain.amax(Gd), seed, ns, operand=per)
    assert torch.equal(cg, cg2) and al.item() == al2.item()
    dA = ctx.gemm_bwd(cg, al, ns, cw, sw, M, N, K, g_operand=one, w_operand=bw)
    dW = ctx.gemm_wgrad(cg, al, ns, ca, sa, M, N, K, g_operand=one, a_operand=ba)
    dA2 = plain.gemm_bwd(cg, al, ns, cw, sw, M, N, K, g_operand=per, w_operand=bw)
    dW2 = plain.gemm_wgrad(cg, al, ns, ca, sa, M, N, K, g_operand=per, a_operand=ba)
    dA3 = plain.gemm_bwd(cg, al, ns, cw, sw, M, N, K)          # codes only
    assert torch.equal(dA, dA2) and torch.equal(dW, dW2) and torch.equal(dA, dA3)
    og = cg.cpu().numpy().reshape(ns, -1)
    assert_gemm_close(dA.cpu().numpy(), oracle.gemm_bwd(og, al.item(), ns, cw.cpu().numpy(), sw.item(), M, N, K))
    assert_gemm_close(dW.cpu().numpy(), oracle.gemm_wgrad(og, al.item(), ns, ca.cpu().numpy(), sa.item(), M, N, K))
    assert plain.status() == 0


def test_e4m3_operands_refuse_the_summed_plane(ctx):
    M, K, N, ns = 256, 64, 64, 2
    A, W, G = inputs.small_layer(M, K, N, 1)
    Wd, Gd = to_dev(W), to_dev(G)
    cw, sw = ctx.quant_int4(Wd, ctx.amax(Wd))
    one = fresh_bytes(M * N)
    cg, al = ctx.quant_grad(Gd, ctx.amax(Gd), 3, ns, operand=one)
    ctx.set_option(binding.OPT_MMA_KIND, 0)
    try:
        with pytest.raises(binding.LuqError):
            ctx.gemm_bwd(cg, al, ns, cw, sw, M, N, K, g_operand=one)
    finally:
        ctx.set_option(binding.OPT_MMA_KIND, 2)
