"""Unsigned INT4 activations (grid 0..15, scale clip/15) through the quantizer and the two GEMMs that
read activation codes.  Codes and operand bytes bit-exact against the oracle; GEMM outputs within 1e-5
of the float64 product of the oracle's dequantized operands."""
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
    c.set_option(binding.OPT_UNSIGNED_ACTIVATIONS, 1)
    yield c
    assert c.status() == 0
    c.close()


@pytest.mark.parametrize("n", [2, 6, 8, 10, 1000, 4098, 65536, (1 << 20) + 2, 3_000_004])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_quant_uint4_bit_exact(ctx, n, dtype):
    x = np.maximum(np.random.default_rng(n).standard_normal(n), 0).astype(np.float32)
    x[n // 2] = np.float32(4.75)
    if n > 8:
        x[3] = np.float32(-1.0)                     # a stray negative value clamps to 0
    if dtype == "bf16":
        x = inputs.to_bf16_bits(x)
    clip, _ = oracle.amax(x)
    want, s_want, _ = oracle.quant_uint4(x, clip)
    xd = to_dev(x)
    ob = torch.full((n + 16,), 0x5A, dtype=torch.int8, device="cuda")
    codes, scale = ctx.quant_uint4(xd, ctx.amax(xd), operand=ob)
    assert scale.item() == s_want
    np.testing.assert_array_equal(codes.cpu().numpy(), want)
    np.testing.assert_array_equal(ob[:n].cpu().numpy(), oracle.unpack(want, n).astype(np.int8))
    assert (ob[n:] == 0x5A).all().item()


def test_quant_uint4_caller_clip_and_specials(ctx):
    y = np.array([-3.0, 0.5, 1.5, 2.5, 14.5, 15.5, 99.0, np.nan, 7.49, 7.51], dtype=np.float32)
    codes, scale = ctx.quant_uint4(to_dev(y), torch.tensor([15.0], device="cuda"))
    want, s_want, _ = oracle.quant_uint4(y, np.float32(15.0))
    assert scale.item() == s_want == 1.0
    np.testing.assert_array_equal(codes.cpu().numpy(), want)
    z = to_dev(np.zeros(1000, dtype=np.float32))
    codes, scale = ctx.quant_uint4(z, ctx.amax(z))
    assert scale.item() == 0 and not codes.any().item()


def reference_products(A, W, G, ca, sa, cw, sw, cg, al, ns):
    M, K = A.shape
    N = W.shape[0]
    return (oracle.gemm_general("fwd", ca, "uint4", sa, 1, cw, "int4", sw, M, N, K),
            oracle.gemm_general("wgrad", cg, "luq", al, ns, ca, "uint4", sa, M, N, K))


@pytest.mark.parametrize("mma_kind", [0, 2])
@pytest.mark.parametrize("M,K,N,ns,with_bytes", [(300, 160, 96, 1, False), (300, 160, 96, 2, True),
                                                 (1024, 1024, 1024, 1, True), (1152, 1056, 800, 2, False)])
def test_forward_and_update_with_unsigned_activations(ctx, M, K, N, ns, with_bytes, mma_kind):
    A, W, G = inputs.small_layer(M, K, N, 300 + M)
    A = np.maximum(A, 0)
    Ad, Wd, Gd = to_dev(A), to_dev(W), to_dev(G)
    ba = torch.empty(M * K, dtype=torch.int8, device="cuda") if with_bytes else None
    ca, sa = ctx.quant_uint4(Ad, ctx.amax(Ad), operand=ba)
    cw, sw = ctx.quant_int4(Wd, ctx.amax(Wd))
    cg, al = ctx.quant_grad(Gd, ctx.amax(Gd), 7, ns)
    oa, osa, _ = oracle.quant_uint4(A, oracle.amax(A)[0])
    np.testing.assert_array_equal(ca.cpu().numpy(), oa)
    assert oracle.unpack(oa, M * K).max() == 15
    ctx.set_option(binding.OPT_MMA_KIND, mma_kind)
    try:
        Z = ctx.gemm_fwd(ca, sa, cw, sw, M, N, K, a_operand=ba)
        dW = ctx.gemm_wgrad(cg, al, ns, ca, sa, M, N, K, a_operand=ba)
    finally:
        ctx.set_option(binding.OPT_MMA_KIND, 2)
    Zr, dWr = reference_products(A, W, G, oa, float(osa), cw.cpu().numpy(), sw.item(),
                                 cg.cpu().numpy().reshape(ns, -1), al.item(), ns)
    assert_gemm_close(Z.cpu().numpy(), Zr)
    assert_gemm_close(dW.cpu().numpy(), dWr)
    # the option matters: read as signed codes the same bytes give another product
    ctx.set_option(binding.OPT_UNSIGNED_ACTIVATIONS, 0)
    Z_signed = ctx.gemm_fwd(ca, sa, cw, sw, M, N, K)
    ctx.set_option(binding.OPT_UNSIGNED_ACTIVATIONS, 1)
    assert not torch.equal(Z_signed, Z)


def test_plane_that_does_not_fit_the_workspace_is_an_error(ctx):
    M, K, N = 50176, 2304, 256                      # 115 MB of activation bytes against 76 MiB of plane room
    ca = torch.zeros(M * K // 2, dtype=torch.uint8, device="cuda")
    cw = torch.zeros(N * K // 2, dtype=torch.uint8, device="cuda")
    one = torch.ones(1, device="cuda")
    with pytest.raises(binding.LuqError) as e:
        ctx.gemm_fwd(ca, one, cw, one, M, N, K)
    assert e.value.code == binding.ERR_WORKSPACE
    ba = torch.zeros(M * K, dtype=torch.int8, device="cuda")
    Z = ctx.gemm_fwd(ca, one, cw, one, M, N, K, a_operand=ba)      # with the caller's bytes it runs
    assert not Z.any().item()
