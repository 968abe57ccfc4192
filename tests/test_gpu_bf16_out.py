"""LUQ_OPT_OUTPUT_BF16: the GEMMs round their fp32 result to bf16 (nearest even) in the epilogue.
The bf16 outputs must be exactly the fp32 outputs rounded once, and within one bf16 rounding
(2^-8 relative) of the CPU oracle's float64 product, exact zeros exact."""
import numpy as np
import pytest
import torch

import oracle
from paper_2112_10769_b200 import binding, inputs

from test_gpu_parity import to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture()
def ctx():
    c = binding.Context(0)
    yield c
    assert c.status() == 0
    c.close()


SHAPES = [
    (128, 128, 256, 1),      # one tile
    (300, 160, 96, 2),       # ragged everywhere, update GEMM split
    (1152, 1056, 800, 1),    # several tiles, operand bytes in use
    (2500, 160, 96, 2),      # long batch: the update GEMM's split partial tiles stay fp32
    (4096, 2304, 256, 1),    # ResNet-like layer
]


@pytest.mark.parametrize("mma_kind", [0, 2])
@pytest.mark.parametrize("M,K,N,ns", SHAPES)
def test_bf16_outputs_are_the_rounded_fp32_outputs(ctx, M, K, N, ns, mma_kind):
    A, W, G = inputs.small_layer(M, K, N, 40 + M)
    Ad, Wd, Gd = to_dev(A), to_dev(W), to_dev(G)
    bw = torch.empty(N * K, dtype=torch.int8, device="cuda")
    bg = torch.empty(ns * M * N, dtype=torch.int8, device="cuda")
    ca, sa = ctx.quant_int4(Ad, ctx.amax(Ad))
    cw, sw = ctx.quant_int4(Wd, ctx.amax(Wd), operand=bw)
    cg, al = ctx.quant_grad(Gd, ctx.amax(Gd), 9, ns, operand=bg)
    ctx.set_option(binding.OPT_MMA_KIND, mma_kind)
    try:
        def products():
            return (ctx.gemm_fwd(ca, sa, cw, sw, M, N, K, w_operand=bw),
                    ctx.gemm_bwd(cg, al, ns, cw, sw, M, N, K, g_operand=bg, w_operand=bw),
                    ctx.gemm_wgrad(cg, al, ns, ca, sa, M, N, K, g_operand=bg))
        full = products()
        ctx.set_option(binding.OPT_OUTPUT_BF16, 1)
        half = products()
    finally:
        ctx.set_option(binding.OPT_OUTPUT_BF16, 0)
        ctx.set_option(binding.OPT_MMA_KIND, 2)
    for f, h in zip(full, half):
        assert f.dtype == torch.float32 and h.dtype == torch.bfloat16 and h.shape == f.shape
        assert torch.equal(h, f.to(torch.bfloat16))
    if M * K * N <= 1152 * 1056 * 800:     # the oracle's triple loops finish in seconds up to here
        oa, ow, og = ca.cpu().numpy(), cw.cpu().numpy(), cg.cpu().numpy()
        refs = (oracle.gemm_fwd(oa, sa.item(), ow, sw.item(), M, N, K),
                oracle.gemm_bwd(og, al.item(), ns, ow, sw.item(), M, N, K),
                oracle.gemm_wgrad(og, al.item(), ns, oa, sa.item(), M, N, K))
        for h, ref in zip(half, refs):
            got = h.float().cpu().numpy().astype(np.float64)
            assert (got[ref == 0] == 0).all()
            assert (np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref)).all()


def test_bf16_output_rows_must_stay_aligned(ctx):
    M, K, N = 128, 64, 100                       # N % 4 == 0 is enough for fp32 rows, not for bf16 rows
    ca = torch.zeros(M * K // 2, dtype=torch.uint8, device="cuda")
    cw = torch.zeros(N * K // 2, dtype=torch.uint8, device="cuda")
    one = torch.ones(1, device="cuda")
    assert not ctx.gemm_fwd(ca, one, cw, one, M, N, K).any().item()
    ctx.set_option(binding.OPT_OUTPUT_BF16, 1)
    with pytest.raises(binding.LuqError):
        ctx.gemm_fwd(ca, one, cw, one, M, N, K)
    with pytest.raises(TypeError):               # the caller's output tensor must have the output type
        ctx.gemm_fwd(ca, one, cw, one, M, 104, K, out=torch.empty(M, 104, device="cuda"))
    ctx.set_option(binding.OPT_OUTPUT_BF16, 0)
