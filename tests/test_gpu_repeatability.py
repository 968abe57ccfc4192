"""Every product is deterministic: the same call repeated many times, on few fast CTAs and on all of them,
returns the same bits.  The kernels hand shared-memory slots between a copy engine, converter warps and the
tensor core through barriers; a hand-over that let one side overtake the other would show as a result that
differs in some calls (one such case was found this way in the forward kernel that quantizes its
activations, see test_gpu_fused_fwd.py)."""
import pytest
import torch

from paper_2112_10769_b200 import binding, inputs

from test_gpu_parity import to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("limit", [2, 7, 0])
@pytest.mark.parametrize("M,K,N", [(1700, 352, 256), (2048, 1024, 512)])
@pytest.mark.parametrize("with_bytes", [False, True])
def test_products_repeat_bit_for_bit(M, K, N, limit, with_bytes):
    ctx = binding.Context(0)
    try:
        ctx.set_option(binding.OPT_SM_LIMIT, limit)
        A, W, G = inputs.small_layer(M, K, N, 5 + M)
        Ad, Wd, Gd = to_dev(A), to_dev(W), to_dev(G)
        i8 = lambda n: torch.empty(n, dtype=torch.int8, device="cuda") if with_bytes else None  # noqa: E731
        ba, bw, bg = i8(M * K), i8(N * K), i8(2 * M * N)
        ca, sa = ctx.quant_int4(Ad, ctx.amax(Ad), operand=ba)
        cw, sw = ctx.quant_int4(Wd, ctx.amax(Wd), operand=bw)
        cg, al = ctx.quant_grad(Gd, ctx.amax(Gd), 3, 2, operand=bg)
        first = None
        for _ in range(60):
            now = (ctx.gemm_fwd(ca, sa, cw, sw, M, N, K, a_operand=ba, w_operand=bw),
                   ctx.gemm_bwd(cg, al, 2, cw, sw, M, N, K, g_operand=bg, w_operand=bw),
                   ctx.gemm_wgrad(cg, al, 2, ca, sa, M, N, K, g_operand=bg, a_operand=ba))
            if first is None:
                first = tuple(t.clone() for t in now)
            else:
                for name, a, b in zip(("forward", "backward", "update"), first, now):
                    assert torch.equal(a, b), name
        assert ctx.status() == 0
    finally:
        ctx.close()
