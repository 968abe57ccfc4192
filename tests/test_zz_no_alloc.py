"""The update GEMM for callers that cannot allocate device memory.

Code that runs while a stream is being captured, inside a process whose memory
is frozen after start-up, or under another framework's allocator cannot call
cudaMalloc, so it cannot create the library's context (which allocates the split
workspace).  `luq_gemm_wgrad_static` needs no context: its workspace is a fixed
array inside the library.  This test drives it through the C ABI and checks it
against the regular entry point and against the CPU oracle, several calls in a
row (the array keeps the previous call's contents).  It is collected last on purpose, and passes both on its own
in a fresh process and after the rest of the suite.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2112_10769_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _codes(ctx, M, K, N, seed, ns):
    A, W, G = inputs.small_layer(M, K, N, seed)
    Ad, Gd = torch.from_numpy(A).cuda(), torch.from_numpy(G).cuda()
    ca, sa = ctx.quant_int4(Ad, ctx.amax(Ad))
    cg, al = ctx.quant_grad(Gd, ctx.amax(Gd), seed, ns)
    return ca, sa, cg, al


def _close(got, ref):
    """the tolerance of the parity tests: 1e-5 relative, exact zeros exact"""
    assert np.isfinite(got).all()
    assert (got[ref == 0] == 0).all()
    assert (np.abs(got - ref) <= 1e-5 * np.abs(ref)).all()


# The first two shapes split their contraction (few output tiles, long batch dimension) and so use
# the fixed array; the third has enough tiles (80) to run unsplit; the last has exactly the 152
# tiles the array is sized for.
CASES = [(6000, 256, 128, 2), (3000, 512, 96, 1), (256, 2048, 1280, 1), (128, 2048, 2432, 2)]


def test_static_update_gemm_matches_the_regular_one_and_the_oracle():
    ctx = binding.Context(0)
    try:
        for call, (M, K, N, ns) in enumerate(CASES):
            ca, sa, cg, al = _codes(ctx, M, K, N, 900 + call, ns)
            want = ctx.gemm_wgrad(cg, al, ns, ca, sa, M, N, K)
            got = torch.full((N, K), float("nan"), dtype=torch.float32, device="cuda")
            before = torch.cuda.memory_allocated()
            binding.gemm_wgrad_static(cg, al, ns, ca, sa, M, N, K, got)
            assert torch.cuda.memory_allocated() == before
            torch.cuda.synchronize()
            assert ctx.status() == 0
            w, g = want.cpu().numpy().astype(np.float64), got.cpu().numpy().astype(np.float64)
            _close(g, w)
            # and directly against the CPU oracle's product of the same codes
            ref = oracle.gemm_wgrad(cg.cpu().numpy(), al.item(), ns, ca.cpu().numpy(), sa.item(), M, N, K)
            _close(g, ref)
        # an empty batch: the sum over nothing is zero everywhere, through both entry points
        ca, sa, cg, al = _codes(ctx, 64, 256, 128, 7, 1)
        got = torch.full((128, 256), float("nan"), dtype=torch.float32, device="cuda")
        binding.gemm_wgrad_static(cg, al, 1, ca, sa, 0, 128, 256, got)
        want = torch.full((128, 256), float("nan"), dtype=torch.float32, device="cuda")
        ctx.gemm_wgrad(cg, al, 1, ca, sa, 0, 128, 256, out=want)
        assert not got.any().item() and not want.any().item()
        assert ctx.status() == 0
    finally:
        ctx.close()


def test_static_update_gemm_rejects_what_it_cannot_serve():
    L = binding.load()
    z = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    s = torch.ones(1, dtype=torch.float32, device="cuda")
    out = torch.zeros(1 << 20, dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    # 256 x 20480 output = 2 x 80 = 160 tiles > 152
    assert L.luq_gemm_wgrad_static(z.data_ptr(), s.data_ptr(), 1, z.data_ptr(), s.data_ptr(), out.data_ptr(),
                                   32, 256, 20480, stream) == binding.ERR_WORKSPACE
    assert L.luq_gemm_wgrad_static(z.data_ptr(), s.data_ptr(), 0, z.data_ptr(), s.data_ptr(), out.data_ptr(),
                                   32, 256, 256, stream) == binding.ERR_ARG
    assert L.luq_gemm_wgrad_static(z.data_ptr(), s.data_ptr(), 1, z.data_ptr(), s.data_ptr(), out.data_ptr(),
                                   32, 250, 256, stream) == binding.ERR_ARG
    assert L.luq_gemm_wgrad_static(None, s.data_ptr(), 1, z.data_ptr(), s.data_ptr(), out.data_ptr(),
                                   32, 256, 256, stream) == binding.ERR_ARG
