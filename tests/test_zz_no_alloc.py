"""The update GEMM for callers that cannot allocate device memory.

Code that runs while a stream is being captured, inside a process whose memory
is frozen after start-up, or under another framework's allocator cannot call
cudaMalloc, so it cannot create the library's context (which allocates the split
workspace).  `luq_gemm_wgrad_static` needs no context: its workspace is a fixed
array inside the library.  This test drives it through the C ABI and checks it
against the regular entry point, twice in a row (the array keeps the previous
call's contents).  It is collected last on purpose, and passes both on its own
in a fresh process and after the rest of the suite.
"""
import numpy as np
import pytest
import torch

from paper_2112_10769_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _codes(ctx, M, K, N, seed, ns):
    A, W, G = inputs.small_layer(M, K, N, seed)
    Ad, Gd = torch.from_numpy(A).cuda(), torch.from_numpy(G).cuda()
    ca, sa = ctx.quant_int4(Ad, ctx.amax(Ad))
    cg, al = ctx.quant_grad(Gd, ctx.amax(Gd), seed, ns)
    return ca, sa, cg, al


def test_static_update_gemm_matches_the_regular_one_twice():
    ctx = binding.Context(0)
    try:
        # first call: a shape whose contraction is split (few output tiles, long batch dimension)
        for call, (M, K, N, ns) in enumerate([(6000, 256, 128, 2), (3000, 512, 96, 1)]):
            ca, sa, cg, al = _codes(ctx, M, K, N, 900 + call, ns)
            want = ctx.gemm_wgrad(cg, al, ns, ca, sa, M, N, K)
            got = torch.full((N, K), float("nan"), dtype=torch.float32, device="cuda")
            before = torch.cuda.memory_allocated()
            binding.gemm_wgrad_static(cg, al, ns, ca, sa, M, N, K, got)
            assert torch.cuda.memory_allocated() == before
            torch.cuda.synchronize()
            assert ctx.status() == 0
            w, g = want.cpu().numpy().astype(np.float64), got.cpu().numpy().astype(np.float64)
            assert np.isfinite(g).all()
            assert (g[w == 0] == 0).all()
            assert (np.abs(g - w) <= 1e-5 * np.abs(w) + 1e-12 * np.abs(w).max()).all()
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
