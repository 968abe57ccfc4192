"""The bounds-checking build of the library (compiled from the same sources with -DLUQ_DEBUG): every
shared-memory, tensor-memory and global address that the converters, epilogues and streaming loops form
is checked against its region, a violation raises LUQ_STATUS_BOUNDS and skips the access.  The pool
this library is developed on offers no compute-sanitizer; this build run over the ragged shapes stands in.
The checking library is loaded in a child process (LUQ_LIB), the normal one stays loaded here."""
import os
import subprocess
import sys

import pytest
import torch

from paper_2112_10769_b200 import binding
from paper_2112_10769_b200 import build as lib_build

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r'''
import numpy as np, torch
import oracle
from paper_2112_10769_b200 import binding, inputs
assert binding.debug_build()
ctx = binding.Context(0)
ctx.debug_bounds_probe()
assert ctx.status() == binding.STATUS_BOUNDS          # the check fires (nothing was accessed)
assert ctx.status() == 0
dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
def close(got, ref):
    got = got.cpu().numpy().astype(np.float64)
    assert (got[ref == 0] == 0).all() and (np.abs(got - ref) <= 1e-5 * np.abs(ref)).all()
# the three products, ragged in every dimension: converters, box and whole-row epilogues, CTA pairs,
# split contraction, both operand types; with and without the quantizers' operand bytes
for (M, K, N, ns), with_bytes in (((300, 160, 96, 1), False), ((130, 416, 544, 2), False), ((1000, 32, 32, 1), True),
                                  ((2500, 160, 96, 2), True), ((1152, 1056, 800, 1), True), ((700, 96, 256, 1), True)):
    A, W, G = inputs.small_layer(M, K, N, 60 + M)
    Ad, Wd, Gd = dev(A), dev(W), dev(G)
    i8 = lambda n: torch.empty(n, dtype=torch.int8, device="cuda") if with_bytes else None
    ba, bw, bg = i8(M * K), i8(N * K), i8(ns * M * N)
    ca, sa = ctx.quant_int4(Ad, ctx.amax(Ad), operand=ba)
    cw, sw = ctx.quant_int4(Wd, ctx.amax(Wd), operand=bw)
    cg, al = ctx.quant_grad(Gd, ctx.amax(Gd), 3, ns, operand=bg)
    for kind in (0, 2):
        ctx.set_option(binding.OPT_MMA_KIND, kind)
        Z = ctx.gemm_fwd(ca, sa, cw, sw, M, N, K, a_operand=ba, w_operand=bw)
        dA = ctx.gemm_bwd(cg, al, ns, cw, sw, M, N, K, g_operand=bg, w_operand=bw)
        dW = ctx.gemm_wgrad(cg, al, ns, ca, sa, M, N, K, g_operand=bg, a_operand=ba)
        assert ctx.status() == 0, (M, K, N, kind)
    ctx.set_option(binding.OPT_MMA_KIND, 2)
    oa, ow, og = ca.cpu().numpy(), cw.cpu().numpy(), cg.cpu().numpy()
    close(Z, oracle.gemm_fwd(oa, sa.item(), ow, sw.item(), M, N, K))
    close(dA, oracle.gemm_bwd(og, al.item(), ns, ow, sw.item(), M, N, K))
    close(dW, oracle.gemm_wgrad(og, al.item(), ns, oa, sa.item(), M, N, K))
    if N <= 256:   # the forward product that quantizes its activations itself
        c2, s2, Z2 = ctx.quant_int4_gemm_fwd(Ad, ctx.amax(Ad), cw, sw, M, N, K, w_operand=bw)
        assert ctx.status() == 0 and torch.equal(c2, ca) and torch.equal(Z2, Z)
# the streaming kernels on ragged sizes, fp32 and bf16
for n in (2, 10, 4098, (1 << 20) + 6, 3_000_004):
    x = inputs.lognormal_gradient((n,), -6.0, 3.0, 0.2, n)
    for xx in (x, inputs.to_bf16_bits(x)):
        xd = dev(xx.view(np.int16)).view(torch.bfloat16) if xx.dtype == np.uint16 else dev(xx)
        mx = ctx.amax(xd)
        c4, _ = ctx.quant_int4(xd, mx)
        cl, _ = ctx.quant_grad(xd, mx, 9, 2)
        assert ctx.status() == 0, n
        assert np.array_equal(c4.cpu().numpy(), oracle.quant_int4(xx, oracle.amax(xx)[0])[0])
        assert np.array_equal(cl.cpu().numpy().reshape(2, -1), oracle.quant_luq(xx, oracle.amax(xx)[0], 9, 2)[0])
ctx.close()
print("checked build ok")
'''


def test_bounds_checking_build_finds_nothing_on_ragged_shapes():
    lib = lib_build.LIB_DEBUG
    if not os.path.exists(lib):
        lib = lib_build.build(debug=True)
    env = dict(os.environ, LUQ_LIB=lib, PYTHONPATH=ROOT + os.pathsep + os.environ.get("PYTHONPATH", ""))
    out = subprocess.run([sys.executable, "-c", CHILD], env=env, cwd=ROOT, capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    assert "checked build ok" in out.stdout


def test_the_normal_build_has_no_checks():
    assert not binding.debug_build()
    ctx = binding.Context(0)
    ctx.debug_bounds_probe()
    assert ctx.status() == 0
    ctx.close()
