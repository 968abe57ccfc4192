"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

Codes are compared bit for bit over the whole tensors (the scalar oracle still
finishes in seconds); GEMM outputs are compared on sampled entries that the
oracle computes one by one from the codes.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2112_10769_b200 import binding, inputs

pytestmark = pytest.mark.gpu
RTOL = 1e-5


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    assert c.status() == 0
    c.close()


def to_dev(a):
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


def sample_entries(rows, cols, count, seed):
    rng = np.random.default_rng(seed)
    r = rng.integers(0, rows, count)
    c = rng.integers(0, cols, count)
    # always include the corners and the last tile's edge
    r[:4] = [0, rows - 1, 0, rows - 1]
    c[:4] = [0, cols - 1, cols - 1, 0]
    return r.astype(np.int64), c.astype(np.int64)


def check_entries(got, ref):
    got = got.astype(np.float64)
    assert (got[ref == 0] == 0).all()
    assert (np.abs(got - ref) <= RTOL * np.abs(ref)).all()


@pytest.mark.parametrize("operand_bytes", [True, False, "timed"])
@pytest.mark.parametrize("name", ["cfg2", "cfg3", "cfg5"])
def test_layer_configs_full_size(ctx, name, operand_bytes):
    """operand_bytes=True: the quantizers also write the 8-bit operand form of W and G (and of A for
    wide layers) and the GEMMs are handed those bytes.  "timed" is the configuration bench.py times:
    the same, and in addition the forward product quantizes A itself where one column of output tiles
    allows it (luq_quant_int4_gemm_fwd) and several samples share one summed operand plane."""
    cfg = inputs.CONFIGS[name]
    M, K, N, ns, seed = cfg.M, cfg.K, cfg.N, cfg.n_samples, cfg.luq_seed
    timed = operand_bytes == "timed"
    fused = timed and N <= 256
    if timed and not fused and ns == 1:
        pytest.skip("the timed configuration of this layer is operand_bytes=True")
    ctx.set_option(binding.OPT_SUM_SAMPLES, 1 if (timed and ns > 1) else 0)   # the context is shared by the module
    A, W, G = inputs.layer_inputs(cfg)
    Ad, Wd, Gd = to_dev(A), to_dev(W), to_dev(G)
    mA, mW, mG = ctx.amax(Ad), ctx.amax(Wd), ctx.amax(Gd)
    i8 = lambda n: torch.empty(n, dtype=torch.int8, device="cuda")  # noqa: E731
    bW = i8(N * K) if operand_bytes else None
    bG = i8((1 if timed else ns) * M * N) if operand_bytes else None
    bA = i8(M * K) if operand_bytes and N >= 1024 else None
    cw, sw = ctx.quant_int4(Wd, mW, operand=bW)
    cg, al = ctx.quant_grad(Gd, mG, seed, ns, operand=bG)
    if fused:
        ca, sa, Z = ctx.quant_int4_gemm_fwd(Ad, mA, cw, sw, M, N, K, w_operand=bW)
    else:
        ca, sa = ctx.quant_int4(Ad, mA, operand=bA)
        Z = ctx.gemm_fwd(ca, sa, cw, sw, M, N, K, a_operand=bA, w_operand=bW)
    dA = ctx.gemm_bwd(cg, al, ns, cw, sw, M, N, K, g_operand=bG, w_operand=bW)
    dW = ctx.gemm_wgrad(cg, al, ns, ca, sa, M, N, K, g_operand=bG, a_operand=bA)
    assert ctx.status() == 0

    # maxima, scales and every code, bit for bit
    oA, oW, oG = oracle.amax(A)[0], oracle.amax(W)[0], oracle.amax(G)[0]
    assert (mA.item(), mW.item(), mG.item()) == (oA, oW, oG)
    oa, osa, _ = oracle.quant_int4(A, oA)
    ow, osw, _ = oracle.quant_int4(W, oW)
    og, oal, _ = oracle.quant_luq(G, oG, seed, ns)
    assert (sa.item(), sw.item(), al.item()) == (osa, osw, oal)
    assert np.array_equal(ca.cpu().numpy(), oa)
    assert np.array_equal(cw.cpu().numpy(), ow)
    assert np.array_equal(cg.cpu().numpy().reshape(ns, -1), og)

    # sampled GEMM outputs
    r, c = sample_entries(M, N, 300, 1)
    check_entries(Z[torch.from_numpy(r).cuda(), torch.from_numpy(c).cuda()].cpu().numpy(),
                  oracle.gemm_entries("fwd", oa, osa, 1, ow, osw, M, N, K, r, c))
    r, c = sample_entries(M, K, 300, 2)
    check_entries(dA[torch.from_numpy(r).cuda(), torch.from_numpy(c).cuda()].cpu().numpy(),
                  oracle.gemm_entries("bwd", og, oal, ns, ow, osw, M, N, K, r, c))
    r, c = sample_entries(N, K, 300, 3)
    check_entries(dW[torch.from_numpy(r).cuda(), torch.from_numpy(c).cuda()].cpu().numpy(),
                  oracle.gemm_entries("wgrad", og, oal, ns, oa, osa, M, N, K, r, c))

    # properties that hold at any size: two samples are two single-sample runs
    if ns == 2:
        c0, _ = ctx.quant_grad(Gd, mG, seed, 1)
        c1, _ = ctx.quant_grad(Gd, mG, seed + 1, 1)
        assert torch.equal(c0[0], cg[0]) and torch.equal(c1[0], cg[1])
        w0 = ctx.gemm_wgrad(c0, al, 1, ca, sa, M, N, K)
        w1 = ctx.gemm_wgrad(c1, al, 1, ca, sa, M, N, K)
        mean = (w0.double() + w1.double()) / 2
        assert torch.allclose(dW.double(), mean, rtol=1e-6, atol=0.0)
    assert ctx.status() == 0


@pytest.mark.parametrize("exponent", [20, 22, 24, 26])
@pytest.mark.parametrize("ns", [1, 2])
def test_quantizer_sweep_sizes(ctx, exponent, ns):
    x = inputs.sweep_tensor(exponent)
    xd = to_dev(x)
    mx = ctx.amax(xd)
    codes, alpha = ctx.quant_grad(xd, mx, 0, ns)
    omx, _ = oracle.amax(x)
    want, oal, _ = oracle.quant_luq(x, omx, 0, ns)
    assert mx.item() == omx and alpha.item() == oal
    assert np.array_equal(codes.cpu().numpy(), want)
    assert ctx.status() == 0


@pytest.mark.parametrize("e", [28, 30])
def test_quantizer_sweep_largest_sizes_windows(ctx, e):
    """2^28 and 2^30 elements (1 and 4 GiB of input): the maximum is checked against numpy, codes
    on windows at the start, in the middle (for 2^30: across the 2^32-byte boundary) and at the end."""
    assert e in inputs.SWEEP_EXPONENTS
    n = 1 << e
    x = inputs.sweep_tensor(e)
    xd = to_dev(x)
    mx = ctx.amax(xd)
    omx = np.abs(x).max()
    assert mx.item() == omx
    codes, alpha = ctx.quant_grad(xd, mx, 0, 2)
    assert alpha.item() == oracle.luq_alpha(omx)
    win = 1 << 18
    for first in (0, n // 2 - win // 2, n - win, 123456 * 8):
        want, _, _ = oracle.quant_luq(x[first:first + win], omx, 0, 2, first_index=first)
        got = codes[:, first // 2:(first + win) // 2].cpu().numpy()
        assert np.array_equal(got, want)
    # whole-tensor property: no code above the top level kmax + 1 anywhere
    for s in range(2):
        plane = codes[s]
        assert int(((plane & 7) > 5).sum().item()) == 0 and int((((plane >> 4) & 7) > 5).sum().item()) == 0
    assert ctx.status() == 0
    del xd, codes
    torch.cuda.empty_cache()


def test_in_hindsight_forward_kernel_full_size(ctx):
    """Config 2's forward half as bench.py's in-hindsight variant runs it: A quantized with a lagging estimate
    inside the forward product, its maximum measured by the same kernel."""
    ctx.set_option(binding.OPT_SUM_SAMPLES, 0)
    cfg = inputs.CONFIGS["cfg2"]
    M, K, N = cfg.M, cfg.K, cfg.N
    A, W, _ = inputs.layer_inputs(cfg)
    Ad, Wd = to_dev(A), to_dev(W)
    bW = torch.empty(N * K, dtype=torch.int8, device="cuda")
    cw, sw = ctx.quant_int4(Wd, ctx.amax(Wd), operand=bW)
    true_max = oracle.amax(A)[0]
    start = np.float32(true_max * np.float32(0.8))          # the estimate lags: the largest values saturate
    est = torch.tensor([start], dtype=torch.float32, device="cuda")
    ca, sa, measured, Z = ctx.quant_int4_hindsight_gemm_fwd(Ad, est, 0.1, cw, sw, M, N, K, w_operand=bW)
    want, s_want, fl, meas_want, next_want = oracle.quant_int4_hindsight(A, start, 0.1)
    assert fl == 0 and meas_want == true_max
    assert (sa.item(), measured.item(), est.item()) == (s_want, meas_want, next_want)
    assert np.array_equal(ca.cpu().numpy(), want)
    ow = cw.cpu().numpy()
    r, c = sample_entries(M, N, 300, 4)
    check_entries(Z[torch.from_numpy(r).cuda(), torch.from_numpy(c).cuda()].cpu().numpy(),
                  oracle.gemm_entries("fwd", want, s_want, 1, ow, sw.item(), M, N, K, r, c))
    assert ctx.status() == 0
